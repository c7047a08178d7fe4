"""ctypes binding of the C-ABI CUDA library declared in ``include/pods.h``.

Argument marshalling only: every function takes torch CUDA tensors (torch is used for device
memory and streams), checks dtypes/contiguity, passes raw pointers and sizes to the library
call of the same name on the current stream, and raises on a non-zero status.  All computation
happens in the library's kernels; there is no CPU or eager fallback, and a missing library is
an error.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# PODS_B200_LIBRARY names another build of the same library (the tests load the checked build through it)
LIB_PATH = os.environ.get("PODS_B200_LIBRARY") or os.path.join(_HERE, "libpods_b200.so")

RULE_MAXVAR, RULE_MAXREWARD, RULE_RANDOM, RULE_PERCENTILE = 0, 1, 2, 3
FLAG_ADV_BEFORE, FLAG_STD_SAMPLE, FLAG_EXACT_TIES = 1, 2, 4
STATUS_NONFINITE_REWARD, STATUS_TOKEN_RANGE, STATUS_CAPACITY, STATUS_NEG_LENGTH, STATUS_TIMEOUT = 1, 2, 4, 8, 16
STATUS_INDEX_RANGE, STATUS_INTERNAL = 32, 64
MAX_N = 1024

# name -> (restype, argtypes); mirrors include/pods.h
_p, _i64, _i32, _u64, _u32, _f32, _sz = (C.c_void_p, C.c_int64, C.c_int32, C.c_uint64, C.c_uint32,
                                         C.c_float, C.c_size_t)
SIGNATURES = {
    "pods_version": (C.c_char_p, []),
    "pods_status_string": (C.c_char_p, [C.c_int]),
    "pods_read_status": (C.c_int, [_p, _p, _p]),
    "pods_select": (C.c_int, [_p, _i64, _i32, _i32, _i32, _u64, _u32, _p, _p, _p, _p, _p]),
    "pods_compact": (C.c_int, [_p, _i64, _i32, _i32, _p, _p, _i64, _p, _i32, _p, _p, _p, _i64, _p, _p]),
    "grpo_seq_weights": (C.c_int, [_p, _p, _i64, _p, _p]),
    "grpo_loss_chunk_workspace_bytes": (_sz, [_i64]),
    "grpo_loss_chunk": (C.c_int, [_p, _i64, _p, _p, _p, _p, _p, _p, _i64, _i64, _p, _i64, _i32, _f32, _f32,
                                  _f32, _p, _p, _p, _i64, _p, _sz, _p, _p]),
    "grpo_loss_chunk_static_max_rows": (_i64, []),
    "grpo_loss_chunk_static": (C.c_int, [_p, _i64, _p, _p, _p, _p, _p, _p, _i64, _i64, _p, _i64, _i32, _f32, _f32,
                                         _f32, _p, _p, _p, _i64, _p, _p]),
    "grpo_loss_workspace_bytes": (_sz, [_i64, _i64, _i64]),
    "grpo_loss_fwd_bwd": (C.c_int, [_p, _i64, _p, _p, _p, _p, _p, _i64, _p, _i64, _i32, _f32, _f32, _i64,
                                    _p, _p, _p, _i64, _p, _sz, _p, _p]),
    "grpo_loss_finalize": (C.c_int, [_p, _p, _p]),
    "grpo_logp_from_hidden_workspace_bytes": (_sz, [_i64, _i32, _i32]),
    "grpo_logp_from_hidden": (C.c_int, [_p, _i64, _p, _i64, _p, _i64, _i32, _i32, _p, _p, _p, _sz, _p, _p]),
    "grpo_loss_from_hidden_workspace_bytes": (_sz, [_i64, _i32, _i32]),
    "pods_set_loss_from_hidden_panel_bytes": (_sz, [_sz]),
    "grpo_loss_from_hidden": (C.c_int, [_p, _i64, _p, _i64, _p, _p, _p, _p, _p, _p, _i64, _i64, _p, _i64, _i32, _i32,
                                        _f32, _f32, _f32, _p, _p, _p, _i64, _p, _i64, _p, _sz, _p, _p]),
    "pods_selftest_bounded_wait": (C.c_int, [_u32, _p, _p]),
    "pods_set_loss_cluster_min_vocab": (_i32, [_i32]),
    "pods_host_step_create": (C.c_int, [_i64, _i32, _i32, _i64, _i64, _i32, _i64, _p]),
    "pods_host_step_run": (C.c_int, [_p, _p, _p, _p, _p, _p, _p, _i64, _f32, _f32, _i32, _u64, _u32,
                                     _p, _p, _p, _p, _p, _p]),
    "pods_host_step_dlogits": (_p, [_p]),
    "pods_host_step_destroy": (C.c_int, [_p]),
}

_lib = None


class PodsError(RuntimeError):
    pass


def load():
    """Load libpods_b200.so (built in-tree by csrc/build.py).  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise PodsError("CUDA library %s is missing: run `python -m paper_2504_13818_b200.csrc.build` "
                        "(there is no CPU fallback)" % LIB_PATH)
    lib = C.CDLL(LIB_PATH)
    for name, (res, args) in SIGNATURES.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


def _check(rc, what):
    if rc != 0:
        raise PodsError("%s failed: %s (status %d)" % (what, load().pods_status_string(rc).decode(), rc))


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev(t, dtype, name, optional=False):
    if t is None:
        if optional:
            return None
        raise PodsError("%s is required" % name)
    if not (isinstance(t, torch.Tensor) and t.is_cuda):
        raise PodsError("%s must be a CUDA tensor" % name)
    if t.dtype != dtype:
        raise PodsError("%s must have dtype %s, got %s" % (name, dtype, t.dtype))
    if not t.is_contiguous():
        raise PodsError("%s must be contiguous" % name)
    return C.c_void_p(t.data_ptr())


def _require(cond, message):
    if not cond:
        raise PodsError(message)


def _numel(t, count, name):
    """The C ABI sees pointers only: a short buffer would be read or written past its end on the device,
    so every length is checked here, before the call."""
    _require(t is None or t.numel() == count, "%s must hold %d entries, got %d" % (name, count, 0 if t is None else t.numel()))


def _check_loss_shapes(logits, dlogits, tokens, old_logp, ref_logp, adv, seq_weight, cu_seqlens, mask, logp):
    _require(isinstance(logits, torch.Tensor) and logits.dim() == 2, "logits must be [T,V]")
    T = logits.shape[0]
    _require(tuple(dlogits.shape) == tuple(logits.shape), "dlogits must have the shape of logits %s, got %s"
             % (tuple(logits.shape), tuple(dlogits.shape)))
    M = cu_seqlens.numel() - 1
    _require(M >= 1, "cu_seqlens must hold M+1 >= 2 entries")
    for t, name in ((tokens, "tokens"), (old_logp, "old_logp"), (ref_logp, "ref_logp"), (mask, "mask"), (logp, "logp")):
        _numel(t, T, name)
    _numel(adv, M, "adv")
    _numel(seq_weight, M, "seq_weight")


def _rows(t, name):
    """Pointer and row pitch of a 2-D bf16 tensor whose rows are contiguous."""
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.bfloat16 and t.dim() == 2):
        raise PodsError("%s must be a 2-D CUDA bfloat16 tensor" % name)
    if t.stride(1) != 1:
        raise PodsError("%s rows must be contiguous" % name)
    return C.c_void_p(t.data_ptr()), (t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1]))


def version() -> str:
    return load().pods_version().decode()


def new_status(device=None):
    return torch.zeros(1, dtype=torch.int32, device=device or "cuda")


def read_status(status) -> int:
    out = C.c_uint32(0)
    _check(load().pods_read_status(_dev(status, torch.int32, "status"), C.byref(out), _stream()), "pods_read_status")
    return int(out.value)


def pods_select(rewards, m, rule=RULE_MAXVAR, seed=0, flags=0, status=None, want_k=True):
    """rewards [G,n] fp32 -> (idx [G,m] int32, adv [G,m] fp32, k [G] int32 or None)."""
    rp = _dev(rewards, torch.float32, "rewards")
    if rewards.dim() != 2:
        raise PodsError("rewards must be [G,n]")
    G, n = rewards.shape
    _require(1 <= m <= n, "need 1 <= m <= n, got m=%d n=%d" % (m, n))
    idx = torch.empty((G, m), dtype=torch.int32, device=rewards.device)
    adv = torch.empty((G, m), dtype=torch.float32, device=rewards.device)
    k = torch.empty((G,), dtype=torch.int32, device=rewards.device) if want_k else None
    rc = load().pods_select(rp, G, n, m, rule, seed, flags, C.c_void_p(idx.data_ptr()), C.c_void_p(adv.data_ptr()),
                            C.c_void_p(k.data_ptr()) if want_k else None,
                            _dev(status, torch.int32, "status", True), _stream())
    _check(rc, "pods_select")
    return idx, adv, k


def pods_select_into(rewards, m, idx, adv, k=None, rule=RULE_MAXVAR, seed=0, flags=0, status=None):
    """As pods_select with caller-provided outputs (no allocation)."""
    _require(isinstance(rewards, torch.Tensor) and rewards.dim() == 2, "rewards must be [G,n]")
    G, n = rewards.shape
    _require(1 <= m <= n, "need 1 <= m <= n, got m=%d n=%d" % (m, n))
    _numel(idx, G * m, "idx")
    _numel(adv, G * m, "adv")
    _numel(k, G, "k")
    rc = load().pods_select(_dev(rewards, torch.float32, "rewards"), G, n, m, rule, seed, flags,
                            _dev(idx, torch.int32, "idx"), _dev(adv, torch.float32, "adv"),
                            _dev(k, torch.int32, "k", True), _dev(status, torch.int32, "status", True), _stream())
    _check(rc, "pods_select")


def pods_compact(idx, n, lengths, src_tokens, src_f32=(), T_cap=None, status=None, out=None):
    """Pack the kept rollouts.  Returns (cu_seqlens int64 [M+1], tokens int32 [T_cap], [fp32 streams]).

    ``T_cap`` defaults to M * src_ld (always enough).  ``out`` may carry pre-allocated
    (cu_seqlens, tokens, [streams]) to write into.
    """
    G, m = idx.shape
    src_ld = src_tokens.shape[1]
    M = G * m
    if T_cap is None:
        T_cap = M * src_ld
    dev = idx.device
    if out is None:
        cu = torch.empty(M + 1, dtype=torch.int64, device=dev)
        toks = torch.empty(T_cap, dtype=torch.int32, device=dev)
        dst = [torch.empty(T_cap, dtype=torch.float32, device=dev) for _ in src_f32]
    else:
        cu, toks, dst = out
    _require(idx.dim() == 2 and src_tokens.dim() == 2, "idx must be [G,m] and src_tokens [G*n, src_ld]")
    _require(1 <= m <= n, "need 1 <= m <= n, got m=%d n=%d" % (m, n))
    _numel(lengths, G * n, "lengths")
    _require(src_tokens.shape[0] == G * n, "src_tokens must have G*n = %d rows, got %d" % (G * n, src_tokens.shape[0]))
    _numel(cu, M + 1, "cu_seqlens")
    _require(toks.numel() >= T_cap, "dst_tokens must hold T_cap = %d entries, got %d" % (T_cap, toks.numel()))
    _require(len(dst) == len(src_f32), "one destination stream per source stream")
    for d in dst:
        _require(d.numel() >= T_cap, "dst_f32 streams must hold T_cap = %d entries, got %d" % (T_cap, d.numel()))
    k = len(src_f32)
    src_arr = (C.c_void_p * max(k, 1))(*[_dev(s, torch.float32, "src_f32").value for s in src_f32])
    dst_arr = (C.c_void_p * max(k, 1))(*[_dev(d, torch.float32, "dst_f32").value for d in dst])
    for s in src_f32:
        if tuple(s.shape) != tuple(src_tokens.shape):
            raise PodsError("src_f32 streams must have the shape of src_tokens")
    rc = load().pods_compact(_dev(idx, torch.int32, "idx"), G, n, m, _dev(lengths, torch.int32, "lengths"),
                             _dev(src_tokens, torch.int32, "src_tokens"), src_ld,
                             C.cast(src_arr, C.c_void_p) if k else None, k,
                             _dev(cu, torch.int64, "cu_seqlens"), _dev(toks, torch.int32, "dst_tokens"),
                             C.cast(dst_arr, C.c_void_p) if k else None, T_cap,
                             _dev(status, torch.int32, "status", True), _stream())
    _check(rc, "pods_compact")
    return cu, toks, dst


def grpo_seq_weights(mask, cu_seqlens, out=None):
    M = cu_seqlens.shape[0] - 1
    w = out if out is not None else torch.empty(M, dtype=torch.float64, device=cu_seqlens.device)
    _require(M >= 1, "cu_seqlens must hold M+1 >= 2 entries")
    _numel(w, M, "seq_weight")
    rc = load().grpo_seq_weights(_dev(mask, torch.uint8, "mask", True), _dev(cu_seqlens, torch.int64, "cu_seqlens"),
                                 M, _dev(w, torch.float64, "seq_weight"), _stream())
    _check(rc, "grpo_seq_weights")
    return w


def grpo_loss_chunk_workspace_bytes(T_chunk) -> int:
    return int(load().grpo_loss_chunk_workspace_bytes(T_chunk))


def grpo_loss_workspace_bytes(T, M, chunk_rows=0) -> int:
    return int(load().grpo_loss_workspace_bytes(T, M, chunk_rows))


def grpo_loss_chunk(logits, tokens, old_logp, ref_logp, adv, seq_weight, cu_seqlens, row0, mask, eps, beta,
                    loss_acc, logp, dlogits, workspace, grad_scale=1.0, status=None):
    """One chunk of rows [row0, row0+T_chunk).  Per-token tensors hold this chunk's rows only."""
    _check_loss_shapes(logits, dlogits, tokens, old_logp, ref_logp, adv, seq_weight, cu_seqlens, mask, logp)
    _numel(loss_acc, 1, "loss_acc")
    lp, ldl = _rows(logits, "logits")
    dp, ldd = _rows(dlogits, "dlogits")
    T, V = logits.shape
    rc = load().grpo_loss_chunk(lp, ldl, _dev(tokens, torch.int32, "tokens"), _dev(old_logp, torch.float32, "old_logp"),
                                _dev(ref_logp, torch.float32, "ref_logp", True), _dev(adv.reshape(-1), torch.float32, "adv"),
                                _dev(seq_weight, torch.float64, "seq_weight"), _dev(cu_seqlens, torch.int64, "cu_seqlens"),
                                cu_seqlens.shape[0] - 1, row0, _dev(mask, torch.uint8, "mask", True), T, V,
                                eps, beta, grad_scale, _dev(loss_acc, torch.float64, "loss_acc"),
                                _dev(logp, torch.float32, "logp"), dp, ldd,
                                _dev(workspace, torch.uint8, "workspace"), workspace.numel(),
                                _dev(status, torch.int32, "status", True), _stream())
    _check(rc, "grpo_loss_chunk")


def grpo_loss_chunk_static_max_rows() -> int:
    return int(load().grpo_loss_chunk_static_max_rows())


def grpo_loss_chunk_static(logits, tokens, old_logp, ref_logp, adv, seq_weight, cu_seqlens, row0, mask, eps, beta,
                           loss_acc, logp, dlogits, grad_scale=1.0, status=None):
    """grpo_loss_chunk for callers that may not allocate: no workspace, the scratch is inside the library.

    At most grpo_loss_chunk_static_max_rows() rows per call; calls on one device share the scratch, so
    they must not overlap on the GPU.  This wrapper itself creates no tensor."""
    _check_loss_shapes(logits, dlogits, tokens, old_logp, ref_logp, adv, seq_weight, cu_seqlens, mask, logp)
    _numel(loss_acc, 1, "loss_acc")
    lp, ldl = _rows(logits, "logits")
    dp, ldd = _rows(dlogits, "dlogits")
    T, V = logits.shape
    rc = load().grpo_loss_chunk_static(lp, ldl, _dev(tokens, torch.int32, "tokens"),
                                       _dev(old_logp, torch.float32, "old_logp"),
                                       _dev(ref_logp, torch.float32, "ref_logp", True),
                                       _dev(adv.reshape(-1), torch.float32, "adv"),
                                       _dev(seq_weight, torch.float64, "seq_weight"),
                                       _dev(cu_seqlens, torch.int64, "cu_seqlens"), cu_seqlens.shape[0] - 1, row0,
                                       _dev(mask, torch.uint8, "mask", True), T, V, eps, beta, grad_scale,
                                       _dev(loss_acc, torch.float64, "loss_acc"), _dev(logp, torch.float32, "logp"),
                                       dp, ldd, _dev(status, torch.int32, "status", True), _stream())
    _check(rc, "grpo_loss_chunk_static")


def set_loss_cluster_min_vocab(min_vocab) -> int:
    """Rows of V >= min_vocab take the cluster-resident loss kernel; returns the previous setting."""
    return int(load().pods_set_loss_cluster_min_vocab(int(min_vocab)))


def selftest_bounded_wait(polls, status):
    """A wait on a barrier that nothing completes: must end by itself and set STATUS_TIMEOUT in ``status``."""
    _check(load().pods_selftest_bounded_wait(polls, _dev(status, torch.int32, "status"), _stream()),
           "pods_selftest_bounded_wait")


def grpo_loss_finalize(loss_acc, loss):
    _check(load().grpo_loss_finalize(_dev(loss_acc, torch.float64, "loss_acc"), _dev(loss, torch.float32, "loss"),
                                     _stream()), "grpo_loss_finalize")


def grpo_loss_fwd_bwd(logits, tokens, old_logp, ref_logp, adv, mask, eps, beta, cu_seqlens, chunk_rows=0,
                      dlogits=None, logp=None, loss=None, workspace=None, status=None):
    """(logits, tokens, old_logp, ref_logp, adv, mask, eps, beta) -> (loss [1] fp32, logp [T] fp32, dlogits).

    ``dlogits`` may be ``logits`` itself (in place).  Missing outputs / workspace are allocated here.
    """
    T, V = logits.shape
    M = cu_seqlens.shape[0] - 1
    dev = logits.device
    if dlogits is None:
        dlogits = torch.empty_like(logits)
    if logp is None:
        logp = torch.empty(T, dtype=torch.float32, device=dev)
    if loss is None:
        loss = torch.empty(1, dtype=torch.float32, device=dev)
    need = grpo_loss_workspace_bytes(T, M, chunk_rows)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    _check_loss_shapes(logits, dlogits, tokens, old_logp, ref_logp, adv, None, cu_seqlens, mask, logp)
    _numel(loss, 1, "loss")
    _require(workspace.numel() >= need, "workspace must hold %d bytes, got %d" % (need, workspace.numel()))
    lp, ldl = _rows(logits, "logits")
    dp, ldd = _rows(dlogits, "dlogits")
    rc = load().grpo_loss_fwd_bwd(lp, ldl, _dev(tokens, torch.int32, "tokens"), _dev(old_logp, torch.float32, "old_logp"),
                                  _dev(ref_logp, torch.float32, "ref_logp", True),
                                  _dev(adv.reshape(-1), torch.float32, "adv"),
                                  _dev(cu_seqlens, torch.int64, "cu_seqlens"), M,
                                  _dev(mask, torch.uint8, "mask", True), T, V, eps, beta, chunk_rows,
                                  _dev(loss, torch.float32, "loss"), _dev(logp, torch.float32, "logp"), dp, ldd,
                                  _dev(workspace, torch.uint8, "workspace"), workspace.numel(),
                                  _dev(status, torch.int32, "status", True), _stream())
    _check(rc, "grpo_loss_fwd_bwd")
    return loss, logp, dlogits


def grpo_logp_from_hidden_workspace_bytes(T, V, d) -> int:
    return int(load().grpo_logp_from_hidden_workspace_bytes(T, V, d))


def grpo_logp_from_hidden(hidden, W, tokens, logp=None, lse=None, want_lse=False, workspace=None, status=None):
    """hidden [T,d] bf16, W [V,d] bf16, tokens [T] int32 -> (logp [T] fp32, lse [T] fp32 or None).

    log softmax(hidden W^T)[token] without the logits ever being stored.  Missing outputs and the workspace
    are allocated here; rows of hidden and W may have a pitch (a column slice of a wider tensor)."""
    _require(isinstance(hidden, torch.Tensor) and hidden.dim() == 2 and isinstance(W, torch.Tensor) and W.dim() == 2,
             "hidden must be [T,d] and W [V,d]")
    T, d = hidden.shape
    V = W.shape[0]
    _require(W.shape[1] == d, "W must have d = %d columns, got %d" % (d, W.shape[1]))
    _numel(tokens, T, "tokens")
    dev = hidden.device
    if logp is None:
        logp = torch.empty(T, dtype=torch.float32, device=dev)
    if lse is None and want_lse:
        lse = torch.empty(T, dtype=torch.float32, device=dev)
    _numel(logp, T, "logp")
    _numel(lse, T, "lse")
    need = grpo_logp_from_hidden_workspace_bytes(T, V, d)
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
    _require(workspace.numel() >= need, "workspace must hold %d bytes, got %d" % (need, workspace.numel()))
    hp, ldh = _rows(hidden, "hidden")
    wp, ldw = _rows(W, "W")
    rc = load().grpo_logp_from_hidden(hp, ldh, wp, ldw, _dev(tokens, torch.int32, "tokens"), T, V, d,
                                      _dev(logp, torch.float32, "logp"), _dev(lse, torch.float32, "lse", True),
                                      _dev(workspace, torch.uint8, "workspace"), workspace.numel(),
                                      _dev(status, torch.int32, "status", True), _stream())
    _check(rc, "grpo_logp_from_hidden")
    return logp, lse


def grpo_loss_from_hidden_workspace_bytes(T, V, d) -> int:
    return int(load().grpo_loss_from_hidden_workspace_bytes(T, V, d))


def set_loss_from_hidden_panel_bytes(nbytes) -> int:
    """Limit of the gradient panel grpo_loss_from_hidden keeps in its workspace; returns the previous setting."""
    return int(load().pods_set_loss_from_hidden_panel_bytes(int(nbytes)))


def _f32_rows(t, rows, cols, name):
    """Pointer and row pitch of a 2-D fp32 CUDA tensor [rows, cols] whose rows are contiguous."""
    _require(isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.float32 and t.dim() == 2 and
             tuple(t.shape) == (rows, cols) and t.stride(1) == 1,
             "%s must be a CUDA float32 tensor [%d, %d] with contiguous rows" % (name, rows, cols))
    return C.c_void_p(t.data_ptr()), (t.stride(0) if rows > 1 else max(t.stride(0), cols))


def grpo_loss_from_hidden(hidden, W, tokens, old_logp, ref_logp, adv, seq_weight, cu_seqlens, row0, mask, eps, beta,
                          loss_acc, dW, logp=None, dhidden=None, workspace=None, grad_scale=1.0, status=None):
    """Rows [row0, row0+T) of the objective on logits = hidden W^T, with dhidden (written) and dW (added to).

    hidden [T,d] bf16, W [V,d] bf16; loss_acc [1] fp64 and dW [V,d] fp32 accumulate (the caller zeroes them before
    the first chunk).  Returns (logp [T] fp32, dhidden [T,d] fp32); missing ones and the workspace are allocated here."""
    _require(isinstance(hidden, torch.Tensor) and hidden.dim() == 2 and isinstance(W, torch.Tensor) and W.dim() == 2,
             "hidden must be [T,d] and W [V,d]")
    T, d = hidden.shape
    V = W.shape[0]
    _require(W.shape[1] == d, "W must have d = %d columns, got %d" % (d, W.shape[1]))
    M = cu_seqlens.shape[0] - 1
    dev = hidden.device
    if logp is None:
        logp = torch.empty(T, dtype=torch.float32, device=dev)
    if dhidden is None:
        dhidden = torch.empty((T, d), dtype=torch.float32, device=dev)
    for t, name in ((tokens, "tokens"), (old_logp, "old_logp"), (ref_logp, "ref_logp"), (mask, "mask"), (logp, "logp")):
        _numel(t, T, name)
    _numel(adv, M, "adv")
    _numel(seq_weight, M, "seq_weight")
    _numel(loss_acc, 1, "loss_acc")
    _require(isinstance(dhidden, torch.Tensor) and tuple(dhidden.shape) == (T, d), "dhidden must have the shape [%d, %d]" % (T, d))
    _require(isinstance(dW, torch.Tensor) and tuple(dW.shape) == (V, d), "dW must have the shape [%d, %d]" % (V, d))
    need = grpo_loss_from_hidden_workspace_bytes(T, V, d)
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
    _require(workspace.numel() >= need, "workspace must hold %d bytes, got %d" % (need, workspace.numel()))
    hp, ldh = _rows(hidden, "hidden")
    wp, ldw = _rows(W, "W")
    dhp, lddh = _f32_rows(dhidden, T, d, "dhidden")
    dwp, lddw = _f32_rows(dW, V, d, "dW")
    rc = load().grpo_loss_from_hidden(hp, ldh, wp, ldw, _dev(tokens, torch.int32, "tokens"),
                                      _dev(old_logp, torch.float32, "old_logp"),
                                      _dev(ref_logp, torch.float32, "ref_logp", True),
                                      _dev(adv.reshape(-1), torch.float32, "adv"),
                                      _dev(seq_weight, torch.float64, "seq_weight"),
                                      _dev(cu_seqlens, torch.int64, "cu_seqlens"), M, row0,
                                      _dev(mask, torch.uint8, "mask", True), T, V, d, eps, beta, grad_scale,
                                      _dev(loss_acc, torch.float64, "loss_acc"), _dev(logp, torch.float32, "logp"),
                                      dhp, lddh, dwp, lddw, _dev(workspace, torch.uint8, "workspace"),
                                      workspace.numel(), _dev(status, torch.int32, "status", True), _stream())
    _check(rc, "grpo_loss_from_hidden")
    return logp, dhidden


class HostStep:
    """pods_host_step_*: the whole path for inputs in host memory (pinned torch CPU tensors).

    Marshalling only: ``set_inputs`` keeps references to the caller's host tensors (and pins a host
    copy of the logits if they are handed over as a device tensor), ``run`` passes their addresses to
    pods_host_step_run, which does every copy and every step."""

    def __init__(self, G, n, m, src_ld, T_cap, V, chunk_rows=2048):
        self.G, self.n, self.m, self.src_ld, self.T_cap, self.V = G, n, m, src_ld, T_cap, V
        self._h = C.c_void_p()
        _check(load().pods_host_step_create(G, n, m, src_ld, T_cap, V, chunk_rows, C.byref(self._h)),
               "pods_host_step_create")
        pin = dict(pin_memory=True)
        self.loss_h = torch.zeros(1, dtype=torch.float32, **pin)
        self.logp_h = torch.zeros(T_cap, dtype=torch.float32, **pin)
        self.idx_h = torch.zeros((G, m), dtype=torch.int32, **pin)
        self.adv_h = torch.zeros((G, m), dtype=torch.float32, **pin)
        self.T_h = C.c_int64(0)
        self.status_h = C.c_uint32(0)
        self._in = None

    @staticmethod
    def _host(a, dtype):
        t = a if isinstance(a, torch.Tensor) else torch.from_numpy(a)
        t = t.to(dtype=dtype, device="cpu").contiguous()
        return t if t.is_pinned() else t.pin_memory()

    def set_inputs(self, rewards, lengths, src_tokens, src_old, src_ref, logits):
        """Host arrays (numpy or CPU tensors) of one batch; ``logits`` [T,V] bf16 (a device tensor is copied to pinned host memory)."""
        lg = logits.detach().to("cpu") if logits.is_cuda else logits
        lg = lg.contiguous()
        self._in = (self._host(rewards, torch.float32), self._host(lengths, torch.int32),
                    self._host(src_tokens, torch.int32), self._host(src_old, torch.float32),
                    None if src_ref is None else self._host(src_ref, torch.float32),
                    lg if lg.is_pinned() else lg.pin_memory())
        r, l, st, so, sr, lg = self._in
        self.h2d_bytes = sum(t.numel() * t.element_size() for t in self._in if t is not None)
        self.d2h_bytes = 4 + 8 + 4 + 4 * lg.shape[0] + 8 * self.G * self.m

    def run(self, eps, beta, rule=RULE_MAXVAR, seed=0, flags=0):
        r, l, st, so, sr, lg = self._in
        rc = load().pods_host_step_run(self._h, r.data_ptr(), l.data_ptr(), st.data_ptr(), so.data_ptr(),
                                       None if sr is None else sr.data_ptr(), lg.data_ptr(), lg.shape[0], eps, beta,
                                       rule, seed, flags, self.loss_h.data_ptr(), self.logp_h.data_ptr(),
                                       self.idx_h.data_ptr(), self.adv_h.data_ptr(), C.byref(self.T_h),
                                       C.byref(self.status_h))
        _check(rc, "pods_host_step_run")
        return float(self.loss_h[0])

    def loss(self) -> float:
        return float(self.loss_h[0])

    def dlogits(self):
        """The gradient [T,V] bf16 left on the device by the last run (a view; valid until the next run)."""
        T = int(self.T_h.value)
        ptr = load().pods_host_step_dlogits(self._h)
        # wrap the device pointer without copying: torch has no public from-pointer constructor, so go through
        # the CUDA array interface
        class _Arr:
            __cuda_array_interface__ = {"shape": (T, self.V), "typestr": "<u2", "data": (int(ptr), False), "version": 2}
        return torch.as_tensor(_Arr(), device="cuda").view(torch.bfloat16)

    def close(self):
        if self._h:
            load().pods_host_step_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
