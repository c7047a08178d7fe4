"""The C-ABI library: it loads without a GPU, exports every symbol include/pods.h declares, and the
binding's signature table covers the same set.  Host-visible argument errors come back as status
codes before any launch (no compute call is made here)."""
import ctypes as C
import re

from paper_2504_13818_b200 import binding
from paper_2504_13818_b200.csrc import build as cuda_build


def _declared(rootpath):
    text = (rootpath / "include" / "pods.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return set(re.findall(r"\b((?:pods|grpo)_[a-z0-9_]+)\s*\(", text))


def test_library_builds_loads_and_exports_every_declared_symbol(request):
    cuda_build.build()
    lib = binding.load()
    names = _declared(request.config.rootpath)
    assert {"pods_select", "pods_compact", "grpo_loss_fwd_bwd", "grpo_loss_chunk"} <= names
    for name in names:
        assert hasattr(lib, name), name
    assert names == set(binding.SIGNATURES), names ^ set(binding.SIGNATURES)
    assert b"sm_100a" in lib.pods_version()


def test_host_side_argument_checks_return_codes_without_launching():
    lib = binding.load()
    bad = lib.pods_select(None, 4, 16, 17, 0, 0, 0, None, None, None, None, None)      # m > n
    assert bad == 1 and lib.pods_status_string(bad) == b"invalid argument"
    assert lib.pods_select(None, 4, 2048, 4, 0, 0, 0, None, None, None, None, None) == 2   # n > PODS_MAX_N
    assert lib.pods_select(None, 4, 16, 4, 9, 0, 0, None, None, None, None, None) == 2     # unknown rule
    assert lib.pods_select(None, 4, 16, 4, 0, 0, 0, None, None, None, None, None) == 1     # null pointers
    assert lib.pods_select(None, 0, 16, 4, 0, 0, 0, None, None, None, None, None) == 0     # empty batch
    assert lib.pods_compact(None, 1, 4, 2, None, None, 8, None, 0, None, None, None, 16, None, None) == 1
    assert lib.grpo_loss_chunk_workspace_bytes(1000) >= 8000
    assert lib.grpo_loss_workspace_bytes(1000, 16, 0) >= 8000 + 128
    fake = C.c_void_p(256)      # non-null, never dereferenced: the size checks come first
    rc = lib.grpo_loss_chunk(fake, 8, fake, fake, fake, fake, fake, fake, 1, 0, None, 4, 16, 0.2, 0.0, 1.0,
                             fake, fake, fake, 16, None, 0, None, None)
    assert rc == 1              # ldl < V
    rc = lib.grpo_loss_chunk(fake, 16, fake, fake, fake, fake, fake, fake, 1, 0, None, 4, 16, 0.2, 0.0, 1.0,
                             fake, fake, fake, 16, None, 0, None, None)
    assert rc == 3              # no workspace
    rc = lib.grpo_loss_chunk(fake, 16, fake, fake, None, fake, fake, fake, 1, 0, None, 4, 16, 0.2, 0.04, 1.0,
                             fake, fake, fake, 16, fake, 4096, None, None)
    assert rc == 1              # beta != 0 needs ref_logp


def test_binding_refuses_host_tensors():
    import pytest
    import torch
    with pytest.raises(binding.PodsError):
        binding.pods_select(torch.zeros(2, 4), 2)


def test_cluster_vocabulary_limit_is_a_process_wide_setting_with_a_floor():
    lib = binding.load()
    default = lib.pods_set_loss_cluster_min_vocab(100000)
    assert default == 8192
    assert lib.pods_set_loss_cluster_min_vocab(5) == 100000       # values below 2048 are raised to 2048
    assert lib.pods_set_loss_cluster_min_vocab(default) == 2048
    assert lib.pods_set_loss_cluster_min_vocab(default) == default


def test_binding_checks_every_buffer_length_before_the_call():
    """The C ABI cannot see buffer sizes, so the binding does: a short or mis-shaped tensor is refused on
    the host.  Host tensors are enough to show it - the length checks come before anything is marshalled,
    so nothing can have been launched when they raise."""
    import pytest
    import torch
    T, V, M = 12, 16, 3
    bf = torch.zeros((T, V), dtype=torch.bfloat16)

    def loss_args(**over):
        a = dict(logits=bf, tokens=torch.zeros(T, dtype=torch.int32), old_logp=torch.zeros(T), ref_logp=torch.zeros(T),
                 adv=torch.zeros(M), seq_weight=torch.zeros(M, dtype=torch.float64),
                 cu_seqlens=torch.zeros(M + 1, dtype=torch.int64), row0=0, mask=torch.ones(T, dtype=torch.uint8),
                 eps=0.2, beta=0.04, loss_acc=torch.zeros(1, dtype=torch.float64), logp=torch.zeros(T),
                 dlogits=torch.zeros_like(bf))
        a.update(over)
        return a

    wrong = {"dlogits": torch.zeros((T - 1, V), dtype=torch.bfloat16), "tokens": torch.zeros(T - 1, dtype=torch.int32),
             "old_logp": torch.zeros(T + 1), "ref_logp": torch.zeros(1), "mask": torch.ones(T - 2, dtype=torch.uint8),
             "logp": torch.zeros(T - 1), "adv": torch.zeros(M + 1), "seq_weight": torch.zeros(M - 1, dtype=torch.float64),
             "cu_seqlens": torch.zeros(M, dtype=torch.int64), "loss_acc": torch.zeros(2, dtype=torch.float64)}
    ws = torch.zeros(1 << 16, dtype=torch.uint8)
    for name, bad in wrong.items():
        with pytest.raises(binding.PodsError, match="must hold|must have the shape"):
            binding.grpo_loss_chunk(workspace=ws, **loss_args(**{name: bad}))
        with pytest.raises(binding.PodsError, match="must hold|must have the shape"):
            binding.grpo_loss_chunk_static(**loss_args(**{name: bad}))
    for name in ("dlogits", "tokens", "old_logp", "ref_logp", "mask", "logp", "adv", "cu_seqlens"):
        a = loss_args(**{name: wrong[name]})
        for drop in ("seq_weight", "row0", "loss_acc"):
            a.pop(drop)
        with pytest.raises(binding.PodsError, match="must hold|must have the shape"):
            binding.grpo_loss_fwd_bwd(workspace=ws, loss=torch.zeros(1), **a)
    a = loss_args()
    for drop in ("seq_weight", "row0", "loss_acc"):
        a.pop(drop)
    with pytest.raises(binding.PodsError, match="workspace must hold"):
        binding.grpo_loss_fwd_bwd(workspace=torch.zeros(8, dtype=torch.uint8), loss=torch.zeros(1), **a)
    # with every length right the first complaint is that these are host tensors: the checks above all passed
    with pytest.raises(binding.PodsError, match="CUDA"):
        binding.grpo_loss_chunk(workspace=ws, **loss_args())

    G, n, m, ld = 2, 4, 2, 8
    idx = torch.zeros((G, m), dtype=torch.int32)
    lengths, src = torch.zeros(G * n, dtype=torch.int32), torch.zeros((G * n, ld), dtype=torch.int32)
    good = (torch.zeros(G * m + 1, dtype=torch.int64), torch.zeros(G * m * ld, dtype=torch.int32), [])
    with pytest.raises(binding.PodsError, match="lengths must hold"):
        binding.pods_compact(idx, n, lengths[:-1], src, out=good)
    with pytest.raises(binding.PodsError, match="rows"):
        binding.pods_compact(idx, n, lengths, src[:-1], out=good)
    with pytest.raises(binding.PodsError, match="cu_seqlens must hold"):
        binding.pods_compact(idx, n, lengths, src, out=(good[0][:-1], good[1], []))
    with pytest.raises(binding.PodsError, match="dst_tokens must hold"):
        binding.pods_compact(idx, n, lengths, src, out=(good[0], good[1][:-1], []))
    with pytest.raises(binding.PodsError, match="dst_f32 streams must hold"):
        binding.pods_compact(idx, n, lengths, src, src_f32=[torch.zeros((G * n, ld))],
                             out=(good[0], good[1], [torch.zeros(3)]))
    r = torch.zeros((G, n))
    with pytest.raises(binding.PodsError, match="idx must hold"):
        binding.pods_select_into(r, m, torch.zeros((G, m + 1), dtype=torch.int32), torch.zeros((G, m)))
    with pytest.raises(binding.PodsError, match="adv must hold"):
        binding.pods_select_into(r, m, idx, torch.zeros((G, m - 1)))
    with pytest.raises(binding.PodsError, match="k must hold"):
        binding.pods_select_into(r, m, idx, torch.zeros((G, m)), torch.zeros(G + 1, dtype=torch.int32))
    with pytest.raises(binding.PodsError, match="1 <= m <= n"):
        binding.pods_select_into(r, n + 1, idx, torch.zeros((G, m)))
    with pytest.raises(binding.PodsError, match="seq_weight must hold"):
        binding.grpo_seq_weights(None, torch.zeros(M + 1, dtype=torch.int64), out=torch.zeros(M + 2, dtype=torch.float64))


def test_loss_from_hidden_checks_sizes_on_the_host():
    """grpo_loss_from_hidden: the library refuses impossible sizes before launching, the binding refuses short or
    mis-shaped buffers before marshalling, and the panel limit is a process-wide setting with a floor."""
    import pytest
    import torch
    lib = binding.load()
    fake = C.c_void_p(256)

    def call(T=4, V=16, d=8, ldh=8, ldw=8, lddh=8, lddw=8, beta=0.0, ref=None, ws=None, ws_bytes=0):
        return lib.grpo_loss_from_hidden(fake, ldh, fake, ldw, fake, fake, ref, fake, fake, fake, 1, 0, None, T, V, d,
                                         0.2, beta, 1.0, fake, fake, fake, lddh, fake, lddw, ws, ws_bytes, None, None)

    assert call(d=12) == 1 and call(ldh=4) == 1 and call(lddw=6) == 1 and call(V=0) == 1     # sizes
    assert call(beta=0.04) == 1                                                              # beta != 0 needs ref_logp
    assert call() == 3                                                                       # no workspace
    assert call(T=0) == 0                                                                    # empty chunk
    need = lib.grpo_loss_from_hidden_workspace_bytes(300, 1000, 64)
    assert need >= 384 * 1024 * 2                       # at least the panel of one launch: 384 rows x 4 tiles, bf16
    default = lib.pods_set_loss_from_hidden_panel_bytes(1)
    assert default == 512 << 20
    assert lib.grpo_loss_from_hidden_workspace_bytes(300, 1000, 64) < need        # one tile per panel now
    assert lib.pods_set_loss_from_hidden_panel_bytes(default) == 65536            # the floor
    assert lib.grpo_loss_from_hidden_workspace_bytes(300, 1000, 64) == need

    T, V, d, M = 12, 40, 16, 3
    def args(**over):
        a = dict(hidden=torch.zeros((T, d), dtype=torch.bfloat16), W=torch.zeros((V, d), dtype=torch.bfloat16),
                 tokens=torch.zeros(T, dtype=torch.int32), old_logp=torch.zeros(T), ref_logp=torch.zeros(T),
                 adv=torch.zeros(M), seq_weight=torch.zeros(M, dtype=torch.float64),
                 cu_seqlens=torch.zeros(M + 1, dtype=torch.int64), row0=0, mask=torch.ones(T, dtype=torch.uint8),
                 eps=0.2, beta=0.04, loss_acc=torch.zeros(1, dtype=torch.float64), dW=torch.zeros((V, d)),
                 logp=torch.zeros(T), dhidden=torch.zeros((T, d)))
        a.update(over)
        return a

    wrong = {"W": torch.zeros((V, d + 8), dtype=torch.bfloat16), "tokens": torch.zeros(T - 1, dtype=torch.int32),
             "old_logp": torch.zeros(T + 1), "ref_logp": torch.zeros(1), "mask": torch.ones(T - 2, dtype=torch.uint8),
             "logp": torch.zeros(T - 1), "adv": torch.zeros(M + 1), "seq_weight": torch.zeros(M - 1, dtype=torch.float64),
             "loss_acc": torch.zeros(2, dtype=torch.float64), "dW": torch.zeros((V - 1, d)),
             "dhidden": torch.zeros((T, d + 1)), "workspace": torch.zeros(8, dtype=torch.uint8)}
    for name, bad in wrong.items():
        with pytest.raises(binding.PodsError, match="must hold|must have"):
            binding.grpo_loss_from_hidden(**args(**{name: bad}))
    with pytest.raises(binding.PodsError, match="CUDA"):           # every length right: only the device is wrong
        binding.grpo_loss_from_hidden(**args())
