"""grpo_loss_chunk_static: the chunk call for callers that cannot allocate device memory (code inside a
framework's planned-memory region, plug-ins handed only inputs and outputs, embedders that forbid
cudaMalloc after start-up).  Its scratch is an array inside the library, so the check is simply that it
returns what grpo_loss_chunk returns with a caller workspace - on two calls in a row, because the
array is shared between calls and keeps the previous call's contents."""
import numpy as np
import pytest
import torch

from paper_2504_13818_b200 import binding, workloads as wl
from parity import DLOGITS_ULPS, LOGP_ATOL, LOSS_RTOL, bf16_ulp, build_batch, shrink

pytestmark = pytest.mark.gpu


def _t(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    return (t if dtype is None else t.view(dtype)).cuda()


def _inputs(seed, V, len_hi):
    w = shrink(wl.WORKLOADS["c1_tiny"], G=3, n=8, m=4, V=V, len_lo=8, len_hi=len_hi, seed=seed)
    b = build_batch(w)
    cu = _t(b["cu"])
    return w, {"logits": _t(b["logits"], torch.bfloat16), "tokens": _t(b["tokens"]), "old": _t(b["old"]),
               "ref": _t(b["ref"]), "adv": _t(b["adv32"]), "cu": cu,
               "sw": binding.grpo_seq_weights(None, cu)}


def _run(w, x, static):
    T = x["logits"].shape[0]
    acc = torch.zeros(1, dtype=torch.float64, device="cuda")
    logp = torch.empty(T, dtype=torch.float32, device="cuda")
    dl = torch.empty_like(x["logits"])
    status = binding.new_status()
    args = (x["logits"], x["tokens"], x["old"], x["ref"], x["adv"], x["sw"], x["cu"], 0, None, w.eps, w.beta,
            acc, logp, dl)
    if static:
        binding.grpo_loss_chunk_static(*args, status=status)
    else:
        ws = torch.empty(binding.grpo_loss_chunk_workspace_bytes(T), dtype=torch.uint8, device="cuda")
        binding.grpo_loss_chunk(*args, ws, status=status)
    torch.cuda.synchronize()
    assert binding.read_status(status) == 0
    return float(acc.item()), logp.cpu().numpy(), dl.float().cpu().numpy().astype(np.float64)


def _assert_same(got, want):
    assert abs(got[0] - want[0]) <= LOSS_RTOL * abs(want[0])
    assert np.abs(got[1] - want[1]).max() <= LOGP_ATOL
    assert (np.abs(got[2] - want[2]) <= DLOGITS_ULPS * bf16_ulp(want[2])).all()


def test_static_scratch_variant_matches_workspace_variant_on_two_calls_in_a_row():
    # a longer chunk first, a shorter one second: the second call finds the first call's terms in the
    # shared scratch and must not pick any of them up
    first = _inputs(seed=31, V=1024, len_hi=40)
    second = _inputs(seed=32, V=520, len_hi=12)
    assert second[1]["logits"].shape[0] < first[1]["logits"].shape[0]
    want_first, want_second = _run(*first, static=False), _run(*second, static=False)
    got_first = _run(*first, static=True)
    got_second = _run(*second, static=True)
    _assert_same(got_first, want_first)
    _assert_same(got_second, want_second)


def _free_device_bytes():
    free, _ = torch.cuda.mem_get_info()
    return free


@pytest.mark.parametrize("V,rows", [(16384, 16384), (151936, 2048)])
def test_static_variant_on_the_cluster_path_against_the_oracle_without_allocating(V, rows):
    """Long rows take the kernel that also keeps a 32-byte record per row in the built-in array (the half of it
    that the short-row cases above never touch).  Checked against the CPU oracle, not against the sibling entry
    point: a full-capacity chunk (V = 16384: exactly grpo_loss_chunk_static_max_rows() rows) and the Qwen
    vocabulary, each followed by a shorter second call that finds the first call's records still in the array.
    The free device memory is read around each call: a call that allocated anything would lower it."""
    import oracle
    from parity import assert_dlogits_close, dlogits_report, gradient_slack, record
    cap = binding.grpo_loss_chunk_static_max_rows()
    assert rows <= cap and (V != 16384 or rows == cap)
    M = 8
    rng = np.random.default_rng(V)
    # rollouts of uneven length that add up to `rows`
    cuts = np.sort(rng.choice(np.arange(1, rows), size=M - 1, replace=False))
    cu = np.concatenate([[0], cuts, [rows]]).astype(np.int64)
    seq_of_row = oracle.seq_of_rows(cu)
    tokens = rng.integers(0, V, size=rows, dtype=np.int32)
    adv32 = rng.normal(size=M).astype(np.float32)
    mask = np.ones(rows, np.uint8)
    dev = torch.device("cuda:0")
    gen = torch.Generator(device=dev)
    gen.manual_seed(1000 + V)
    logits = (torch.randn((rows, V), generator=gen, device=dev) * 3.0).to(torch.bfloat16)
    tok_d = torch.from_numpy(tokens).to(dev)
    lt = wl.library_logp(logits, tok_d).cpu().numpy().astype(np.float64)
    old = (lt + rng.normal(0, 0.05, rows)).astype(np.float32)
    ref = (lt + rng.normal(0, 0.05, rows)).astype(np.float32)
    sw = oracle.seq_weights(mask, cu)
    eps, beta = 0.2, 0.04

    cu_d = torch.from_numpy(cu).to(dev)
    sw_d = binding.grpo_seq_weights(None, cu_d)
    old_d, ref_d, adv_d = torch.from_numpy(old).to(dev), torch.from_numpy(ref).to(dev), torch.from_numpy(adv32).to(dev)
    dl = torch.empty_like(logits)
    logp = torch.empty(rows, dtype=torch.float32, device=dev)
    acc = torch.zeros(1, dtype=torch.float64, device=dev)
    status = binding.new_status(dev)

    def call(n_rows, check=True):
        acc.zero_()
        torch.cuda.synchronize()
        before = _free_device_bytes()
        binding.grpo_loss_chunk_static(logits[:n_rows], tok_d[:n_rows], old_d[:n_rows], ref_d[:n_rows], adv_d, sw_d, cu_d,
                                       0, None, eps, beta, acc, logp[:n_rows], dl[:n_rows], status=status)
        torch.cuda.synchronize()
        assert not check or _free_device_bytes() == before, "the call changed the free device memory"
        assert binding.read_status(status) == 0
        return float(acc.item())

    # the first call on a device looks up the array's address, and the first launch of a kernel loads its code
    # (the driver's own bookkeeping, not an allocation of the call): not measured
    call(min(rows, 64), check=False)
    for n_rows in (rows, rows // 3):                     # full chunk, then a shorter one over the stale records
        got_acc = call(n_rows)
        want_acc, worst = 0.0, {"literal_ulps": 0.0, "allowance_ulps": 0.0, "allowance_rows": 0, "logp_abs": 0.0}
        size = 0.0
        block = 1024 if V > 50000 else 4096
        for lo in range(0, n_rows, block):
            hi = min(n_rows, lo + block)
            out = oracle.grpo_rows(logits[lo:hi].view(torch.uint16).cpu().numpy(), tokens[lo:hi], old[lo:hi], ref[lo:hi],
                                   adv32, sw, seq_of_row[lo:hi], mask[lo:hi], eps, beta, want_dlogits=True)
            worst["logp_abs"] = max(worst["logp_abs"], float(np.abs(logp[lo:hi].cpu().numpy() - out["logp"]).max()))
            b = {"w": wl.Workload("static", G=1, n=M, m=M, rewards="", seed=0, V=V, eps=eps, beta=beta),
                 "mask": mask, "cu": cu, "seq_of_row": seq_of_row, "adv32": adv32, "old": old, "ref": ref}
            rep = dlogits_report(dl[lo:hi].view(torch.uint16).cpu().numpy(), out["dlogits"],
                                 gradient_slack(b, out, rows=np.arange(lo, hi)))
            assert_dlogits_close(rep)
            worst["literal_ulps"] = max(worst["literal_ulps"], rep["literal_ulps"])
            worst["allowance_ulps"] = max(worst["allowance_ulps"], rep["allowance_ulps"])
            worst["allowance_rows"] += rep["allowance_rows"]
            terms = sw[seq_of_row[lo:hi]] * out["ell"]
            want_acc += float(terms.sum())
            size += float(np.abs(terms).sum())
        assert worst["logp_abs"] <= LOGP_ATOL
        assert abs(got_acc - want_acc) <= LOSS_RTOL * max(abs(want_acc), size / 1e3)
        record("grpo_loss_chunk_static V=%d rows=%d" % (V, n_rows), V=V, rows=n_rows, loss_acc=want_acc,
               acc_rel_literal=abs(got_acc - want_acc) / abs(want_acc), **worst)


def test_static_variant_rejects_chunks_beyond_its_scratch():
    cap = binding.grpo_loss_chunk_static_max_rows()
    assert cap == 16384
    V = 8
    T = cap + 1
    lg = torch.zeros((T, V), dtype=torch.bfloat16, device="cuda")
    z32 = torch.zeros(T, dtype=torch.float32, device="cuda")
    cu = torch.tensor([0, T], dtype=torch.int64, device="cuda")
    acc = torch.zeros(1, dtype=torch.float64, device="cuda")
    with pytest.raises(binding.PodsError, match="built-in scratch"):
        binding.grpo_loss_chunk_static(lg, torch.zeros(T, dtype=torch.int32, device="cuda"), z32, z32,
                                       torch.ones(1, device="cuda"), torch.ones(1, dtype=torch.float64, device="cuda"),
                                       cu, 0, None, 0.2, 0.04, acc, torch.empty_like(z32), torch.empty_like(lg))
    torch.cuda.synchronize()
    assert float(acc.item()) == 0.0
