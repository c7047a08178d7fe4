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
