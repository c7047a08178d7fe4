"""Row sharding on one GPU: the row ranges of 2 and 3 ranks are run one after the other (independent launches,
each with its own loss accumulator), as the ranks of a job would run them on their own GPUs.  Gradient rows and
log-probs must be bit-identical to the unsharded run (a row's result does not depend on which launch holds it),
and the accumulators must add up to the unsharded loss, which is checked against the oracle."""
import numpy as np
import pytest
import torch

from paper_2504_13818_b200 import binding, workloads as wl
from paper_2504_13818_b200.sharding import row_range
from parity import assert_loss_close, build_batch, oracle_loss, shrink

pytestmark = pytest.mark.gpu


def _run(b, lo, hi, d):
    """grpo_loss_chunk over rows [lo, hi) of the batch; returns the fp64 accumulator."""
    w = b["w"]
    acc = torch.zeros(1, dtype=torch.float64, device="cuda")
    if hi > lo:
        ws = torch.empty(binding.grpo_loss_chunk_workspace_bytes(hi - lo), dtype=torch.uint8, device="cuda")
        binding.grpo_loss_chunk(d["logits"][lo:hi], d["tokens"][lo:hi], d["old"][lo:hi], d["ref"][lo:hi], d["adv"],
                                d["sw"], d["cu"], lo, None, w.eps, w.beta, acc, d["logp"][lo:hi], d["dl"][lo:hi], ws,
                                status=d["status"])
    return acc


@pytest.mark.parametrize("V,world", [(1000, 2), (2048, 3), (16384, 2), (151936, 3)])
def test_sharded_rows_equal_the_unsharded_run(V, world):
    w = shrink(wl.WORKLOADS["c2_qwen_vocab"], V=V, G=2, n=8, m=4, len_lo=5, len_hi=13, seed=V % 89)
    b = build_batch(w)
    T = b["tokens"].shape[0]
    cu = torch.from_numpy(b["cu"]).cuda()
    d = {"logits": torch.from_numpy(b["logits"]).view(torch.bfloat16).cuda(), "tokens": torch.from_numpy(b["tokens"]).cuda(),
         "old": torch.from_numpy(b["old"]).cuda(), "ref": torch.from_numpy(b["ref"]).cuda(),
         "adv": torch.from_numpy(b["adv32"]).cuda(), "cu": cu, "sw": binding.grpo_seq_weights(None, cu),
         "status": binding.new_status()}

    def fresh():
        d["logp"] = torch.empty(T, dtype=torch.float32, device="cuda")
        d["dl"] = torch.empty_like(d["logits"])

    fresh()
    whole = _run(b, 0, T, d)
    torch.cuda.synchronize()
    want_dl, want_logp = d["dl"].view(torch.int16).cpu().numpy(), d["logp"].cpu().numpy()

    fresh()
    edges = [row_range(T, world, r, multiple=3) for r in range(world)]
    assert any(lo not in b["cu"] for lo, _ in edges[1:])          # a boundary inside a rollout
    parts = [_run(b, lo, hi, d) for lo, hi in edges]
    torch.cuda.synchronize()
    assert binding.read_status(d["status"]) == 0
    assert d["dl"].view(torch.int16).cpu().numpy().tobytes() == want_dl.tobytes()
    assert d["logp"].cpu().numpy().tobytes() == want_logp.tobytes()
    total = sum(float(p.item()) for p in parts)
    assert abs(total - float(whole.item())) <= 1e-12 * abs(float(whole.item())) + 1e-18      # fp64 sums, regrouped

    loss = torch.empty(1, dtype=torch.float32, device="cuda")
    binding.grpo_loss_finalize(torch.tensor([total], dtype=torch.float64, device="cuda"), loss)
    assert_loss_close(float(loss.item()), oracle_loss(b, want_dlogits=False), b)
