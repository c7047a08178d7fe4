"""pods_host_step_*: the whole path from host buffers (rewards and rollout storage in, loss / logp / idx /
adv out, gradient left on the device) against the oracle's chain, with the logits uploaded in several
chunks through the two staging buffers."""
import numpy as np
import pytest
import torch

from paper_2504_13818_b200 import binding, workloads as wl
from parity import (DLOGITS_ULPS, LOGP_ATOL, assert_adv_close, assert_loss_close, build_batch, dlogits_ulp_error,
                    gradient_slack, oracle_loss, shrink)

pytestmark = pytest.mark.gpu


def _rollout_storage(b):
    """Scatter the packed old/ref log-probs back to padded all-rollouts storage (zeros elsewhere)."""
    w = b["w"]
    src_old = np.zeros(b["src_tokens"].shape, np.float32)
    src_ref = np.zeros(b["src_tokens"].shape, np.float32)
    for i in range(b["cu"].shape[0] - 1):
        g, j = divmod(i, w.m)
        row = g * w.n + int(b["sel"]["idx"][g, j])
        lo, hi = int(b["cu"][i]), int(b["cu"][i + 1])
        src_old[row, :hi - lo] = b["old"][lo:hi]
        src_ref[row, :hi - lo] = b["ref"][lo:hi]
    return src_old, src_ref


@pytest.mark.parametrize("V,chunk_rows", [(1024, 37), (16384, 50), (16384, 100000)])
def test_host_step_matches_the_oracle_chain(V, chunk_rows):
    w = shrink(wl.WORKLOADS["c1_tiny"], V=V, G=4, n=16, m=4, len_lo=8, len_hi=40, seed=100 + V % 7)
    b = build_batch(w)
    want = oracle_loss(b)
    T = b["tokens"].shape[0]
    src_old, src_ref = _rollout_storage(b)
    step = binding.HostStep(w.G, w.n, w.m, b["src_tokens"].shape[1], T, V, chunk_rows=chunk_rows)
    step.set_inputs(b["rewards"], b["lengths"], b["src_tokens"], src_old, src_ref,
                    torch.from_numpy(b["logits"]).view(torch.bfloat16))
    for _ in range(2):                                   # a second run on the same object reuses every buffer
        loss = step.run(w.eps, w.beta)
        assert int(step.T_h.value) == T and int(step.status_h.value) == 0
        assert (step.idx_h.numpy() == b["sel"]["idx"]).all()
        assert_adv_close(step.adv_h.numpy(), b["sel"]["adv"])
        assert np.abs(step.logp_h.numpy()[:T] - want["logp"]).max() <= LOGP_ATOL
        assert_loss_close(loss, want, b)
        dl = step.dlogits().view(torch.uint16).cpu().numpy()
        assert dlogits_ulp_error(dl, want["dlogits"], gradient_slack(b, want)).max() <= DLOGITS_ULPS
    assert step.h2d_bytes >= T * V * 2 and step.d2h_bytes >= 4 * T
    step.close()


def test_host_step_refuses_logits_of_another_row_count():
    w = shrink(wl.WORKLOADS["c1_tiny"], V=1024, G=2, n=8, m=4, seed=3)
    b = build_batch(w)
    T = b["tokens"].shape[0]
    src_old, src_ref = _rollout_storage(b)
    step = binding.HostStep(w.G, w.n, w.m, b["src_tokens"].shape[1], T, w.V)
    step.set_inputs(b["rewards"], b["lengths"], b["src_tokens"], src_old, src_ref,
                    torch.from_numpy(b["logits"][:T - 1]).view(torch.bfloat16))
    with pytest.raises(binding.PodsError, match="invalid argument"):
        step.run(w.eps, w.beta)
    assert int(step.T_h.value) == T                       # the device's count is reported
    step.close()
