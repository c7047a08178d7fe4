"""Gradient-accumulation batching on the GPU: per-rollout-batch selection through pods_select, then the steps'
grpo_loss_chunk calls over their row ranges, against the oracle and against the one-call objective."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_13818_b200 import accumulation as ga, binding, workloads as wl
from parity import LOGP_ATOL, assert_adv_close, assert_dlogits_close, dlogits_report, gradient_slack

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("V", [520, 16384])
def test_accumulation_steps_equal_one_batch_and_the_oracle(V):
    w = wl.Workload("ga", G=3, n=32, m=8, rewards="bernoulli_uniform", seed=5, V=V, len_kind="uniform",
                    len_lo=4, len_hi=12, logit_sigma=2.0)
    plan = ga.make_plan(w.G, w.n, w.m, steps=4)
    rewards = wl.make_rewards(w)
    lengths, src_tokens = wl.make_rollouts(w)
    L = src_tokens.shape[1]
    dev = torch.device("cuda:0")
    status = binding.new_status(dev)

    # selection per rollout batch: indices and k bit-exact, advantages within tolerance
    idx, adv, k = ga.select(torch.from_numpy(rewards).to(dev), plan, status=status)
    want = oracle.select(ga.step_major(rewards, plan), plan.m_step)
    np.testing.assert_array_equal(idx.cpu().numpy(), want["idx"])
    np.testing.assert_array_equal(k.cpu().numpy(), want["k"])
    assert_adv_close(adv.cpu().numpy(), want["adv"])

    len_sm = ga.step_major(lengths.reshape(w.G, w.n), plan).reshape(-1)
    tok_sm = ga.step_major(src_tokens.reshape(w.G, w.n, L), plan).reshape(-1, L)
    cu, toks, _ = binding.pods_compact(idx, plan.n_step, torch.from_numpy(len_sm).to(dev), torch.from_numpy(tok_sm).to(dev),
                                       status=status)
    cu_o, tokens, _, seq_of_row = oracle.compact(want["idx"], plan.n_step, len_sm, tok_sm)
    np.testing.assert_array_equal(cu.cpu().numpy(), cu_o)
    T = int(cu_o[-1])
    tokens_d = toks[:T].contiguous()
    logits = wl.make_logits_host(w, tokens)
    old, ref = wl.make_old_ref(w, wl.host_logp_tilde(logits, tokens))
    lg = torch.from_numpy(logits).view(torch.bfloat16).to(dev)
    old_d, ref_d = torch.from_numpy(old).to(dev), torch.from_numpy(ref).to(dev)

    # the whole batch in one call
    loss1, logp1, dl1 = binding.grpo_loss_fwd_bwd(lg, tokens_d, old_d, ref_d, adv, None, w.eps, w.beta, cu, status=status)

    # the same batch as four accumulation steps
    sw = binding.grpo_seq_weights(None, cu)
    ranges = ga.step_ranges(cu.cpu(), plan)
    acc = torch.zeros(1, dtype=torch.float64, device=dev)
    logp = torch.empty(T, dtype=torch.float32, device=dev)
    dl = torch.empty_like(lg)
    ws = torch.empty(binding.grpo_loss_chunk_workspace_bytes(64), dtype=torch.uint8, device=dev)
    for a, (_, _, lo, hi) in enumerate(ranges):
        ga.loss_step(a, ranges, lg[lo:hi], tokens_d, old_d, ref_d, adv.reshape(-1), sw, cu, None, w.eps, w.beta, acc, logp,
                     dl[lo:hi], ws, chunk_rows=64, status=status)
    loss = torch.empty(1, dtype=torch.float32, device=dev)
    binding.grpo_loss_finalize(acc, loss)
    torch.cuda.synchronize()
    assert binding.read_status(status) == 0
    assert dl.view(torch.int16).cpu().numpy().tobytes() == dl1.view(torch.int16).cpu().numpy().tobytes()
    assert logp.cpu().numpy().tobytes() == logp1.cpu().numpy().tobytes()
    assert abs(float(loss.item()) - float(loss1.item())) <= 1e-6 * abs(float(loss1.item())) + 1e-12

    # and against the oracle with the batch-wide M
    mask = np.ones(T, np.uint8)
    sw_o = oracle.seq_weights(mask, cu_o)
    rows = oracle.grpo_rows(logits, tokens, old, ref, want["adv"].astype(np.float32).reshape(-1), sw_o, seq_of_row, mask,
                            w.eps, w.beta)
    loss_o = oracle.grpo_loss(rows["ell"], mask, cu_o)
    assert np.abs(logp.cpu().numpy() - rows["logp"]).max() <= LOGP_ATOL
    scale = np.mean([abs(rows["ell"][cu_o[i]:cu_o[i + 1]].mean()) for i in range(len(cu_o) - 1)])
    assert abs(float(loss.item()) - loss_o) <= 1e-4 * max(abs(loss_o), scale / 1e3)
    b = {"w": w, "mask": mask, "cu": cu_o, "seq_of_row": seq_of_row, "adv32": want["adv"].astype(np.float32).reshape(-1),
         "old": old, "ref": ref}
    assert_dlogits_close(dlogits_report(dl.view(torch.uint16).cpu().numpy(), rows["dlogits"], gradient_slack(b, rows)))
