"""Gradient-accumulation batching (Appendix A.2 note under Table 2: down-sampling per rollout batch, 128 -> 32,
times 4 accumulation steps = effective 512 -> 128), host logic against the oracle on CPU."""
import numpy as np
import pytest

import oracle
from paper_2504_13818_b200 import accumulation as ga, workloads as wl


def test_plan_and_step_major_index_arithmetic():
    plan = ga.make_plan(G=3, n=12, m=6, steps=3)
    assert (plan.n_step, plan.m_step, plan.groups) == (4, 2, 9)
    x = np.arange(3 * 12).reshape(3, 12)
    y = ga.step_major(x, plan)
    assert y.shape == (9, 4)
    for group in range(plan.groups):
        for j in range(plan.n_step):
            g, i = ga.original_rollout(plan, group, j)
            assert y[group, j] == x[g, i]
    assert list(y[0]) == [0, 1, 2, 3] and list(y[1]) == [12, 13, 14, 15] and list(y[3]) == [4, 5, 6, 7]
    import torch
    assert (ga.step_major(torch.from_numpy(x), plan).numpy() == y).all()
    with pytest.raises(ValueError):
        ga.make_plan(2, 10, 4, 4)            # n not a multiple of steps
    with pytest.raises(ValueError):
        ga.make_plan(2, 8, 6, 4)             # m not a multiple of steps
    with pytest.raises(ValueError):
        ga.step_major(np.zeros((2, 12)), plan)
    # the paper's shape: 512 -> 128 in 4 steps of 128 -> 32
    paper = ga.make_plan(G=1, n=512, m=128, steps=4)
    assert (paper.n_step, paper.m_step) == (128, 32)


def test_per_rollout_batch_selection_is_not_the_one_shot_selection():
    """Rollout batch 0 holds all the high rewards: per-batch down-sampling must still take m/steps from every
    batch, while one selection over all n rollouts takes its high end from batch 0 only."""
    plan = ga.make_plan(G=1, n=16, m=4, steps=2)
    r = np.zeros((1, 16), np.float32)
    r[0, :8] = [0, 0, 0, 0, 5, 5, 5, 5]
    r[0, 8:] = [1, 1, 1, 1, 2, 2, 2, 2]
    per_batch = oracle.select(ga.step_major(r, plan), plan.m_step)
    kept = sorted(ga.original_rollout(plan, grp, int(j))[1] for grp in range(plan.groups) for j in per_batch["idx"][grp])
    one_shot = sorted(int(i) for i in oracle.select(r, plan.m)["idx"][0])
    assert kept == [0, 7, 8, 15]             # one lowest and one highest of each rollout batch (ties by index)
    assert one_shot == [0, 1, 6, 7]          # two zeros and two fives: all from rollout batch 0
    assert kept != one_shot
    # advantages are normalised within each rollout batch's kept pair: -1, +1
    np.testing.assert_allclose(per_batch["adv"], [[-1.0, 1.0], [-1.0, 1.0]])


def test_steps_add_up_to_the_batch_objective_and_gradient():
    """The accumulated loss and gradient of the steps (each over its own row range, batch-wide weights) equal
    L_PODS over all kept rollouts at once; a 1/steps factor would be wrong."""
    w = wl.Workload("ga", G=2, n=16, m=8, rewards="bernoulli_uniform", seed=11, V=40, len_kind="uniform",
                    len_lo=3, len_hi=9, logit_sigma=2.0)
    plan = ga.make_plan(w.G, w.n, w.m, steps=4)
    rewards = wl.make_rewards(w)
    lengths, src_tokens = wl.make_rollouts(w)
    L = src_tokens.shape[1]
    sel = oracle.select(ga.step_major(rewards, plan), plan.m_step)
    len_sm = ga.step_major(lengths.reshape(w.G, w.n), plan).reshape(-1)
    tok_sm = ga.step_major(src_tokens.reshape(w.G, w.n, L), plan).reshape(-1, L)
    cu, tokens, _, seq_of_row = oracle.compact(sel["idx"], plan.n_step, len_sm, tok_sm)
    T = int(cu[-1])
    M = plan.groups * plan.m_step
    assert M == w.G * w.m and cu.shape[0] == M + 1
    logits = wl.make_logits_host(w, tokens)
    old, ref = wl.make_old_ref(w, wl.host_logp_tilde(logits, tokens))
    mask = np.ones(T, np.uint8)
    sw = oracle.seq_weights(mask, cu)                    # 1 / (M |o_i|) with the batch-wide M
    adv32 = sel["adv"].astype(np.float32).reshape(-1)
    whole = oracle.grpo_rows(logits, tokens, old, ref, adv32, sw, seq_of_row, mask, w.eps, w.beta)
    loss = oracle.grpo_loss(whole["ell"], mask, cu)

    ranges = ga.step_ranges(cu, plan)
    assert ranges[0][2] == 0 and ranges[-1][3] == T and all(a[3] == b[2] for a, b in zip(ranges, ranges[1:]))
    acc = 0.0
    for a, (s_lo, s_hi, lo, hi) in enumerate(ranges):
        assert s_hi - s_lo == w.G * plan.m_step
        assert (seq_of_row[lo:hi] >= s_lo).all() and (seq_of_row[lo:hi] < s_hi).all()
        rows = np.arange(lo, hi)
        part = oracle.grpo_rows(logits[rows], tokens[rows], old[rows], ref[rows], adv32, sw, seq_of_row[rows], mask[rows],
                                w.eps, w.beta)
        acc += float(np.sum(sw[seq_of_row[rows]] * part["ell"]))
        np.testing.assert_array_equal(part["dlogits"], whole["dlogits"][lo:hi])
    assert abs(acc - loss) <= 1e-14 * max(1.0, abs(loss))
    # what a step would compute on its own (its own M) is `steps` times too large per rollout
    own_cu = cu[ranges[1][0]:ranges[1][1] + 1] - cu[ranges[1][0]]
    own_sw = oracle.seq_weights(np.ones(int(own_cu[-1]), np.uint8), own_cu)
    np.testing.assert_allclose(own_sw, plan.steps * sw[ranges[1][0]:ranges[1][1]], rtol=1e-15)
    with pytest.raises(ValueError):
        ga.step_ranges(cu[:-1], plan)
