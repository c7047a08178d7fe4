"""Pins for the loss / gradient oracle: hand-worked values of the Section 3.2 formula, textbook
log-softmax special cases and the framework's library log_softmax, special cases in which terms
vanish, and central finite differences of the loss for the gradient."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_13818_b200 import workloads as wl

RNG = np.random.default_rng(7)


def _one_seq(T):
    cu = np.array([0, T], np.int64)
    return cu, oracle.seq_of_rows(cu), np.ones(T, np.uint8)


def test_hand_worked_token_cases(request):
    path = request.config.rootpath / "tests" / "golden" / "grpo_token_cases.txt"
    rows = [ln.split() for ln in open(path) if not ln.startswith("#") and ln.strip()]
    assert len(rows) == 6
    x = np.array([[0.0, np.log(3.0)]])
    cu, sor, mask = _one_seq(1)
    for row in rows:
        tok, pi_old, a, beta, pi_ref, loss, dl, d0, d1 = [float(v) for v in row]
        out = oracle.grpo_rows_f64(x, [int(tok)], [np.log(pi_old)], [np.log(pi_ref)], [a], [1.0], sor, mask, 0.2, beta)
        assert oracle.grpo_loss(out["ell"], mask, cu) == pytest.approx(loss, rel=1e-13, abs=1e-15)
        assert out["g"][0] == pytest.approx(dl, rel=1e-13, abs=1e-15)
        np.testing.assert_allclose(out["dlogits"][0], [d0, d1], rtol=1e-12, atol=1e-15)


def test_logp_uniform_and_dominant_rows():
    V = 37
    bits = wl.f32_to_bf16_bits(np.full((1, V), 1.25, np.float32))
    cu, sor, mask = _one_seq(1)
    out = oracle.grpo_rows(bits, [5], [0.0], [0.0], [1.0], [1.0], sor, mask, 0.2, 0.0)
    assert out["logp"][0] == pytest.approx(-np.log(V), rel=1e-14)
    x = np.full((1, V), -30.0, np.float32)
    x[0, 3] = 30.0
    out = oracle.grpo_rows(wl.f32_to_bf16_bits(x), [3], [0.0], [0.0], [1.0], [1.0], sor, mask, 0.2, 0.0)
    assert out["logp"][0] == pytest.approx(-(V - 1) * np.exp(-60.0), rel=1e-9)


def test_logp_matches_library_log_softmax_on_bf16_rows():
    T, V = 24, 515
    x = RNG.normal(0, 3, size=(T, V)).astype(np.float32)
    bits = wl.f32_to_bf16_bits(x)
    tok = RNG.integers(0, V, T).astype(np.int32)
    cu, sor, mask = _one_seq(T)
    out = oracle.grpo_rows(bits, tok, np.zeros(T), np.zeros(T), [1.0], [1.0 / T], sor, mask, 0.2, 0.04,
                           want_dlogits=False)
    lib = torch.log_softmax(torch.from_numpy(wl.bf16_bits_to_f32(bits)).double(), dim=-1).numpy()
    np.testing.assert_allclose(out["logp"], lib[np.arange(T), tok], rtol=0, atol=1e-12)


def _random_batch(M=5, V=11, seed=3):
    rng = np.random.default_rng(seed)
    lens = rng.integers(1, 6, M)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    T = int(cu[-1])
    x = rng.normal(0, 2, size=(T, V))
    tok = rng.integers(0, V, T).astype(np.int32)
    adv = rng.normal(0, 1, M)
    mask = (rng.uniform(size=T) < 0.8).astype(np.uint8)
    return cu, x, tok, adv, mask


def _loss_f64(cu, x, tok, old, ref, adv, mask, eps, beta):
    w = oracle.seq_weights(mask, cu)
    out = oracle.grpo_rows_f64(x, tok, old, ref, adv, w, oracle.seq_of_rows(cu), mask, eps, beta)
    return oracle.grpo_loss(out["ell"], mask, cu), out, w


def test_on_policy_no_kl_loss_is_minus_mean_advantage():
    """old = logp, beta = 0: every ratio is 1, so L = -(1/M) sum_i a_i over non-empty sequences."""
    cu, x, tok, adv, mask = _random_batch()
    mask[:] = 1
    logp = torch.log_softmax(torch.from_numpy(x), -1).numpy()[np.arange(len(tok)), tok]
    loss, out, _ = _loss_f64(cu, x, tok, logp, logp, adv, mask, 0.2, 0.0)
    assert loss == pytest.approx(-adv.mean(), rel=1e-12)


def test_kl_term_vanishes_when_reference_equals_policy():
    cu, x, tok, adv, mask = _random_batch()
    logp = torch.log_softmax(torch.from_numpy(x), -1).numpy()[np.arange(len(tok)), tok]
    old = logp + RNG.normal(0, 0.05, len(tok))
    l0, o0, _ = _loss_f64(cu, x, tok, old, logp, adv, mask, 0.2, 0.0)
    l1, o1, _ = _loss_f64(cu, x, tok, old, logp, adv, mask, 0.2, 7.0)
    assert l1 == pytest.approx(l0, rel=1e-12)
    np.testing.assert_allclose(o1["dlogits"], o0["dlogits"], atol=1e-13)


def test_clipped_side_has_zero_policy_gradient():
    """rho > 1+eps with a > 0, or rho < 1-eps with a < 0: the clipped branch is the min, gradient 0."""
    cu, x, tok, adv, mask = _random_batch()
    mask[:] = 1
    logp = torch.log_softmax(torch.from_numpy(x), -1).numpy()[np.arange(len(tok)), tok]
    sor = oracle.seq_of_rows(cu)
    old = logp - np.sign(adv[sor]) * 0.5          # rho = exp(+-0.5) on the penalised side
    _, out, _ = _loss_f64(cu, x, tok, old, logp, adv, mask, 0.2, 0.0)
    assert np.abs(out["dlogits"]).max() == 0.0
    old = logp + np.sign(adv[sor]) * 0.5          # the other side is never clipped by the min
    _, out, _ = _loss_f64(cu, x, tok, old, logp, adv, mask, 0.2, 0.0)
    assert (np.abs(out["g"]) > 0).all()


def test_gradient_by_central_finite_differences():
    cu, x, tok, adv, mask = _random_batch(M=4, V=7, seed=11)
    T, V = x.shape
    logp = torch.log_softmax(torch.from_numpy(x), -1).numpy()[np.arange(T), tok]
    rng = np.random.default_rng(5)
    old = logp + rng.normal(0, 0.15, T)           # some tokens beyond the clip range
    ref = logp + rng.normal(0, 0.1, T)
    _, out, _ = _loss_f64(cu, x, tok, old, ref, adv, mask, 0.2, 0.04)
    h = 1e-6
    fd = np.zeros_like(x)
    for t in range(T):
        for v in range(V):
            xp, xm = x.copy(), x.copy()
            xp[t, v] += h
            xm[t, v] -= h
            fd[t, v] = (_loss_f64(cu, xp, tok, old, ref, adv, mask, 0.2, 0.04)[0]
                        - _loss_f64(cu, xm, tok, old, ref, adv, mask, 0.2, 0.04)[0]) / (2 * h)
    np.testing.assert_allclose(out["dlogits"], fd, rtol=1e-6, atol=2e-9)
    np.testing.assert_allclose(out["dlogits"].sum(axis=1), 0.0, atol=1e-15)
    assert (out["dlogits"][mask == 0] == 0).all()


def test_sequence_mean_then_batch_mean_and_empty_sequences():
    """L_PODS averages tokens within a rollout, then rollouts; a fully masked rollout adds 0."""
    ell = np.array([1.0, 3.0, 10.0, 7.0, 7.0, 7.0])
    cu = np.array([0, 2, 3, 6], np.int64)
    assert oracle.grpo_loss(ell, np.ones(6, np.uint8), cu) == pytest.approx((2.0 + 10.0 + 7.0) / 3)
    mask = np.array([1, 0, 0, 1, 1, 0], np.uint8)
    assert oracle.grpo_loss(ell, mask, cu) == pytest.approx((1.0 + 0.0 + 7.0) / 3)
    np.testing.assert_allclose(oracle.seq_weights(mask, cu), [1 / 3, 0.0, 1 / 6])


def test_bf16_and_f64_entry_points_agree_and_flag_bad_tokens():
    T, V = 6, 16
    bits = wl.f32_to_bf16_bits(RNG.normal(0, 2, size=(T, V)).astype(np.float32))
    x = wl.bf16_bits_to_f32(bits).astype(np.float64)
    tok = RNG.integers(0, V, T).astype(np.int32)
    old = RNG.normal(-2.5, 0.3, T).astype(np.float32)
    ref = RNG.normal(-2.5, 0.3, T).astype(np.float32)
    cu, sor, mask = _one_seq(T)
    adv = np.array([0.7], np.float32)
    eps, beta = np.float32(0.2), np.float32(0.04)
    a = oracle.grpo_rows(bits, tok, old, ref, adv, [1 / T], sor, mask, eps, beta)
    b = oracle.grpo_rows_f64(x, tok, old, ref, adv, [1 / T], sor, mask, float(eps), float(beta))
    for key in ("logp", "ell", "g", "dlogits"):
        np.testing.assert_array_equal(a[key], b[key])
    assert a["bad_tokens"] == 0
    tok[2] = V
    assert oracle.grpo_rows(bits, tok, old, ref, adv, [1 / T], sor, mask, eps, beta)["bad_tokens"] == 1


def test_compact_concatenates_kept_rollouts_in_group_order():
    G, n, m = 2, 4, 2
    lengths = np.array([3, 1, 2, 4, 2, 2, 1, 3], np.int32)
    src = np.arange(8 * 4, dtype=np.int32).reshape(8, 4)
    idx = np.array([[1, 3], [0, 2]], np.int32)
    cu, toks, streams, sor = oracle.compact(idx, n, lengths, src, [src.astype(np.float32) * 0.5])
    assert list(cu) == [0, 1, 5, 7, 8]
    assert list(toks) == [4, 12, 13, 14, 15, 16, 17, 24]
    np.testing.assert_array_equal(streams[0], toks * 0.5)
    assert list(sor) == [0, 1, 1, 1, 1, 2, 2, 3]
