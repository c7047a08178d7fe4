"""Pins of oracle.lm_head.logp_from_hidden against what the mathematics fixes (CPU only):
a hand-worked case, closed forms, shift invariance, the framework's fp64 routines, and agreement with the loss
oracle's log-probs on logits that bf16 represents exactly."""
import os

import numpy as np
import torch

import oracle
from oracle import lm_head
from paper_2504_13818_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "lm_head_case.txt")


def _bits(a):
    return wl.f32_to_bf16_bits(np.asarray(a, np.float32))


def test_hand_worked_case():
    hidden = _bits([[1.0, 2.0], [0.5, -1.0]])
    W = _bits([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]])
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    tokens = np.array([int(r[1]) for r in rows], np.int32)
    out = lm_head.logp_from_hidden(hidden, W, tokens)
    for r in rows:
        t = int(r[0])
        logits = np.array([float(v) for v in r[2:5]])
        assert abs(out["row_max"][t] - logits.max()) == 0.0
        assert abs(out["x_tok"][t] - logits[int(r[1])]) == 0.0
        assert abs(out["lse"][t] - float(r[5])) < 1e-14
        assert abs(out["logp"][t] - float(r[6])) < 1e-14


def test_closed_forms():
    rng = np.random.default_rng(0)
    T, V, d = 5, 37, 16
    W = _bits(rng.normal(size=(V, d)))
    tokens = rng.integers(0, V, T, dtype=np.int32)
    # zero hidden state: every logit is 0, the policy is uniform
    out = lm_head.logp_from_hidden(_bits(np.zeros((T, d))), W, tokens)
    np.testing.assert_allclose(out["logp"], -np.log(V), rtol=0, atol=1e-15)
    # W = scaled unit rows: logits are the hidden features themselves (V = d)
    h = rng.normal(size=(T, d)).astype(np.float32)
    hb = _bits(h)
    hv = wl.bf16_bits_to_f32(hb).astype(np.float64)
    eye2 = _bits(2.0 * np.eye(d))
    tok = rng.integers(0, d, T, dtype=np.int32)
    out = lm_head.logp_from_hidden(hb, eye2, tok)
    x = 2.0 * hv
    want = x[np.arange(T), tok] - np.log(np.exp(x).sum(axis=1))
    np.testing.assert_allclose(out["logp"], want, rtol=0, atol=1e-13)
    # one logit far above the rest: log-prob of that token -> 0, of any other -> -(gap)
    Wd = np.zeros((V, d), np.float32)
    Wd[3, 0] = 64.0
    hd = np.zeros((2, d), np.float32)
    hd[:, 0] = 1.0
    out = lm_head.logp_from_hidden(_bits(hd), _bits(Wd), np.array([3, 4], np.int32))
    assert abs(out["logp"][0]) < 1e-15 and abs(out["logp"][1] + 64.0) < 1e-12


def test_adding_the_same_vector_to_every_row_of_w_changes_no_probability():
    """softmax is invariant to a shift of all logits of a row: (W + 1 c^T) shifts row t by hidden[t] . c."""
    rng = np.random.default_rng(1)
    T, V, d = 6, 20, 8
    h = rng.integers(-3, 4, size=(T, d)).astype(np.float32)        # small integers: every product is exact in bf16
    W = rng.integers(-3, 4, size=(V, d)).astype(np.float32)
    c = rng.integers(-2, 3, size=(1, d)).astype(np.float32)
    tok = rng.integers(0, V, T, dtype=np.int32)
    a = lm_head.logp_from_hidden(_bits(h), _bits(W), tok)
    b = lm_head.logp_from_hidden(_bits(h), _bits(W + c), tok)
    np.testing.assert_allclose(a["logp"], b["logp"], rtol=0, atol=1e-12)
    np.testing.assert_allclose(b["lse"] - a["lse"], (h.astype(np.float64) @ c.T.astype(np.float64))[:, 0], atol=1e-12)


def test_against_the_framework_fp64_matmul_and_log_softmax():
    rng = np.random.default_rng(2)
    T, V, d = 33, 1000, 96
    hb, wb = _bits(rng.normal(size=(T, d))), _bits(rng.normal(size=(V, d)) / np.sqrt(d) * 3.0)
    tok = rng.integers(0, V, T, dtype=np.int32)
    out = lm_head.logp_from_hidden(hb, wb, tok, block_rows=7)      # several blocks and a ragged last one
    h = torch.from_numpy(wl.bf16_bits_to_f32(hb)).double()
    w = torch.from_numpy(wl.bf16_bits_to_f32(wb)).double()
    ls = torch.log_softmax(h @ w.T, dim=-1)
    want = ls[torch.arange(T), torch.from_numpy(tok).long()].numpy()
    np.testing.assert_allclose(out["logp"], want, rtol=0, atol=1e-12)
    # a transposed operand or a wrong token column would not survive this
    assert np.abs(out["logp"] - ls[torch.arange(T), (torch.from_numpy(tok).long() + 1) % V].numpy()).max() > 1e-3


def test_agrees_with_the_loss_oracle_where_bf16_holds_the_logits_exactly():
    """Small-integer hidden states and weights give small-integer logits, which bf16 represents exactly: the loss
    oracle's log-prob on those logits (a different code path: C, two-pass over bf16 inputs) must be the same."""
    rng = np.random.default_rng(3)
    T, V, d = 12, 64, 4
    h = rng.integers(-2, 3, size=(T, d)).astype(np.float32)
    W = rng.integers(-2, 3, size=(V, d)).astype(np.float32)
    tok = rng.integers(0, V, T, dtype=np.int32)
    out = lm_head.logp_from_hidden(_bits(h), _bits(W), tok)
    logits = (h.astype(np.float64) @ W.T.astype(np.float64)).astype(np.float32)
    assert np.abs(logits).max() <= 128                             # integers up to 2^8 are exact in bf16
    bits = wl.f32_to_bf16_bits(logits)
    assert (wl.bf16_bits_to_f32(bits) == logits).all()
    cu = np.array([0, T], np.int64)
    mask = np.ones(T, np.uint8)
    rows = oracle.grpo_rows(bits, tok, np.zeros(T, np.float32), np.zeros(T, np.float32), np.ones(1, np.float32),
                            oracle.seq_weights(mask, cu), np.zeros(T, np.int32), mask, 0.2, 0.0, want_dlogits=False)
    np.testing.assert_allclose(out["logp"], rows["logp"], rtol=0, atol=1e-13)


def test_token_ids_out_of_range_are_counted_and_read_as_zero():
    hb, wb = _bits(np.ones((3, 4))), _bits(np.arange(20).reshape(5, 4) / 8.0)
    out = lm_head.logp_from_hidden(hb, wb, np.array([5, -1, 2], np.int32))
    ref = lm_head.logp_from_hidden(hb, wb, np.array([0, 0, 2], np.int32))
    assert out["bad_tokens"] == 2 and (out["logp"] == ref["logp"]).all()


# ---------------------------------------------------------------------------------------------------------
# loss_grad_from_hidden: the objective on projected logits and its gradient through the projection
# ---------------------------------------------------------------------------------------------------------

def _case(seed, T=9, V=13, d=6, M=3, beta=0.04, masked=()):
    rng = np.random.default_rng(seed)
    hb = _bits(rng.normal(size=(T, d)))
    wb = _bits(rng.normal(size=(V, d)))
    tok = rng.integers(0, V, T, dtype=np.int32)
    cu = np.array([0, 2, 5, T], np.int64)[: M + 1]
    cu[-1] = T
    mask = np.ones(T, np.uint8)
    mask[list(masked)] = 0
    adv = np.array([1.0, -0.5, 0.75], np.float32)[:M]
    base = lm_head.logp_from_hidden(hb, wb, tok)["logp"]
    old = (base + rng.normal(0, 0.3, T)).astype(np.float32)        # wide enough that some tokens clip
    ref = (base + rng.normal(0, 0.3, T)).astype(np.float32)
    return dict(hb=hb, wb=wb, tok=tok, cu=cu, mask=mask, adv=adv, old=old, ref=ref, eps=0.2, beta=beta)


def _loss_of(c, h, w):
    """The objective as a function of fp64 hidden and W, from the loss oracle's row routine and outer sums."""
    T = h.shape[0]
    sw = oracle.seq_weights(c["mask"], c["cu"])
    rows = oracle.grpo_rows_f64(h @ w.T, c["tok"], c["old"].astype(np.float64), c["ref"].astype(np.float64),
                                c["adv"].astype(np.float64), sw, oracle.seq_of_rows(c["cu"]), c["mask"],
                                float(np.float32(c["eps"])), float(np.float32(c["beta"])), want_dlogits=False)
    return oracle.grpo_loss(rows["ell"], c["mask"], c["cu"])


def _grad_of(c):
    sw = oracle.seq_weights(c["mask"], c["cu"])
    return lm_head.loss_grad_from_hidden(c["hb"], c["wb"], c["tok"], c["old"], c["ref"], c["adv"], sw,
                                         oracle.seq_of_rows(c["cu"]), c["mask"], c["eps"], c["beta"], block_rows=4)


def test_gradient_by_central_finite_differences_in_single_entries():
    c = _case(10, masked=(4,))
    out = _grad_of(c)
    h = wl.bf16_bits_to_f32(c["hb"]).astype(np.float64)
    w = wl.bf16_bits_to_f32(c["wb"]).astype(np.float64)
    step = 1e-6
    worst = 0.0
    for (t, j) in [(0, 0), (3, 5), (4, 2), (8, 1), (6, 3)]:
        hp, hm = h.copy(), h.copy()
        hp[t, j] += step
        hm[t, j] -= step
        fd = (_loss_of(c, hp, w) - _loss_of(c, hm, w)) / (2 * step)
        worst = max(worst, abs(fd - out["dhidden"][t, j]))
    for (v, j) in [(0, 0), (12, 5), (int(c["tok"][2]), 1), (int(c["tok"][7]), 4), (5, 2)]:
        wp, wm = w.copy(), w.copy()
        wp[v, j] += step
        wm[v, j] -= step
        fd = (_loss_of(c, h, wp) - _loss_of(c, h, wm)) / (2 * step)
        worst = max(worst, abs(fd - out["dW"][v, j]))
    assert worst < 1e-9
    assert np.abs(out["dhidden"][4]).max() == 0.0                  # a masked token sends nothing back
    assert np.abs(out["dhidden"]).max() > 1e-3 and np.abs(out["dW"]).max() > 1e-3


def test_gradient_closed_forms_at_a_uniform_policy():
    """W = 0 or hidden = 0 makes every logit 0 and the policy uniform; on-policy (old = -ln V) without KL the token
    factor is g_t = -a_i / (M |o_i|), so
      hidden = 0:  dhidden[t] = g_t (W[tok_t] - mean_v W[v]),   dW = 0;
      W = 0:       dW[v] = sum_t g_t ([v == tok_t] - 1/V) hidden[t],   dhidden = 0."""
    rng = np.random.default_rng(11)
    T, V, d, M = 6, 7, 4, 2
    cu = np.array([0, 2, T], np.int64)
    mask = np.ones(T, np.uint8)
    sw = oracle.seq_weights(mask, cu)
    seq = oracle.seq_of_rows(cu)
    adv = np.array([1.5, -0.5], np.float32)
    tok = rng.integers(0, V, T, dtype=np.int32)
    old = np.full(T, -np.log(V), np.float32)
    g = -(adv.astype(np.float64) * sw)[seq] * np.exp(-np.log(V) - old.astype(np.float64))
    onehot = np.zeros((T, V))
    onehot[np.arange(T), tok] = 1.0
    wv = wl.bf16_bits_to_f32(_bits(rng.normal(size=(V, d)))).astype(np.float64)
    out = lm_head.loss_grad_from_hidden(_bits(np.zeros((T, d))), _bits(wv), tok, old, None, adv, sw, seq, mask, 0.2, 0.0)
    np.testing.assert_allclose(out["dhidden"], g[:, None] * (wv[tok] - wv.mean(axis=0)), rtol=0, atol=1e-15)
    assert np.abs(out["dW"]).max() == 0.0
    hv = wl.bf16_bits_to_f32(_bits(rng.normal(size=(T, d)))).astype(np.float64)
    out = lm_head.loss_grad_from_hidden(_bits(hv), _bits(np.zeros((V, d))), tok, old, None, adv, sw, seq, mask, 0.2, 0.0)
    np.testing.assert_allclose(out["dW"], ((onehot - 1.0 / V) * g[:, None]).T @ hv, rtol=0, atol=1e-15)
    assert np.abs(out["dhidden"]).max() == 0.0


def test_gradient_against_the_framework_fp64_automatic_differentiation():
    c = _case(12, T=17, V=29, d=10, masked=(1, 16))
    out = _grad_of(c)
    h = torch.from_numpy(wl.bf16_bits_to_f32(c["hb"])).double().requires_grad_(True)
    w = torch.from_numpy(wl.bf16_bits_to_f32(c["wb"])).double().requires_grad_(True)
    T = h.shape[0]
    seq = torch.from_numpy(oracle.seq_of_rows(c["cu"])).long()
    lp = torch.log_softmax(h @ w.T, dim=-1)[torch.arange(T), torch.from_numpy(c["tok"]).long()]
    a = torch.from_numpy(c["adv"]).double()[seq]
    rho = torch.exp(lp - torch.from_numpy(c["old"]).double())
    eps = float(np.float32(c["eps"]))
    surrogate = torch.minimum(rho * a, torch.clamp(rho, 1 - eps, 1 + eps) * a)
    dd = torch.from_numpy(c["ref"]).double() - lp
    ell = -surrogate + float(np.float32(c["beta"])) * (torch.exp(dd) - dd - 1)
    wts = torch.from_numpy(oracle.seq_weights(c["mask"], c["cu"]))[seq] * torch.from_numpy(c["mask"]).double()
    (wts * ell).sum().backward()
    np.testing.assert_allclose(out["dhidden"], h.grad.numpy(), rtol=0, atol=1e-14)
    np.testing.assert_allclose(out["dW"], w.grad.numpy(), rtol=0, atol=1e-14)
    np.testing.assert_allclose(out["logp"], lp.detach().numpy(), rtol=0, atol=1e-13)
    # the magnitudes bound the sums they are made of
    assert (np.abs(out["dhidden"]) <= out["abs_dhidden"] + 1e-18).all() and (np.abs(out["dW"]) <= out["abs_dW"] + 1e-18).all()
