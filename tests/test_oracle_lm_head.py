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
