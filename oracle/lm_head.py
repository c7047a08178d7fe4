"""Log-probability of the sampled token when the logits are the LM-head projection.  TEST INFRASTRUCTURE ONLY.

pi_theta(o_{i,t} | p, o_{i,<t}) of L_GRPO (Section 3.1) and L_PODS (Section 3.2) is, for a transformer policy,
the softmax over the vocabulary of  logits[t, :] = hidden[t, :] . W^T  taken at the sampled token.  The oracle is
that definition written out in fp64 on the bf16 inputs: a library matrix product for the projection, then the
two-pass log-softmax (maximum, sum of exponentials).  The logits are NOT rounded to bf16 on the way: they are an
intermediate, not an input.  Pinned in tests/test_oracle_lm_head.py (a hand-worked case, closed forms, the
framework's fp64 log_softmax, and the loss oracle's log-probs where the logits are exactly representable).
"""
import numpy as np


def _bf16_bits_to_f64(bits):
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def logp_from_hidden(hidden_bits, w_bits, tokens, block_rows=256):
    """hidden_bits [T,d], w_bits [V,d]: uint16 bf16 bit patterns; tokens [T] int32.

    Returns dict(logp [T], lse [T], row_max [T], x_tok [T]: float64; bad_tokens: ids outside [0,V), read as 0)."""
    h = _bf16_bits_to_f64(hidden_bits)
    w = _bf16_bits_to_f64(w_bits)
    T, d = h.shape
    V = w.shape[0]
    assert w.shape[1] == d
    tok = np.asarray(tokens, np.int64).copy()
    bad = (tok < 0) | (tok >= V)
    tok[bad] = 0
    logp = np.empty(T)
    lse = np.empty(T)
    row_max = np.empty(T)
    x_tok = np.empty(T)
    for lo in range(0, T, block_rows):
        hi = min(T, lo + block_rows)
        x = h[lo:hi] @ w.T                                  # logits of the block, fp64
        mx = x.max(axis=1)
        z = np.exp(x - mx[:, None]).sum(axis=1)
        row_max[lo:hi] = mx
        lse[lo:hi] = mx + np.log(z)
        x_tok[lo:hi] = x[np.arange(hi - lo), tok[lo:hi]]
        logp[lo:hi] = x_tok[lo:hi] - lse[lo:hi]
    return {"logp": logp, "lse": lse, "row_max": row_max, "x_tok": x_tok, "bad_tokens": int(bad.sum())}
