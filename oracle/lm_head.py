"""Log-probability of the sampled token when the logits are the LM-head projection.  TEST INFRASTRUCTURE ONLY.

pi_theta(o_{i,t} | p, o_{i,<t}) of L_GRPO (Section 3.1) and L_PODS (Section 3.2) is, for a transformer policy,
the softmax over the vocabulary of  logits[t, :] = hidden[t, :] . W^T  taken at the sampled token.  The oracle is
that definition written out in fp64 on the bf16 inputs: a library matrix product for the projection, then the
two-pass log-softmax (maximum, sum of exponentials).  The logits are NOT rounded to bf16 on the way: they are an
intermediate, not an input.  Pinned in tests/test_oracle_lm_head.py (a hand-worked case, closed forms, the
framework's fp64 log_softmax, and the loss oracle's log-probs where the logits are exactly representable).

loss_grad_from_hidden adds the objective on those logits and its gradient with respect to hidden and W (the chain
rule through the projection); pinned there by central finite differences of the loss in single entries of hidden
and W, closed forms at a uniform policy, and the framework's fp64 automatic differentiation.
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


def loss_grad_from_hidden(hidden_bits, w_bits, tokens, old_logp, ref_logp, adv, seq_weight, seq_of_row, mask,
                          eps, beta, block_rows=256):
    """L_PODS (Section 3.2) when the logits are the projection hidden W^T, with its gradient carried back through
    the projection by the chain rule.

    Per block of rows: logits = hidden W^T in fp64 (a library product), the token terms of the objective and
    d loss / d logits from the loss oracle's fp64 row routine (the Section 3.2 formula), then
        dhidden[t, :] = sum_v dlogits[t, v] W[v, :]          dW[v, :] = sum_t dlogits[t, v] hidden[t, :]
    which is all the projection adds.  Nothing is rounded on the way.  old_logp, ref_logp (None iff beta == 0) and
    adv are the fp32 inputs widened; eps and beta fp32 values widened.

    Returns dict(logp, ell, g [T]; dhidden [T,d]; dW [V,d]; abs_dhidden [T,d] = sum_v |dlogits||W| and
    abs_dW [V,d] = sum_t |dlogits||hidden|, the magnitudes the sums are made of; all float64)."""
    from . import grpo_rows_f64               # the package imports this module last

    h = _bf16_bits_to_f64(hidden_bits)
    w = _bf16_bits_to_f64(w_bits)
    T, d = h.shape
    V = w.shape[0]
    tok = np.asarray(tokens, np.int64).copy()
    tok[(tok < 0) | (tok >= V)] = 0
    old = np.asarray(old_logp, np.float32).astype(np.float64)
    ref = None if ref_logp is None else np.asarray(ref_logp, np.float32).astype(np.float64)
    a = np.asarray(adv, np.float32).astype(np.float64)
    sw = np.asarray(seq_weight, np.float64)
    seq = np.asarray(seq_of_row, np.int32)
    msk = np.ones(T, np.uint8) if mask is None else np.asarray(mask, np.uint8)
    e, b = float(np.float32(eps)), float(np.float32(beta))
    out = {k: np.empty(T) for k in ("logp", "ell", "g")}
    dhidden = np.zeros((T, d))
    abs_dhidden = np.zeros((T, d))
    dW = np.zeros((V, d))
    abs_dW = np.zeros((V, d))
    aw, ah = np.abs(w), np.abs(h)
    for lo in range(0, T, block_rows):
        hi = min(T, lo + block_rows)
        x = h[lo:hi] @ w.T
        r = grpo_rows_f64(x, tok[lo:hi].astype(np.int32), old[lo:hi], None if ref is None else ref[lo:hi], a, sw,
                          seq[lo:hi], msk[lo:hi], e, b)
        for k in out:
            out[k][lo:hi] = r[k]
        dl = r["dlogits"]
        dhidden[lo:hi] = dl @ w
        abs_dhidden[lo:hi] = np.abs(dl) @ aw
        dW += dl.T @ h[lo:hi]
        abs_dW += np.abs(dl).T @ ah[lo:hi]
    out.update(dhidden=dhidden, dW=dW, abs_dhidden=abs_dhidden, abs_dW=abs_dW)
    return out
