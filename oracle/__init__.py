"""CPU oracle for the PODS hot path.  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the product (the CUDA library and its binding) never does, and this
package imports nothing from the product.

Four parts:
  * ``definition``  - the selection rule as the paper defines it (maximise the
    variance over every m-subset), exact rational arithmetic, tiny inputs only;
  * ``pods_oracle.c`` (wrapped here) - Algorithm 2, the advantages and the
    GRPO-PODS objective with its gradient, fp64, any size;
  * ``compact`` - concatenation of the kept rollouts (text after Algorithm 1);
  * ``lm_head`` - the token log-probability when the logits are the projection hidden W^T
    (pi_theta of Sections 3.1 / 3.2), fp64.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

RULE_MAXVAR, RULE_MAXREWARD, RULE_RANDOM, RULE_PERCENTILE = 0, 1, 2, 3
FLAG_ADV_BEFORE, FLAG_STD_SAMPLE = 1, 2

_lib = None


def _load():
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build()
    lib = C.CDLL(path)
    p = C.c_void_p
    lib.oracle_num_threads.restype = C.c_int
    lib.oracle_set_threads.argtypes = [C.c_int]
    lib.oracle_philox4x32_10.argtypes = [p, p, p]
    lib.oracle_select.restype = C.c_int
    lib.oracle_select.argtypes = [p, C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_uint64,
                                  C.c_uint32, p, p, p, p]
    lib.oracle_seq_weights.argtypes = [p, p, C.c_int64, p]
    lib.oracle_grpo_rows.restype = C.c_int64
    lib.oracle_grpo_rows.argtypes = [p, C.c_int64, C.c_int64, C.c_int32, p, p, p, p, p, p, p,
                                     C.c_float, C.c_float, p, p, p, p, p]
    lib.oracle_grpo_rows_f64.argtypes = [p, C.c_int64, C.c_int32, p, p, p, p, p, p, p,
                                         C.c_double, C.c_double, p, p, p, p]
    lib.oracle_grpo_loss.restype = C.c_double
    lib.oracle_grpo_loss.argtypes = [p, p, p, C.c_int64]
    _lib = lib
    return lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _arr(a, dtype):
    return None if a is None else np.ascontiguousarray(a, dtype=dtype)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_threads(t: int) -> None:
    _load().oracle_set_threads(int(t))


def philox4x32_10(ctr, key):
    ctr = _arr(ctr, np.uint32)
    key = _arr(key, np.uint32)
    out = np.empty(4, np.uint32)
    _load().oracle_philox4x32_10(_ptr(ctr), _ptr(key), _ptr(out))
    return out


def select(rewards, m, rule=RULE_MAXVAR, seed=0, flags=0):
    """Down-sample every group of ``rewards`` [G,n] to m rollouts.

    Returns dict(idx [G,m] int32 ascending, adv [G,m] float64, k [G] int32,
    gap [G] float64).  Algorithm 2 for RULE_MAXVAR; Section 3.2 for the others.
    """
    r = _arr(rewards, np.float32)
    assert r.ndim == 2
    G, n = r.shape
    idx = np.empty((G, m), np.int32)
    adv = np.empty((G, m), np.float64)
    k = np.empty(G, np.int32)
    gap = np.empty(G, np.float64)
    rc = _load().oracle_select(_ptr(r), G, n, m, rule, seed, flags, _ptr(idx), _ptr(adv), _ptr(k), _ptr(gap))
    if rc != 0:
        raise ValueError("oracle_select: invalid sizes")
    return {"idx": idx, "adv": adv, "k": k, "gap": gap}


def seq_weights(mask, cu_seqlens):
    """w_i = 1/(M |o_i|) with |o_i| the unmasked token count (L_PODS, Section 3.2)."""
    mask = _arr(mask, np.uint8)
    cu = _arr(cu_seqlens, np.int64)
    M = cu.shape[0] - 1
    w = np.empty(M, np.float64)
    _load().oracle_seq_weights(_ptr(mask), _ptr(cu), M, _ptr(w))
    return w


def seq_of_rows(cu_seqlens):
    cu = np.asarray(cu_seqlens, np.int64)
    return np.repeat(np.arange(cu.shape[0] - 1, dtype=np.int32), np.diff(cu))


def grpo_rows(logits_bits, tokens, old_logp, ref_logp, adv, seq_weight, seq_of_row, mask, eps, beta,
              want_dlogits=True):
    """Per-token terms of L_PODS and the logits gradient for a block of rows.

    ``logits_bits`` is a [T,V] uint16 array of bf16 bit patterns.  Returns dict
    with logp, ell, g, margin [T] float64, dlogits [T,V] float64 (or None) and
    bad_tokens (count of ids outside [0,V)).
    """
    lg = _arr(logits_bits, np.uint16)
    T, V = lg.shape
    tokens = _arr(tokens, np.int32)
    old_logp = _arr(old_logp, np.float32)
    ref_logp = _arr(ref_logp, np.float32)
    adv = _arr(adv, np.float32)
    seq_weight = _arr(seq_weight, np.float64)
    seq_of_row = _arr(seq_of_row, np.int32)
    mask = _arr(mask, np.uint8)
    logp = np.empty(T, np.float64)
    ell = np.empty(T, np.float64)
    g = np.empty(T, np.float64)
    margin = np.empty(T, np.float64)
    dlogits = np.empty((T, V), np.float64) if want_dlogits else None
    bad = _load().oracle_grpo_rows(_ptr(lg), V, T, V, _ptr(tokens), _ptr(old_logp), _ptr(ref_logp), _ptr(adv),
                                   _ptr(seq_weight), _ptr(seq_of_row), _ptr(mask),
                                   np.float32(eps), np.float32(beta),
                                   _ptr(logp), _ptr(ell), _ptr(g), _ptr(margin), _ptr(dlogits))
    return {"logp": logp, "ell": ell, "g": g, "margin": margin, "dlogits": dlogits, "bad_tokens": int(bad)}


def grpo_rows_f64(logits, tokens, old_logp, ref_logp, adv, seq_weight, seq_of_row, mask, eps, beta,
                  want_dlogits=True):
    """As grpo_rows but on fp64 logits [T,V] (for finite differences)."""
    lg = _arr(logits, np.float64)
    T, V = lg.shape
    tokens = _arr(tokens, np.int32)
    old_logp = _arr(old_logp, np.float64)
    ref_logp = _arr(ref_logp, np.float64)
    adv = _arr(adv, np.float64)
    seq_weight = _arr(seq_weight, np.float64)
    seq_of_row = _arr(seq_of_row, np.int32)
    mask = _arr(mask, np.uint8)
    logp = np.empty(T, np.float64)
    ell = np.empty(T, np.float64)
    g = np.empty(T, np.float64)
    dlogits = np.empty((T, V), np.float64) if want_dlogits else None
    _load().oracle_grpo_rows_f64(_ptr(lg), T, V, _ptr(tokens), _ptr(old_logp), _ptr(ref_logp), _ptr(adv),
                                 _ptr(seq_weight), _ptr(seq_of_row), _ptr(mask), float(eps), float(beta),
                                 _ptr(logp), _ptr(ell), _ptr(g), _ptr(dlogits))
    return {"logp": logp, "ell": ell, "g": g, "dlogits": dlogits}


def grpo_loss(ell, mask, cu_seqlens):
    """(1/M) sum_i (1/|o_i|) sum_t ell: the outer sums of L_PODS."""
    ell = _arr(ell, np.float64)
    mask = _arr(mask, np.uint8)
    cu = _arr(cu_seqlens, np.int64)
    return float(_load().oracle_grpo_loss(_ptr(ell), _ptr(mask), _ptr(cu), cu.shape[0] - 1))


from .definition import max_variance_subsets, variance_exact  # noqa: E402,F401
from .compact import compact  # noqa: E402,F401
from . import lm_head  # noqa: E402,F401
