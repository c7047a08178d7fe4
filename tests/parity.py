"""Helpers shared by the parity tests: build one batch from a workload, run the oracle over it,
and compare arrays under the stated tolerances.  Not collected by pytest."""
import dataclasses

import numpy as np

import oracle
from paper_2504_13818_b200 import workloads as wl

# Tolerances of the parity bar: indices bit-exact; advantages rel <= 1e-6; per-token log-prob abs
# <= 1e-3; loss rel <= 1e-4; dlogits within 2 bf16 ulps (ulp taken at max(|oracle|, 2^-126), the
# oracle value first rounded to bf16).
ADV_RTOL = 1e-6
LOGP_ATOL = 1e-3
LOSS_RTOL = 1e-4
LOSS_COND = 1e3         # the loss is a mean of signed rollout terms; cancellation beyond this factor is not resolved
DLOGITS_ULPS = 2
CLIP_MARGIN = 1e-5      # rows whose min() is closer than this to switching branch are compared on logp only


def shrink(w, **kw):
    return dataclasses.replace(w, **kw)


def bf16_round(x64):
    """fp64 -> nearest-even bf16, returned as float64 values."""
    bits = wl.f32_to_bf16_bits(np.asarray(x64, np.float64).astype(np.float32))
    # the double rounding fp64 -> fp32 -> bf16 differs from direct rounding only on exact fp32 ties
    return wl.bf16_bits_to_f32(bits).astype(np.float64)


def bf16_ulp(x64):
    a = np.maximum(np.abs(x64), 2.0 ** -126)
    _, e = np.frexp(a)                       # a = f * 2^e, f in [0.5, 1)
    return np.ldexp(1.0, e - 1 - 7)


LOGP_RESOLUTION = 5e-7  # one fp32 ulp of a log-prob in [-8, -4): the grain of the old/ref inputs and the logp output


# A row "uses the allowance" when its relative slack is worth more than a quarter of a bf16 ulp
# (|x| / ulp(x) < 2^8 for every bf16 x); every other row is held to the literal 2-ulp bound.
SLACK_ROW_THRESHOLD = 0.25 / 256.0

RECORD_PATH = None      # set by conftest: the JSON-lines file the achieved maxima are appended to


def record(case, **values):
    """Append the achieved parity maxima of one test case to the record file (and to stdout)."""
    import json
    line = json.dumps({"case": case, **{k: (float(v) if isinstance(v, (float, np.floating)) else v)
                                        for k, v in values.items()}})
    print("parity:", line)
    if RECORD_PATH:
        try:
            with open(RECORD_PATH, "a") as f:
                f.write(line + "\n")
        except OSError:
            pass


def dlogits_report(gpu_bits, oracle64, slack, skip_rows=None):
    """Gradient parity of a block of rows.  Rows whose allowance is below SLACK_ROW_THRESHOLD are held to the
    literal bound (no allowance taken off); the others get the allowance.  Returns the worst literal error of
    the first kind, the worst conditioned error of the second kind, and how many rows were of the second kind."""
    want = bf16_round(oracle64)
    diff = np.abs(wl.bf16_bits_to_f32(gpu_bits).astype(np.float64) - want)
    ulp = bf16_ulp(want)
    row_ulps = (diff / ulp).max(axis=1) if diff.shape[1] else np.zeros(diff.shape[0])
    slack = np.zeros(diff.shape[0]) if slack is None else np.asarray(slack, np.float64)
    live = np.ones(diff.shape[0], bool) if skip_rows is None else ~np.asarray(skip_rows, bool)
    allowed = (slack > SLACK_ROW_THRESHOLD) & live
    literal = live & ~allowed
    cond = 0.0
    if allowed.any():
        cond = float((np.maximum(diff[allowed] - slack[allowed, None] * np.abs(oracle64[allowed]), 0.0) / ulp[allowed]).max())
    return {"literal_ulps": float(row_ulps[literal].max()) if literal.any() else 0.0,
            "allowance_rows": int(allowed.sum()), "allowance_ulps": cond, "rows": int(live.sum())}


def assert_dlogits_close(rep):
    assert rep["literal_ulps"] <= DLOGITS_ULPS, "dlogits off by %.2f bf16 ulps" % rep["literal_ulps"]
    assert rep["allowance_ulps"] <= DLOGITS_ULPS, ("dlogits off by %.2f bf16 ulps beyond the row allowance (%d rows)"
                                                   % (rep["allowance_ulps"], rep["allowance_rows"]))


def dlogits_ulp_error(gpu_bits, oracle64, slack=None):
    """|gpu - bf16(oracle)| in units of the bf16 ulp at the oracle value.

    ``slack`` [T] (optional) is a relative allowance per row (the uncertainty of the row factor g_t,
    see gradient_slack), taken off the error first."""
    want = bf16_round(oracle64)
    got = wl.bf16_bits_to_f32(gpu_bits).astype(np.float64)
    err = np.abs(got - want)
    if slack is not None:
        err = np.maximum(err - np.asarray(slack)[:, None] * np.abs(oracle64), 0.0)
    return err / bf16_ulp(want)


def gradient_slack(b, want, rows=None):
    """Per-row allowance for the row factor g_t when it is itself a cancellation.

    g_t = w (-a rho [unclipped] + beta (1 - e^d)) with d = ref - logp.  For a token with zero advantage
    or on the clipped side only beta (1 - e^d) ~ -beta d is left, and when |d| is of the order of the
    fp32 grain of the log-probs (ref_logp is an fp32 input) g_t depends on digits of logp that fp32
    softmax statistics do not carry: two bf16 ulps of such a g_t are out of reach by construction.  The
    allowance is the relative uncertainty |dg/dlogp| LOGP_RESOLUTION / |g_t| of the row factor; on rows
    whose g_t is not a cancellation it is ~1e-6, far below a bf16 ulp (4e-3), so the 2-ulp bar stands."""
    w = b["w"]
    sl = slice(None) if rows is None else rows
    sw = oracle.seq_weights(b["mask"], b["cu"])[b["seq_of_row"][sl]] * (b["mask"][sl] != 0)
    a = np.abs(b["adv32"][b["seq_of_row"][sl]].astype(np.float64))
    with np.errstate(over="ignore", invalid="ignore"):
        rho = np.exp(want["logp"] - b["old"][sl].astype(np.float64))
        ed = np.exp(b["ref"][sl].astype(np.float64) - want["logp"])
        dg = np.where(sw > 0, LOGP_RESOLUTION * sw * (a * rho + float(np.float32(w.beta)) * ed), 0.0)
    g = np.abs(want["g"])
    return np.where(g > 0, dg / np.where(g > 0, g, 1.0), 0.0)


def assert_adv_close(gpu_adv, oracle_adv):
    o = np.asarray(oracle_adv, np.float64)
    g = np.asarray(gpu_adv, np.float64)
    err = np.abs(g - o)
    tol = ADV_RTOL * np.abs(o) + 1e-12
    assert (err <= tol).all(), "adv rel err %.3g" % (err / np.maximum(np.abs(o), 1e-300)).max()
    assert (g[o == 0] == 0).all()


def build_batch(w, lengths_all=None):
    """All host-side inputs of one step for workload ``w`` plus the oracle's results.

    Selection, compaction and the loss are chained on the oracle's own outputs."""
    rewards = wl.make_rewards(w)
    lengths, src_tokens = wl.make_rollouts(w)
    sel = oracle.select(rewards, w.m)
    cu, tokens, _, seq_of_row = oracle.compact(sel["idx"], w.n, lengths, src_tokens)
    logits = wl.make_logits_host(w, tokens)
    logp_tilde = wl.host_logp_tilde(logits, tokens)
    old, ref = wl.make_old_ref(w, logp_tilde)
    mask = np.ones(tokens.shape[0], np.uint8)
    return {"w": w, "rewards": rewards, "lengths": lengths, "src_tokens": src_tokens, "sel": sel,
            "cu": cu, "tokens": tokens, "seq_of_row": seq_of_row, "logits": logits, "old": old, "ref": ref,
            "mask": mask, "adv32": sel["adv"].astype(np.float32).reshape(-1)}


def oracle_loss(b, rows=None, want_dlogits=True):
    """Oracle rows (all, or the given row indices) and, when all rows are run, the loss."""
    w = b["w"]
    sw = oracle.seq_weights(b["mask"], b["cu"])
    sl = slice(None) if rows is None else rows
    out = oracle.grpo_rows(b["logits"][sl], b["tokens"][sl], b["old"][sl], b["ref"][sl], b["adv32"], sw,
                           b["seq_of_row"][sl], b["mask"][sl], w.eps, w.beta, want_dlogits=want_dlogits)
    if rows is None:
        out["loss"] = oracle.grpo_loss(out["ell"], b["mask"], b["cu"])
    return out


def loss_scale(ell, mask, cu):
    """(1/M) sum_i |mean_t ell_{i,t}|: the size of the rollout terms the loss is a signed mean of."""
    M = cu.shape[0] - 1
    tot = 0.0
    for i in range(M):
        sl = slice(int(cu[i]), int(cu[i + 1]))
        mk = mask[sl] != 0
        if mk.any():
            tot += abs(float(ell[sl][mk].mean()))
    return tot / M


def loss_errors(gpu_loss, want, b):
    """Literal relative error of the loss, and the error relative to max(|loss|, scale / LOSS_COND)."""
    scale = loss_scale(want["ell"], b["mask"], b["cu"])
    d = abs(gpu_loss - want["loss"])
    return {"loss_rel_literal": d / abs(want["loss"]) if want["loss"] != 0 else (0.0 if d == 0 else float("inf")),
            "loss_rel_conditioned": d / max(abs(want["loss"]), scale / LOSS_COND, 1e-300),
            "loss": want["loss"], "loss_term_scale": scale}


def assert_loss_close(gpu_loss, want, b):
    """|gpu - oracle| <= 1e-4 max(|oracle|, scale / 1e3).

    With zero-sum advantages the loss is a cancelling sum (config 1: terms of +-0.06 add up to 1.7e-6);
    relative error against the result alone would then demand more digits than the stated per-token
    log-prob tolerance carries.  The bound is relative to the loss wherever the sum cancels by less than
    a factor of 1000, and to the size of its terms beyond that."""
    scale = loss_scale(want["ell"], b["mask"], b["cu"])
    tol = LOSS_RTOL * max(abs(want["loss"]), scale / LOSS_COND)
    assert abs(gpu_loss - want["loss"]) <= tol, (gpu_loss, want["loss"], scale)
