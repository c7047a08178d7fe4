"""grpo_loss_from_hidden (CUDA, tensor cores) against the fp64 oracle: the objective on logits = hidden W^T and its
gradient with respect to hidden and W, the [T,V] logits and their gradient never stored in full.

Tolerances.  logp abs <= 1e-3 and the loss as everywhere else.  The gradients are sums of products
dlogits[t,v] W[v,j] (over v) and dlogits[t,v] hidden[t,j] (over t) in which the kernel rounds dlogits to bf16 - as the
unfused path's stored gradient is - so every term carries a relative error of at most 2^-8, the unit roundoff of bf16
(reached by values just above a power of two); the fp32 evaluation of the softmax (logits accumulated in fp32 over d
terms, the fp32 log-sum-exp) and the fp32 accumulation of the sums add a few 1e-5 relative to the terms, for which
2^-12 is allowed.  Hence, element by element,
    |gpu - oracle| <= (2^-8 + 2^-12) * sum |dlogits| |W|   (dhidden)      (2^-8 + 2^-12) * sum |dlogits| |hidden|   (dW),
the sums of magnitudes coming from the oracle; where one term dominates a sum the measured error comes within a few
per cent of 2^-8, as it must.  The bound assumes that no row's factor g_t is itself a cancellation
(reading of the dlogits tolerance for the unfused kernel); the inputs are drawn so that there is none, which is asserted.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle import lm_head
from paper_2504_13818_b200 import binding
from parity import LOGP_ATOL, LOSS_RTOL, record

pytestmark = pytest.mark.gpu

GRAD_RTOL = 2.0 ** -8 + 2.0 ** -12
EPS, BETA = 0.2, 0.04


def _inputs(T, V, d, M, seed, masked=(), zero_adv=()):
    dev = torch.device("cuda:0")
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    hidden = torch.randn((T, d), generator=gen, device=dev).to(torch.bfloat16)
    W = (torch.randn((V, d), generator=gen, device=dev) * (3.0 / d ** 0.5)).to(torch.bfloat16)
    tokens = torch.randint(0, V, (T,), generator=gen, device=dev, dtype=torch.int32)
    rng = np.random.default_rng(seed)
    cuts = np.sort(rng.choice(np.arange(1, T), size=min(M - 1, T - 1), replace=False)) if M > 1 else np.array([], int)
    cu = np.concatenate([[0], cuts, [T]]).astype(np.int64)
    M = cu.shape[0] - 1
    adv = rng.normal(size=M)
    adv = (np.sign(adv) * (0.2 + np.abs(adv))).astype(np.float32)  # away from 0: a tiny advantage could cancel the KL term
    adv[list(zero_adv)] = 0.0
    mask = np.ones(T, np.uint8)
    mask[list(masked)] = 0
    hb = hidden.view(torch.uint16).cpu().numpy()
    wb = W.view(torch.uint16).cpu().numpy()
    tok = tokens.cpu().numpy()
    base = lm_head.logp_from_hidden(hb, wb, tok)["logp"]
    old = (base + rng.normal(0, 0.15, T)).astype(np.float32)
    # the reference log-prob stays at least 0.02 away from the policy's: no row factor is a cancellation
    noise = rng.normal(0, 0.1, T)
    ref = (base + np.sign(noise) * (0.02 + np.abs(noise))).astype(np.float32)
    return dict(hidden=hidden, W=W, tokens=tokens, hb=hb, wb=wb, tok=tok, cu=cu, adv=adv, mask=mask, old=old, ref=ref,
                T=T, V=V, d=d, M=M)


def _oracle(c, beta=BETA):
    sw = oracle.seq_weights(c["mask"], c["cu"])
    out = lm_head.loss_grad_from_hidden(c["hb"], c["wb"], c["tok"], c["old"], c["ref"] if beta != 0 else None, c["adv"],
                                        sw, oracle.seq_of_rows(c["cu"]), c["mask"], EPS, beta)
    out["loss"] = oracle.grpo_loss(out["ell"], c["mask"], c["cu"])
    return out


def _run(c, beta=BETA, dW=None, grad_scale=1.0, hidden=None, W=None):
    dev = c["hidden"].device
    cu = torch.from_numpy(c["cu"]).to(dev)
    mask = torch.from_numpy(c["mask"]).to(dev)
    sw = torch.empty(c["M"], dtype=torch.float64, device=dev)
    binding.grpo_seq_weights(mask, cu, sw)
    loss_acc = torch.zeros(1, dtype=torch.float64, device=dev)
    if dW is None:
        dW = torch.zeros((c["V"], c["d"]), dtype=torch.float32, device=dev)
    status = binding.new_status()
    logp, dh = binding.grpo_loss_from_hidden(
        c["hidden"] if hidden is None else hidden, c["W"] if W is None else W, c["tokens"],
        torch.from_numpy(c["old"]).to(dev), torch.from_numpy(c["ref"]).to(dev) if beta != 0 else None,
        torch.from_numpy(c["adv"]).to(dev), sw, cu, 0, mask, EPS, beta, loss_acc, dW, grad_scale=grad_scale, status=status)
    torch.cuda.synchronize()
    return dict(logp=logp.cpu().numpy(), dhidden=dh.cpu().numpy().astype(np.float64),
                dW=dW.cpu().numpy().astype(np.float64), loss=float(loss_acc.item()), status=binding.read_status(status))


def _no_cancelling_factor(c, want):
    """|dg/dlogp| * 2e-6 / |g| stays far below the bf16 grain on every live row with a gradient."""
    sw = oracle.seq_weights(c["mask"], c["cu"])[oracle.seq_of_rows(c["cu"])] * (c["mask"] != 0)
    a = c["adv"][oracle.seq_of_rows(c["cu"])].astype(np.float64)
    rho = np.exp(want["logp"] - c["old"].astype(np.float64))
    ed = np.exp(c["ref"].astype(np.float64) - want["logp"])
    flows = rho * a <= np.clip(rho, 1 - float(np.float32(EPS)), 1 + float(np.float32(EPS))) * a   # not on the clipped side
    dg = 2e-6 * sw * (np.abs(a) * rho * flows + BETA * ed)
    g = np.abs(want["g"])
    rel = np.where(g > 0, dg / np.where(g > 0, g, 1.0), 0.0)
    return float(rel.max())


def _compare(case, got, want, c, scale=1.0):
    assert got["status"] == 0
    logp_err = float(np.abs(got["logp"] - want["logp"]).max())
    dh_ratio = float((np.abs(got["dhidden"] - scale * want["dhidden"]) / (scale * want["abs_dhidden"] + 1e-30)).max())
    dw_ratio = float((np.abs(got["dW"] - scale * want["dW"]) / (scale * want["abs_dW"] + 1e-30)).max())
    loss_rel = abs(got["loss"] - want["loss"]) / max(abs(want["loss"]), 1e-300)
    record(case, logp_abs=logp_err, dhidden_over_term_sum=dh_ratio, dW_over_term_sum=dw_ratio, loss_rel_literal=loss_rel,
           bound=GRAD_RTOL)
    assert logp_err <= LOGP_ATOL
    assert dh_ratio <= GRAD_RTOL, "dhidden off by %.3g of its term sum" % dh_ratio
    assert dw_ratio <= GRAD_RTOL, "dW off by %.3g of its term sum" % dw_ratio
    # where nothing is contracted the gradient is exactly zero: masked rows, vocabulary rows no live row reaches
    dead = want["abs_dhidden"].max(axis=1) == 0
    assert (got["dhidden"][dead] == 0).all()
    return loss_rel


@pytest.mark.parametrize("T,V,d,M", [(64, 1024, 128, 3),       # one block of rows, four tiles, one panel
                                     (128, 256, 64, 1),        # exactly one tile, one k-block
                                     (300, 1000, 72, 5),       # ragged rows, vocabulary and features
                                     (1, 8, 8, 1),             # the smallest legal shape
                                     (515, 5000, 320, 7),      # several row blocks; d beyond one 256-column tile
                                     (512, 32000, 1024, 16)])
def test_loss_and_gradients_against_the_oracle(T, V, d, M):
    masked = (0, T // 2) if T > 4 else ()
    c = _inputs(T, V, d, M, seed=T + V + d, masked=masked, zero_adv=(0,) if M > 2 else ())
    want = _oracle(c)
    assert _no_cancelling_factor(c, want) < 2.0 ** -11
    got = _run(c)
    loss_rel = _compare("grpo_loss_from_hidden T=%d V=%d d=%d" % (T, V, d), got, want, c)
    scale = np.abs(want["ell"]).mean()
    assert abs(got["loss"] - want["loss"]) <= LOSS_RTOL * max(abs(want["loss"]), scale / 1e3), loss_rel


def test_several_panels_accumulate_to_the_same_result():
    """With the panel limit at its minimum every 256-column tile is a panel of its own: dhidden is accumulated over
    all of them, dW is assembled from them."""
    c = _inputs(300, 1500, 96, 4, seed=21)
    want = _oracle(c)
    one = _run(c)
    before = binding.set_loss_from_hidden_panel_bytes(1)
    try:
        many = _run(c)
    finally:
        binding.set_loss_from_hidden_panel_bytes(before)
    _compare("grpo_loss_from_hidden six panels", many, want, c)
    assert one["logp"].tobytes() == many["logp"].tobytes() and one["loss"] == many["loss"]
    assert one["dW"].tobytes() == many["dW"].tobytes()              # a tile's dW does not depend on the panelling
    assert np.abs(one["dhidden"] - many["dhidden"]).max() <= 1e-5 * np.abs(want["abs_dhidden"]).max()


def test_dw_accumulates_and_grad_scale_scales():
    c = _inputs(200, 777 * 8, 64, 3, seed=22)
    want = _oracle(c)
    dev = c["hidden"].device
    dW = torch.zeros((c["V"], c["d"]), dtype=torch.float32, device=dev)
    first = _run(c, dW=dW)
    second = _run(c, dW=dW, grad_scale=0.5)                          # the same buffer again: 1 + 0.5 times the gradient
    np.testing.assert_allclose(second["dW"], 1.5 * first["dW"], rtol=0, atol=2e-6 * np.abs(first["dW"]).max())
    half = _run(c, grad_scale=0.5)
    _compare("grpo_loss_from_hidden grad_scale 0.5", half, want, c, scale=0.5)
    assert half["loss"] == first["loss"]


def test_without_kl_strided_inputs_and_token_range():
    c = _inputs(130, 520, 96, 2, seed=23)
    dev = c["hidden"].device
    wide_h = torch.zeros((c["T"], c["d"] + 8), dtype=torch.bfloat16, device=dev)
    wide_w = torch.zeros((c["V"], c["d"] + 16), dtype=torch.bfloat16, device=dev)
    wide_h[:, :c["d"]] = c["hidden"]
    wide_w[:, :c["d"]] = c["W"]
    want = _oracle(c, beta=0.0)
    got = _run(c, beta=0.0, hidden=wide_h[:, :c["d"]], W=wide_w[:, :c["d"]])
    _compare("grpo_loss_from_hidden beta=0, pitched rows", got, want, c)
    tok = c["tokens"].clone()
    tok[3] = c["V"]
    c2 = dict(c, tokens=tok)
    bad = _run(c2, beta=0.0)
    assert bad["status"] == binding.STATUS_TOKEN_RANGE
    tok0 = c["tok"].copy()
    tok0[3] = 0
    want0 = _oracle(dict(c, tok=tok0), beta=0.0)
    assert np.abs(bad["logp"] - want0["logp"]).max() <= LOGP_ATOL


def test_chunks_with_row0_add_up_to_the_whole_batch():
    """Two calls over rows [0, a) and [a, T) with the batch-wide cu_seqlens, weights and advantages (row0 = the chunk's
    first packed row; the cut falls inside a rollout and off the 128-row grid), loss_acc and dW carried from one
    call to the next: the same objective and gradients as one call over all rows."""
    c = _inputs(700, 3000, 128, 5, seed=26, masked=(3, 400))
    want = _oracle(c)
    whole = _run(c)
    dev = c["hidden"].device
    a = 333
    cu = torch.from_numpy(c["cu"]).to(dev)
    mask = torch.from_numpy(c["mask"]).to(dev)
    sw = binding.grpo_seq_weights(mask, cu)
    loss_acc = torch.zeros(1, dtype=torch.float64, device=dev)
    dW = torch.zeros((c["V"], c["d"]), dtype=torch.float32, device=dev)
    status = binding.new_status()
    old, ref, adv = (torch.from_numpy(c[k]).to(dev) for k in ("old", "ref", "adv"))
    logps, dhs = [], []
    for lo, hi in ((0, a), (a, c["T"])):
        lp, dh = binding.grpo_loss_from_hidden(c["hidden"][lo:hi], c["W"], c["tokens"][lo:hi].contiguous(),
                                               old[lo:hi].contiguous(), ref[lo:hi].contiguous(), adv, sw, cu, lo,
                                               mask[lo:hi].contiguous(), EPS, BETA, loss_acc, dW, status=status)
        logps.append(lp)
        dhs.append(dh)
    torch.cuda.synchronize()
    got = dict(logp=torch.cat(logps).cpu().numpy(), dhidden=torch.cat(dhs).cpu().numpy().astype(np.float64),
               dW=dW.cpu().numpy().astype(np.float64), loss=float(loss_acc.item()), status=binding.read_status(status))
    _compare("grpo_loss_from_hidden two chunks", got, want, c)
    assert got["logp"].tobytes() == whole["logp"].tobytes()
    assert got["dhidden"].tobytes() == whole["dhidden"].tobytes()      # a row's results do not depend on its tile mates
    assert abs(got["loss"] - whole["loss"]) <= 1e-12 * abs(whole["loss"]) + 1e-18
    assert np.abs(got["dW"] - whole["dW"]).max() <= 1e-5 * np.abs(want["abs_dW"]).max()


def test_repeated_calls_give_the_same_bits():
    c = _inputs(384, 5000, 192, 5, seed=24)
    a, b = _run(c), _run(c)
    for k in ("logp", "dhidden", "dW"):
        assert a[k].tobytes() == b[k].tobytes()
    assert a["loss"] == b["loss"]


@pytest.mark.skipif(not torch.cuda.is_available() or torch.cuda.get_device_properties(0).total_memory < 20e9,
                    reason="needs a few GB of device memory")
def test_qwen_vocabulary_at_d_2048():
    """The vocabulary and width of the 3B policy on 512 rows (the oracle's five fp64 products take about a minute),
    with the panel limit lowered so that the vocabulary is cut into several panels as it is at 16384 rows."""
    c = _inputs(512, 151936, 2048, 8, seed=25)
    want = _oracle(c)
    assert _no_cancelling_factor(c, want) < 2.0 ** -11
    before = binding.set_loss_from_hidden_panel_bytes(40 << 20)
    try:
        got = _run(c)
    finally:
        binding.set_loss_from_hidden_panel_bytes(before)
    _compare("grpo_loss_from_hidden T=512 V=151936 d=2048", got, want, c)
    assert abs(got["loss"] - want["loss"]) <= LOSS_RTOL * max(abs(want["loss"]), np.abs(want["ell"]).mean() / 1e3)


@pytest.mark.skipif(not torch.cuda.is_available() or torch.cuda.get_device_properties(0).total_memory < 20e9,
                    reason="needs a few GB of device memory")
def test_bench_shape_on_sampled_rows_and_by_identities():
    """T = 16384, V = 151936, d = 2048: the call bench.py times (ten panels).  The oracle takes sampled rows one block
    at a time: their log-probs and rows of dhidden (a row of dhidden depends on that row alone).  dW as a whole is tied
    to dhidden by two identities that hold at any size:
      <dW, W> = sum_{t,v} dlogits[t,v] logits[t,v] = <dhidden, hidden>     and     sum_v dW[v, :] = 0
    (every row of dlogits sums to zero), each up to the rounding of dlogits to bf16."""
    T, V, d, M = 16384, 151936, 2048, 64
    dev = torch.device("cuda:0")
    gen = torch.Generator(device=dev)
    gen.manual_seed(77)
    hidden = torch.randn((T, d), generator=gen, device=dev).to(torch.bfloat16)
    W = (torch.randn((V, d), generator=gen, device=dev) * (3.0 / d ** 0.5)).to(torch.bfloat16)
    tokens = torch.randint(0, V, (T,), generator=gen, device=dev, dtype=torch.int32)
    # old / ref: the framework's stock log-softmax of the same product plus noise - it only shapes the inputs
    base = torch.empty(T, device=dev)
    for lo in range(0, T, 2048):
        x = (hidden[lo:lo + 2048] @ W.t()).float()
        base[lo:lo + 2048] = torch.log_softmax(x, dim=-1).gather(1, tokens[lo:lo + 2048].long()[:, None])[:, 0]
        del x
    noise = 0.1 * torch.randn(T, generator=gen, device=dev)
    old = base + 0.15 * torch.randn(T, generator=gen, device=dev)
    ref = base + torch.sign(noise) * (0.02 + noise.abs())
    rng = np.random.default_rng(77)
    cu_h = np.concatenate([[0], np.sort(rng.choice(np.arange(1, T), size=M - 1, replace=False)), [T]]).astype(np.int64)
    adv_h = rng.normal(size=M)
    adv_h = (np.sign(adv_h) * (0.2 + np.abs(adv_h))).astype(np.float32)
    mask_h = np.ones(T, np.uint8)
    mask_h[rng.integers(0, T, 200)] = 0
    cu, adv, mask = torch.from_numpy(cu_h).to(dev), torch.from_numpy(adv_h).to(dev), torch.from_numpy(mask_h).to(dev)
    sw = binding.grpo_seq_weights(mask, cu)
    loss_acc = torch.zeros(1, dtype=torch.float64, device=dev)
    dW = torch.zeros((V, d), dtype=torch.float32, device=dev)
    status = binding.new_status()
    logp, dh = binding.grpo_loss_from_hidden(hidden, W, tokens, old, ref, adv, sw, cu, 0, mask, EPS, BETA, loss_acc, dW,
                                             status=status)
    torch.cuda.synchronize()
    assert binding.read_status(status) == 0

    rows = np.unique(np.concatenate([[0, 127, 128, T - 1], cu_h[1:5] - 1, cu_h[1:5], np.flatnonzero(mask_h == 0)[:4],
                                     rng.integers(0, T, 80)]))
    seq = oracle.seq_of_rows(cu_h)
    want = lm_head.loss_grad_from_hidden(hidden[rows].view(torch.uint16).cpu().numpy(), W.view(torch.uint16).cpu().numpy(),
                                         tokens.cpu().numpy()[rows], old.cpu().numpy()[rows], ref.cpu().numpy()[rows],
                                         adv_h, oracle.seq_weights(mask_h, cu_h), seq[rows], mask_h[rows], EPS, BETA,
                                         block_rows=32)
    logp_err = float(np.abs(logp.cpu().numpy()[rows] - want["logp"]).max())
    got = dh[rows].cpu().numpy().astype(np.float64)
    dh_ratio = float((np.abs(got - want["dhidden"]) / (want["abs_dhidden"] + 1e-30)).max())
    # the identities, in fp64 on the device
    dW64, W64 = dW.double(), W.double()
    lhs = float((dW64 * W64).sum())
    rhs = float((dh.double() * hidden.double()).sum())
    scale = float((dW64.abs() * W64.abs()).sum() + (dh.double().abs() * hidden.double().abs()).sum())
    col = dW64.sum(dim=0)
    col_ratio = float((col.abs() / dW64.abs().sum(dim=0)).max())
    record("grpo_loss_from_hidden T=%d V=%d d=%d (%d sampled rows)" % (T, V, d, len(rows)), logp_abs=logp_err,
           dhidden_over_term_sum=dh_ratio, inner_product_identity=abs(lhs - rhs) / scale, dW_column_sum_ratio=col_ratio,
           bound=GRAD_RTOL)
    assert logp_err <= LOGP_ATOL
    assert dh_ratio <= GRAD_RTOL
    assert (got[want["abs_dhidden"].max(axis=1) == 0] == 0).all()          # masked rows among the sample
    assert abs(lhs - rhs) <= GRAD_RTOL * scale
    assert col_ratio <= GRAD_RTOL
    assert torch.isfinite(dW).all() and torch.isfinite(dh).all()
