"""grpo_loss_fwd_bwd / grpo_loss_chunk (CUDA) against the oracle.

Bar: per-token log-prob abs <= 1e-3, loss rel <= 1e-4 (see parity.assert_loss_close for sums that
cancel), dlogits within 2 bf16 ulps.  Rows whose
min(rho a, clip(rho) a) is within CLIP_MARGIN of switching branch are compared on logp only (the
branch is a floating-point decision; none is expected with these inputs and the count is asserted)."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2504_13818_b200 import binding, workloads as wl
from parity import (CLIP_MARGIN, DLOGITS_ULPS, LOGP_ATOL, LOSS_RTOL, assert_dlogits_close, assert_loss_close,
                    build_batch, dlogits_report, dlogits_ulp_error, gradient_slack, loss_errors, oracle_loss, record,
                    shrink)

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True, params=["default", "cluster path from V = 2048"])
def _both_loss_kernels(request):
    """Every test runs twice: with the library's own choice between its two loss kernels, and with the
    cluster-resident kernel forced on every vocabulary it can take (V >= 2048, V % 8 == 0, aligned rows)."""
    previous = binding.set_loss_cluster_min_vocab(2048) if request.param != "default" else None
    yield
    if previous is not None:
        binding.set_loss_cluster_min_vocab(previous)


def _t(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    return (t if dtype is None else t.view(dtype)).cuda()


def _gpu_loss(b, chunk_rows=0, in_place=False, ref=True, beta=None, mask=None):
    w = b["w"]
    logits = _t(b["logits"], torch.bfloat16)
    status = binding.new_status()
    dlogits = logits if in_place else None
    loss, logp, dl = binding.grpo_loss_fwd_bwd(
        logits, _t(b["tokens"]), _t(b["old"]), _t(b["ref"]) if ref else None, _t(b["adv32"]),
        _t(b["mask"] if mask is None else mask) if mask is not False else None,
        w.eps, w.beta if beta is None else beta, _t(b["cu"]), chunk_rows=chunk_rows, dlogits=dlogits, status=status)
    torch.cuda.synchronize()
    return (float(loss.item()), logp.cpu().numpy(), dl.view(torch.uint16).cpu().numpy(),
            binding.read_status(status))


def _check(b, got, want, expect_fragile=0, case=None, literal_loss=False):
    """Log-probs, loss and gradient against the oracle.  Gradient rows whose factor g_t is not a cancellation
    (all but a handful) are held to the literal 2-ulp bound; the count of the others is part of the record."""
    loss, logp, dl_bits, status = got
    assert status == 0
    logp_err = float(np.abs(logp - want["logp"]).max())
    assert logp_err <= LOGP_ATOL
    errs = loss_errors(loss, want, b)
    fragile = (want["margin"] < CLIP_MARGIN) & (want["margin"] > 0)
    assert int(fragile.sum()) == expect_fragile
    rep = dlogits_report(dl_bits, want["dlogits"], gradient_slack(b, want), skip_rows=fragile)
    case = case or os.environ.get("PYTEST_CURRENT_TEST", "?").split("::", 1)[-1].replace(" (call)", "")
    record(case, V=int(b["logits"].shape[1]), logp_abs=logp_err, **errs, **rep)
    assert_loss_close(loss, want, b)
    if literal_loss:
        assert errs["loss_rel_literal"] <= LOSS_RTOL, errs
    assert_dlogits_close(rep)
    return rep["literal_ulps"]


def test_config1_whole_path_values(request):
    """Config 1 in full.  Its loss is a nearly cancelling sum (rollout terms of +-0.06 add up to 1.7e-6): the
    chunk is small enough for the exact fp64 sums, so the literal relative bound holds as well."""
    b = build_batch(wl.WORKLOADS["c1_tiny"])
    _check(b, _gpu_loss(b), oracle_loss(b), case="c1_tiny [%s]" % request.node.callspec.id, literal_loss=True)


@pytest.mark.parametrize("V", [1, 2, 7, 8, 9, 1000, 1024, 8200, 40001])
def test_vocab_sizes_span_tiles_and_ragged_tails(V):
    w = shrink(wl.WORKLOADS["c1_tiny"], V=V, G=3, n=8, m=4, seed=V, spike=6.0, spike_frac=0.3)
    b = build_batch(w)
    _check(b, _gpu_loss(b), oracle_loss(b))


def test_many_rows_more_than_one_wave_and_in_place():
    w = shrink(wl.WORKLOADS["c1_tiny"], G=6, n=8, m=4, V=2048, len_lo=20, len_hi=40, seed=9)
    b = build_batch(w)
    want = oracle_loss(b)
    assert b["tokens"].shape[0] > 2 * 148
    a = _gpu_loss(b)
    _check(b, a, want)
    c = _gpu_loss(b, in_place=True)
    assert c[2].tobytes() == a[2].tobytes() and c[0] == a[0]


def test_chunked_equals_whole_bitwise_on_rows_and_within_tolerance_on_loss():
    w = shrink(wl.WORKLOADS["c1_tiny"], G=5, n=8, m=4, V=512, seed=21)
    b = build_batch(w)
    want = oracle_loss(b)
    whole = _gpu_loss(b)
    for rows in (1, 7, 64, 100000):
        part = _gpu_loss(b, chunk_rows=rows)
        assert part[1].tobytes() == whole[1].tobytes() and part[2].tobytes() == whole[2].tobytes()
        assert_loss_close(part[0], want, b)


def test_masked_rows_and_empty_rollouts():
    w = shrink(wl.WORKLOADS["c1_tiny"], G=3, n=8, m=4, V=264, seed=5)
    b = build_batch(w)
    rng = np.random.default_rng(0)
    b["mask"] = (rng.uniform(size=b["tokens"].shape[0]) < 0.7).astype(np.uint8)
    b["mask"][b["cu"][2]:b["cu"][3]] = 0                   # one rollout fully masked
    b["old"][b["mask"] == 0] = np.float32(-1e30)           # garbage under the mask must not leak into the loss
    want = oracle_loss(b)
    got = _gpu_loss(b)
    _check(b, got, want)
    assert (got[2][b["mask"] == 0] == 0).all()


def test_no_reference_policy_when_beta_is_zero():
    w = shrink(wl.WORKLOADS["c1_tiny"], G=3, n=8, m=4, V=520, beta=0.0, seed=6)
    b = build_batch(w)
    want = oracle_loss(b)
    _check(b, _gpu_loss(b, ref=False, mask=False), want)
    _check(b, _gpu_loss(b), want)


def test_clipped_rows_have_exactly_zero_gradient_rows():
    w = shrink(wl.WORKLOADS["c1_tiny"], G=3, n=8, m=4, V=520, beta=0.0, seed=8)
    b = build_batch(w)
    a_row = b["adv32"][b["seq_of_row"]]
    b["old"] = (b["old"] - np.sign(a_row) * 0.5).astype(np.float32)     # rho far on the penalised side
    want = oracle_loss(b)
    got = _gpu_loss(b)
    _check(b, got, want)
    assert (got[2][a_row != 0] & 0x7fff == 0).all()


def test_peaked_rows_keep_relative_accuracy_of_one_minus_p():
    """A policy that is nearly certain: the target's gradient g (1 - p) is tiny and must still be
    accurate to 2 bf16 ulps (the sum excludes the maximum, so Z - 1 is not lost to rounding)."""
    w = shrink(wl.WORKLOADS["c1_tiny"], G=2, n=8, m=4, V=4096, seed=12, logit_sigma=1.0)
    b = build_batch(w)
    x = wl.bf16_bits_to_f32(b["logits"])
    T = x.shape[0]
    boost = np.linspace(6.0, 24.0, T).astype(np.float32)    # 1 - p down to ~1e-7: fp64 still resolves it
    x[np.arange(T), b["tokens"]] += boost
    b["logits"] = wl.f32_to_bf16_bits(x)
    lt = wl.host_logp_tilde(b["logits"], b["tokens"])
    b["old"], b["ref"] = wl.make_old_ref(w, lt)
    want = oracle_loss(b)
    assert (want["logp"] > -1e-3).sum() > T // 3
    _check(b, _gpu_loss(b), want)


def test_token_out_of_range_sets_status_and_uses_token_zero():
    w = shrink(wl.WORKLOADS["c1_tiny"], G=2, n=8, m=4, V=128, seed=13)
    b = build_batch(w)
    b["tokens"] = b["tokens"].copy()
    b["tokens"][3] = w.V
    b["tokens"][5] = -1
    got = _gpu_loss(b)
    assert got[3] & binding.STATUS_TOKEN_RANGE
    want = oracle_loss(b)
    assert want["bad_tokens"] == 2
    assert np.abs(got[1] - want["logp"]).max() <= LOGP_ATOL
    assert dlogits_ulp_error(got[2], want["dlogits"], gradient_slack(b, want)).max() <= DLOGITS_ULPS


def test_strided_and_misaligned_rows_take_the_elementwise_path():
    w = shrink(wl.WORKLOADS["c1_tiny"], G=2, n=8, m=4, V=250, seed=14)
    b = build_batch(w)
    want = oracle_loss(b)
    T, V = b["logits"].shape
    wide = torch.zeros((T, V + 3), dtype=torch.bfloat16, device="cuda")
    wide[:, 1:V + 1] = _t(b["logits"], torch.bfloat16)
    view = wide[:, 1:V + 1]                                   # pitch V+3, base off by 2 bytes
    status = binding.new_status()
    loss, logp, dl = binding.grpo_loss_fwd_bwd(view, _t(b["tokens"]), _t(b["old"]), _t(b["ref"]), _t(b["adv32"]),
                                               None, w.eps, w.beta, _t(b["cu"]), status=status)
    torch.cuda.synchronize()
    _check(b, (float(loss.item()), logp.cpu().numpy(), dl.view(torch.uint16).cpu().numpy(), 0), want)


def test_whole_path_chained_on_its_own_outputs():
    """select -> compact -> loss on the GPU's own intermediate results equals the oracle's chain."""
    w = shrink(wl.WORKLOADS["c2_qwen_vocab"], V=3000, len_lo=8, len_hi=40)
    b = build_batch(w)
    want = oracle_loss(b)
    idx, adv, _ = binding.pods_select(_t(b["rewards"]), w.m)
    src_old = np.zeros(b["src_tokens"].shape, np.float32)
    src_ref = np.zeros(b["src_tokens"].shape, np.float32)
    for i in range(b["cu"].shape[0] - 1):                     # scatter the packed old/ref back to rollout storage
        g, j = divmod(i, w.m)
        row = g * w.n + int(b["sel"]["idx"][g, j])
        L = int(b["cu"][i + 1] - b["cu"][i])
        src_old[row, :L] = b["old"][b["cu"][i]:b["cu"][i + 1]]
        src_ref[row, :L] = b["ref"][b["cu"][i]:b["cu"][i + 1]]
    cu, toks, (old, ref) = binding.pods_compact(idx, w.n, _t(b["lengths"]), _t(b["src_tokens"]),
                                                [_t(src_old), _t(src_ref)])
    T = int(cu[-1].item())
    assert T == b["tokens"].shape[0]
    loss, logp, dl = binding.grpo_loss_fwd_bwd(_t(b["logits"], torch.bfloat16), toks[:T].contiguous(),
                                               old[:T].contiguous(), ref[:T].contiguous(), adv, None,
                                               w.eps, w.beta, cu, chunk_rows=500)
    torch.cuda.synchronize()
    _check(b, (float(loss.item()), logp.cpu().numpy(), dl.view(torch.uint16).cpu().numpy(), 0), want)


# ---- rows large enough for the cluster-resident path (V >= 16384, V % 8 == 0, aligned) -----------

@pytest.mark.parametrize("V,G,len_hi", [(16384, 6, 24),      # one CTA per row; more rows than resident CTAs
                                        (20008, 2, 12),      # two CTAs per row, ragged last segment (2501 vectors)
                                        (50000, 2, 10),
                                        (151936, 1, 8)])     # the Qwen vocabulary
def test_cluster_path_vocab_sizes(V, G, len_hi):
    w = shrink(wl.WORKLOADS["c2_qwen_vocab"], V=V, G=G, n=8, m=4, len_lo=4, len_hi=len_hi, seed=V % 1000)
    b = build_batch(w)
    want = oracle_loss(b)
    got = _gpu_loss(b)
    _check(b, got, want)
    again = _gpu_loss(b, in_place=True)
    assert again[2].tobytes() == got[2].tobytes() and again[1].tobytes() == got[1].tobytes()


def test_cluster_path_many_rows_per_cluster_masks_and_peaks():
    """V = 40960: three CTAs per row, at most 93 clusters resident, so a launch of ~1000 rows gives every
    cluster about ten rows and every ring stage is loaded, read and released several times."""
    w = shrink(wl.WORKLOADS["c2_qwen_vocab"], V=40960, G=16, n=8, m=4, len_lo=8, len_hi=24, seed=77)
    b = build_batch(w)
    T = b["tokens"].shape[0]
    assert T > 8 * 93
    rng = np.random.default_rng(5)
    b["mask"] = (rng.uniform(size=T) < 0.8).astype(np.uint8)
    x = wl.bf16_bits_to_f32(b["logits"])
    peak = rng.uniform(size=T) < 0.25                   # a quarter of the rows nearly certain of their token
    x[peak, b["tokens"][peak]] += rng.uniform(12.0, 22.0, size=int(peak.sum())).astype(np.float32)
    b["logits"] = wl.f32_to_bf16_bits(x)
    b["old"], b["ref"] = wl.make_old_ref(w, wl.host_logp_tilde(b["logits"], b["tokens"]))
    want = oracle_loss(b)
    got = _gpu_loss(b)                                  # one launch over all rows
    _check(b, got, want)
    assert (got[2][b["mask"] == 0] == 0).all()
    again = _gpu_loss(b, chunk_rows=300)                # several launches, about three rows per cluster each
    assert again[2].tobytes() == got[2].tobytes() and again[1].tobytes() == got[1].tobytes()
    _check(b, again, want)


def test_cluster_path_token_in_every_segment_and_duplicate_maxima():
    V = 16384
    w = shrink(wl.WORKLOADS["c2_qwen_vocab"], V=V, G=1, n=8, m=4, len_lo=8, len_hi=8, seed=3, spike_frac=0.0)
    b = build_batch(w)
    T = b["tokens"].shape[0]
    b["tokens"] = ((np.arange(T) * (V // 8) + 7 * np.arange(T)) % V).astype(np.int32)     # walks over the segments
    x = wl.bf16_bits_to_f32(b["logits"])
    x[0, [5, 9000, 16000]] = 14.0                       # the maximum three times, in different segments
    x[1, b["tokens"][1]] = 15.0
    x[1, (b["tokens"][1] + 1) % V] = 15.0               # the maximum twice in one vector, the token being one
    b["logits"] = wl.f32_to_bf16_bits(x)
    b["old"], b["ref"] = wl.make_old_ref(w, wl.host_logp_tilde(b["logits"], b["tokens"]))
    _check(b, _gpu_loss(b), oracle_loss(b))


def test_cluster_path_without_reference_policy_and_single_rows():
    w = shrink(wl.WORKLOADS["c2_qwen_vocab"], V=16384, G=1, n=8, m=4, len_lo=3, len_hi=9, seed=41, beta=0.0)
    b = build_batch(w)
    want = oracle_loss(b)
    _check(b, _gpu_loss(b, ref=False, mask=False), want)
    _check(b, _gpu_loss(b, chunk_rows=1), want)            # one row per launch: a single cluster, one row each


@pytest.mark.parametrize("V", [163840,      # nine CTAs per row: the first non-portable cluster size
                               180224,      # ten
                               196608,      # twelve
                               262144,      # sixteen
                               294912,      # sixteen, the longest segment with three stages and two CTAs per SM
                               294920,      # one vector more: the ring of two stages
                               393216,      # sixteen, twelve vectors per lane: the deepest register-held slice
                               393224])     # one vector more: back to the general row kernel
def test_long_rows_up_to_and_beyond_the_cluster_path_limit(V):
    w = shrink(wl.WORKLOADS["c2_qwen_vocab"], V=V, G=1, n=8, m=4, len_lo=2, len_hi=5, seed=V % 97)
    b = build_batch(w)
    _check(b, _gpu_loss(b), oracle_loss(b))


@pytest.mark.parametrize("V", [65536, 86016, 98304, 114688, 131072])       # four to eight CTAs per row
def test_every_portable_cluster_size(V):
    w = shrink(wl.WORKLOADS["c2_qwen_vocab"], V=V, G=1, n=8, m=4, len_lo=6, len_hi=12, seed=V % 101)
    b = build_batch(w)
    got = _gpu_loss(b)
    _check(b, got, oracle_loss(b))
    assert _gpu_loss(b, in_place=True)[2].tobytes() == got[2].tobytes()


def test_long_rows_on_the_two_stage_ring_with_several_rows_per_cluster():
    """V = 327680 over 16 CTAs: segments of 40 KB, too long for three stages with two CTAs per SM, so the ring
    has two stages; 14 such clusters are resident at most, so with > 80 rows every stage is reused several times."""
    w = shrink(wl.WORKLOADS["c2_qwen_vocab"], V=327680, G=2, n=8, m=4, len_lo=10, len_hi=18, seed=163)
    b = build_batch(w)
    assert b["tokens"].shape[0] > 80
    got = _gpu_loss(b)
    _check(b, got, oracle_loss(b))
    assert _gpu_loss(b, in_place=True)[2].tobytes() == got[2].tobytes()


def test_large_clusters_with_many_rows_masks_and_duplicate_maxima():
    """V = 176128 over ten CTAs (34.4 KB segments), several rows per cluster, some rows masked, maxima repeated across segments."""
    w = shrink(wl.WORKLOADS["c2_qwen_vocab"], V=176128, G=2, n=8, m=4, len_lo=10, len_hi=18, seed=176)
    b = build_batch(w)
    T = b["tokens"].shape[0]
    assert T > 80
    rng = np.random.default_rng(11)
    b["mask"] = (rng.uniform(size=T) < 0.8).astype(np.uint8)
    x = wl.bf16_bits_to_f32(b["logits"])
    x[0, [3, 60000, 120000, 176127]] = 15.0                # the maximum in four different CTAs' segments
    x[1, b["tokens"][1]] += 18.0                           # nearly certain of its token
    b["logits"] = wl.f32_to_bf16_bits(x)
    b["old"], b["ref"] = wl.make_old_ref(w, wl.host_logp_tilde(b["logits"], b["tokens"]))
    got = _gpu_loss(b)
    _check(b, got, oracle_loss(b))
    assert (got[2][b["mask"] == 0] == 0).all()


def test_a_wait_that_nothing_ends_gives_up_with_a_status_bit_and_the_context_stays_usable():
    """The loss kernel's barrier waits are bounded poll loops; the same loop on a barrier nobody completes
    (no fault, no hang: the kernel just stops waiting) must raise STATUS_TIMEOUT, and the next call must work."""
    status = binding.new_status()
    binding.selftest_bounded_wait(1000, status)
    torch.cuda.synchronize()
    assert binding.read_status(status) == binding.STATUS_TIMEOUT
    w = shrink(wl.WORKLOADS["c2_qwen_vocab"], V=16384, G=1, n=8, m=4, len_lo=3, len_hi=6, seed=5)
    b = build_batch(w)
    _check(b, _gpu_loss(b), oracle_loss(b))


def test_zero_length_rollouts_and_an_empty_batch():
    """Rollouts with no tokens (cu_seqlens repeats a value) get weight 0 and own no row; T = 0 is a no-op with loss 0."""
    for V in (520, 16384):
        w = shrink(wl.WORKLOADS["c1_tiny"], G=2, n=8, m=4, V=V, len_lo=3, len_hi=7, seed=23)
        b = build_batch(w)
        # make kept rollouts 2 and 5 empty: drop their rows everywhere
        cu = b["cu"].copy()
        keep = np.ones(b["tokens"].shape[0], bool)
        for i in (2, 5):
            keep[cu[i]:cu[i + 1]] = False
        lens = np.diff(cu)
        lens[[2, 5]] = 0
        b["cu"] = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
        for key in ("tokens", "old", "ref", "mask", "logits"):
            b[key] = np.ascontiguousarray(b[key][keep])
        b["seq_of_row"] = oracle.seq_of_rows(b["cu"])
        want = oracle_loss(b)
        _check(b, _gpu_loss(b), want)
    empty = torch.zeros((0, 16384), dtype=torch.bfloat16, device="cuda")
    z32 = torch.zeros(0, dtype=torch.float32, device="cuda")
    loss, logp, dl = binding.grpo_loss_fwd_bwd(empty, torch.zeros(0, dtype=torch.int32, device="cuda"), z32, z32,
                                               torch.ones(2, device="cuda"), None, 0.2, 0.04,
                                               torch.zeros(3, dtype=torch.int64, device="cuda"))
    torch.cuda.synchronize()
    assert float(loss.item()) == 0.0 and logp.numel() == 0 and dl.numel() == 0


@pytest.mark.parametrize("V", [4096, 32768])      # the general row kernel; the cluster path
def test_masked_vocabulary_ranges_of_minus_infinity(V):
    """Logits of -inf (ids a sampler has ruled out), scattered and as whole ranges longer than a warp's slice
    and than a CTA's segment of the cluster path: probability and gradient exactly 0 there, nothing turns NaN."""
    w = shrink(wl.WORKLOADS["c2_qwen_vocab"], V=V, G=1, n=8, m=4, len_lo=4, len_hi=8, seed=61)
    b = build_batch(w)
    x = wl.bf16_bits_to_f32(b["logits"])
    rng = np.random.default_rng(7)
    x[:, rng.uniform(size=V) < 0.1] = -np.inf            # scattered ids
    lo, hi = (V * 5) // 8, (V * 13) // 16
    x[:, lo:hi] = -np.inf                                # a range that covers whole warp slices and a whole segment
    x[0, :] = -np.inf                                    # row 0: everything but one id
    x[0, 77] = 1.5
    rows = np.arange(x.shape[0])
    tok = b["tokens"].copy()
    tok[0] = 77
    tok[1:] = np.where(np.isinf(x[rows[1:], tok[1:]]), 5, tok[1:])      # targets must be allowed ids
    x[:, 5] = np.where(np.isinf(x[:, 5]), 0.25, x[:, 5])
    b["tokens"] = tok.astype(np.int32)
    b["logits"] = wl.f32_to_bf16_bits(x)
    b["old"], b["ref"] = wl.make_old_ref(w, wl.host_logp_tilde(b["logits"], b["tokens"]))
    want = oracle_loss(b)
    assert np.isfinite(want["logp"]).all() and np.isfinite(want["dlogits"]).all()
    got = _gpu_loss(b)
    _check(b, got, want)
    dl = wl.bf16_bits_to_f32(got[2])
    assert np.isfinite(dl).all() and (dl[:, lo:hi] == 0).all()


@pytest.mark.parametrize("V", [2048, 16384])
def test_flat_rows_and_wide_logit_ranges(V):
    """Rows whose logits are all equal (every element is the maximum; p = 1/V exactly) and rows whose range is
    so wide that most probabilities underflow."""
    w = shrink(wl.WORKLOADS["c2_qwen_vocab"], V=V, G=1, n=8, m=4, len_lo=5, len_hi=9, seed=67)
    b = build_batch(w)
    x = wl.bf16_bits_to_f32(b["logits"])
    x[0, :] = 0.0
    x[1, :] = -7.25
    x[2, :] = 0.0
    x[2, ::2] = -0.0                                      # the two zeros are one value
    x[3:, :] *= 40.0                                      # spread of several hundred: e^(x - max) underflows
    b["logits"] = wl.f32_to_bf16_bits(x)
    b["old"], b["ref"] = wl.make_old_ref(w, wl.host_logp_tilde(b["logits"], b["tokens"]))
    want = oracle_loss(b)
    assert abs(want["logp"][0] + np.log(V)) < 1e-12 and abs(want["logp"][1] + np.log(V)) < 1e-12
    got = _gpu_loss(b)
    assert got[3] == 0
    finite = np.isfinite(want["logp"]) & np.isfinite(want["g"])
    assert finite[:3].all()
    assert finite.all()
    # log-probs of several hundred in magnitude: the fp32 output resolves them to ~3e-5, the bound stays 1e-3
    assert np.abs(got[1] - want["logp"]).max() <= LOGP_ATOL
    ulps = dlogits_ulp_error(got[2], want["dlogits"], gradient_slack(b, want))
    # where the target holds all the mass but 1e-12, fp64 itself no longer resolves 1 - p (the oracle's plain
    # log-sum-exp returns p = 1): the target's own entry is then left out, the rest of the row (zeros) is compared
    unresolved = want["logp"] > -1e-12
    assert 0 < unresolved.sum() < len(unresolved)
    ulps[np.nonzero(unresolved)[0], b["tokens"][unresolved]] = 0.0
    assert ulps.max() <= DLOGITS_ULPS
    got_target = wl.bf16_bits_to_f32(got[2])[np.nonzero(unresolved)[0], b["tokens"][unresolved]]
    assert (np.abs(got_target) < 1e-15).all()


def test_repeated_launches_are_bit_identical_on_every_kernel_in_and_out_of_place():
    """A few hundred launches per shape (row-tile kernel, row kernel, clusters of 1, 3, 9 and 16 CTAs, the last on
    the ring of two stages): any race in the pipelines or the exchange would show as a differing bit or a status
    bit sooner or later."""
    dev = torch.device("cuda")
    g = torch.Generator(device=dev)
    g.manual_seed(11)
    for V, T in [(1024, 700), (6000, 300), (12288, 900), (40960, 500), (151936, 150), (327680, 60)]:
        logits = (torch.randn((T, V), generator=g, device=dev) * 3).to(torch.bfloat16)
        tokens = torch.randint(0, V, (T,), generator=g, device=dev, dtype=torch.int32)
        cu = torch.linspace(0, T, 9, device=dev).long()
        lt = wl.library_logp(logits, tokens)
        old = lt + 0.05 * torch.randn(T, generator=g, device=dev)
        ref = lt + 0.05 * torch.randn(T, generator=g, device=dev)
        adv = torch.randn(8, generator=g, device=dev)
        sw = binding.grpo_seq_weights(None, cu)
        ws = torch.empty(binding.grpo_loss_chunk_workspace_bytes(T), dtype=torch.uint8, device=dev)

        def run(in_place):
            src = logits.clone() if in_place else logits
            dl = src if in_place else torch.empty_like(logits)
            acc = torch.zeros(1, dtype=torch.float64, device=dev)
            logp = torch.empty(T, device=dev)
            status = binding.new_status(dev)
            binding.grpo_loss_chunk(src, tokens, old, ref, adv, sw, cu, 0, None, 0.2, 0.04, acc, logp, dl, ws, status=status)
            return dl, logp, acc, status

        dl0, logp0, acc0, _ = run(False)
        for i in range(120):
            dl, logp, acc, status = run(bool(i & 1))
            assert torch.equal(dl.view(torch.int16), dl0.view(torch.int16)) and torch.equal(logp, logp0)
            assert float(acc.item()) == float(acc0.item()) and binding.read_status(status) == 0
