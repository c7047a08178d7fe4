"""pods_select (CUDA) against the oracle: indices and k bit-exact, advantages rel <= 1e-6."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_13818_b200 import binding, workloads as wl
from parity import assert_adv_close, record, shrink

pytestmark = pytest.mark.gpu


def _run(rewards, m, rule=0, seed=0, flags=0):
    status = binding.new_status()
    r = torch.from_numpy(np.ascontiguousarray(rewards, np.float32)).cuda()
    idx, adv, k = binding.pods_select(r, m, rule=rule, seed=seed, flags=flags, status=status)
    torch.cuda.synchronize()
    return idx.cpu().numpy(), adv.cpu().numpy(), k.cpu().numpy(), binding.read_status(status)


def _compare(rewards, m, rule=0, seed=0, flags=0, expect_status=0):
    idx, adv, k, status = _run(rewards, m, rule, seed, flags)
    want = oracle.select(rewards, m, rule=rule, seed=seed, flags=flags)
    # a split decided by less than 2^-40 of the score is beyond fp64 evaluation: list, do not hide
    fragile = want["gap"] < 2.0 ** -40
    assert fragile.sum() == 0, "groups with near-tied splits: %s" % np.nonzero(fragile)[0][:10]
    np.testing.assert_array_equal(idx, want["idx"])
    np.testing.assert_array_equal(k, want["k"])
    assert_adv_close(adv, want["adv"])
    assert status == expect_status
    return idx, adv, k


def _reward_kinds(rng, G, n):
    yield "normal", rng.normal(0, 1, (G, n)).astype(np.float32)
    yield "binary", (rng.uniform(size=(G, n)) < rng.uniform(size=(G, 1))).astype(np.float32)
    yield "ternary", rng.choice([0.0, 0.5, 1.0], (G, n)).astype(np.float32)
    yield "mixed", (rng.integers(0, 2, (G, n)) + 0.1 * rng.integers(0, 2, (G, n))
                    + rng.normal(0, 0.05, (G, n))).astype(np.float32)
    yield "negatives", rng.choice([-2.0, -0.25, 0.0, 0.25, 3.0], (G, n)).astype(np.float32)
    # values that are not dyadic: sums of their squares are not exact in fp64, yet splits that keep the same
    # multiset of rewards must still tie (an accuracy reward of 1 plus a format credit of 0.1, as in Appendix A.1)
    yield "decimal", rng.choice([0.1, 0.3, 0.7], (G, n)).astype(np.float32)
    yield "accuracy+format", (rng.integers(0, 2, (G, n)) + 0.1 * rng.integers(0, 2, (G, n))).astype(np.float32)


@pytest.mark.parametrize("n", [1, 2, 3, 7, 8, 9, 16, 17, 31, 32, 33, 48, 64, 100, 128, 200, 256, 257, 512, 1000, 1024])
def test_every_kernel_shape_and_ragged_n(n):
    rng = np.random.default_rng(n)
    G = 67                                           # not a multiple of the groups per CTA
    ms = sorted({min(n, 1), min(n, 2), max(1, n // 4), max(1, n // 2), max(1, n - 1), n})
    for m in ms:
        for _, r in _reward_kinds(rng, G, n):
            _compare(r, m)


def test_ties_that_hold_for_any_values_and_ties_by_coincidence():
    """Splits that keep the same multiset, and the mirror pair of a two-valued kept subset, tie whatever the values
    are: the default path must get them right for rewards that fp64 sums do not represent exactly.  Ties that hold
    only because the reward values happen to be commensurate (0.1, 0.2, 0.4 in fp32 are exactly 1 : 2 : 4) are
    settled exactly under FLAG_EXACT_TIES."""
    rng = np.random.default_rng(11)
    for n, m in [(7, 3), (16, 4), (32, 8), (64, 16), (100, 30), (512, 128), (1000, 333)]:
        for values in ([0.1, 0.7], [0.3, 1.1], [0.1, 0.3, 0.7], [0.0, 0.1, 1.0, 1.1]):
            r = rng.choice(values, (53, n)).astype(np.float32)
            _compare(r, m)
            _compare(r, m, flags=binding.FLAG_EXACT_TIES)
        base = np.float32(0.1)
        r = (rng.choice([1.0, 2.0, 4.0], (53, n)).astype(np.float32) * base).astype(np.float32)
        _compare(r, m, flags=binding.FLAG_EXACT_TIES)
    # the exact path agrees with the default one where the default is exact by itself
    for kind, r in _reward_kinds(rng, 67, 48):
        a = _run(r, 12)
        b = _run(r, 12, flags=binding.FLAG_EXACT_TIES)
        assert a[0].tobytes() == b[0].tobytes() and a[2].tobytes() == b[2].tobytes(), kind


def test_workload_rewards_at_full_size():
    for name in ("c1_tiny", "c2_qwen_vocab", "c3_select_mixed", "c4_select_ties", "c5_large_loss"):
        w = wl.WORKLOADS[name]
        r = wl.make_rewards(w)
        idx, adv, k = _compare(r, w.m)                   # indices and k bit-exact, advantages within tolerance
        want = oracle.select(r, w.m)["adv"]
        nz = want != 0
        rel = float((np.abs(adv.astype(np.float64) - want)[nz] / np.abs(want[nz])).max()) if nz.any() else 0.0
        record("%s rewards at full size (G=%d, n=%d, m=%d)" % (name, w.G, w.n, w.m), idx_exact=1, adv_rel=rel)


def test_degenerate_and_special_values():
    r = np.full((5, 40), 0.75, np.float32)
    idx, adv, k = _compare(r, 10)
    assert (k == 0).all() and (adv == 0).all() and (idx == np.arange(10)).all()
    r = np.array([[0.0, -0.0, 1.0, 0.0, 1.0, -0.0]], np.float32)
    idx, _, k = _compare(r, 2)
    assert list(idx[0]) == [0, 4] and k[0] == 1
    rng = np.random.default_rng(1)
    _compare(rng.normal(size=(9, 33)).astype(np.float32), 33)       # m == n: plain GRPO
    _compare(rng.normal(size=(9, 33)).astype(np.float32), 1)
    _compare((rng.normal(size=(64, 24)) * 1e-30).astype(np.float32), 6)    # tiny magnitudes
    _compare((rng.normal(size=(64, 24)) * 1e30).astype(np.float32), 6)     # huge magnitudes
    _compare((1e6 + rng.integers(0, 3, size=(64, 24))).astype(np.float32), 6)   # large offset, small spread
    assert binding.pods_select(torch.zeros((0, 8), device="cuda"), 2)[0].shape == (0, 2)


def test_nonfinite_rewards_raise_the_status_bit_and_stay_in_range():
    r = np.random.default_rng(2).normal(size=(6, 20)).astype(np.float32)
    r[1, 3] = np.nan
    r[4, 0] = np.inf
    idx, adv, k, status = _run(r, 5)
    assert status & binding.STATUS_NONFINITE_REWARD
    assert idx.min() >= 0 and idx.max() < 20 and (np.diff(idx, axis=1) > 0).all()
    clean = [0, 2, 3, 5]
    want = oracle.select(r[clean], 5)
    np.testing.assert_array_equal(idx[clean], want["idx"])
    # +inf sorts last but NaN above it: the group with +inf keeps the oracle's indices too
    np.testing.assert_array_equal(idx[[1, 4]], oracle.select(r[[1, 4]], 5)["idx"])


@pytest.mark.parametrize("rule", [binding.RULE_MAXREWARD, binding.RULE_RANDOM, binding.RULE_PERCENTILE])
def test_baseline_rules(rule):
    rng = np.random.default_rng(rule)
    for n, m in [(8, 3), (16, 4), (32, 8), (64, 16), (100, 7), (512, 128), (1024, 1024)]:
        r = rng.normal(size=(37, n)).astype(np.float32)
        _compare(r, m, rule=rule, seed=0xC0FFEE12345 + n)


def test_advantage_flags():
    rng = np.random.default_rng(5)
    for n, m in [(16, 4), (64, 16), (200, 50)]:
        r = rng.normal(size=(41, n)).astype(np.float32)
        for flags in (binding.FLAG_ADV_BEFORE, binding.FLAG_STD_SAMPLE, binding.FLAG_ADV_BEFORE | binding.FLAG_STD_SAMPLE):
            _compare(r, m, flags=flags)
    _compare(rng.normal(size=(4, 9)).astype(np.float32), 1, flags=binding.FLAG_STD_SAMPLE)   # count-1 = 0 -> adv 0


def test_run_to_run_bit_equality():
    w = shrink(wl.WORKLOADS["c4_select_ties"], G=2048)
    r = wl.make_rewards(w)
    a = _run(r, w.m)
    b = _run(r, w.m)
    for x, y in zip(a[:3], b[:3]):
        assert x.tobytes() == y.tobytes()
