"""pods_compact and grpo_seq_weights (CUDA) against the oracle: integer work, bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_13818_b200 import binding, workloads as wl
from parity import shrink

pytestmark = pytest.mark.gpu


def _case(w):
    rewards = wl.make_rewards(w)
    lengths, src = wl.make_rollouts(w)
    idx = oracle.select(rewards, w.m)["idx"]
    stream = np.random.default_rng(w.seed).normal(size=src.shape).astype(np.float32)
    return idx, lengths, src, stream


@pytest.mark.parametrize("name,kw", [("c1_tiny", {}), ("c2_qwen_vocab", {}), ("c5_large_loss", {}),
                                     ("c1_tiny", {"G": 300, "n": 20, "m": 7})])
def test_compact_matches_oracle(name, kw):
    w = shrink(wl.WORKLOADS[name], **kw)
    idx, lengths, src, stream = _case(w)
    cu_o, tok_o, streams_o, _ = oracle.compact(idx, w.n, lengths, src, [stream])
    status = binding.new_status()
    cu, tok, dst = binding.pods_compact(torch.from_numpy(idx).cuda(), w.n, torch.from_numpy(lengths).cuda(),
                                        torch.from_numpy(src).cuda(), [torch.from_numpy(stream).cuda()],
                                        status=status)
    torch.cuda.synchronize()
    T = int(cu_o[-1])
    np.testing.assert_array_equal(cu.cpu().numpy(), cu_o)
    np.testing.assert_array_equal(tok.cpu().numpy()[:T], tok_o)
    np.testing.assert_array_equal(dst[0].cpu().numpy()[:T], streams_o[0])
    assert binding.read_status(status) == 0


def test_capacity_and_bad_lengths_raise_status_without_overrun():
    w = wl.WORKLOADS["c1_tiny"]
    idx, lengths, src, _ = _case(w)
    cu_o, tok_o, _, _ = oracle.compact(idx, w.n, lengths, src)
    T = int(cu_o[-1])
    cap = T - 5
    status = binding.new_status()
    guard = torch.full((T + 64,), -7, dtype=torch.int32, device="cuda")
    cu = torch.empty(idx.size + 1, dtype=torch.int64, device="cuda")
    binding.pods_compact(torch.from_numpy(idx).cuda(), w.n, torch.from_numpy(lengths).cuda(),
                         torch.from_numpy(src).cuda(), T_cap=cap, status=status, out=(cu, guard, []))
    torch.cuda.synchronize()
    got = guard.cpu().numpy()
    assert binding.read_status(status) & binding.STATUS_CAPACITY
    np.testing.assert_array_equal(got[:cap], tok_o[:cap])
    assert (got[cap:] == -7).all()
    bad = lengths.copy()
    bad[int(idx[0, 0])] = -3
    status = binding.new_status()
    cu2, _, _ = binding.pods_compact(torch.from_numpy(idx).cuda(), w.n, torch.from_numpy(bad).cuda(),
                                     torch.from_numpy(src).cuda(), status=status)
    assert binding.read_status(status) & binding.STATUS_NEG_LENGTH
    assert int(cu2[1]) == 0


def test_kept_indices_outside_the_group_raise_status_and_read_rollout_zero():
    """idx is data: entries outside [0, n) (not pods_select's output) must not become addresses."""
    w = wl.WORKLOADS["c1_tiny"]
    idx, lengths, src, _ = _case(w)
    bad = idx.copy()
    bad[1, 2] = w.n                    # one past the group
    bad[3, 0] = -1000000
    status = binding.new_status()
    cu, toks, _ = binding.pods_compact(torch.from_numpy(bad).cuda(), w.n, torch.from_numpy(lengths).cuda(),
                                       torch.from_numpy(src).cuda(), status=status)
    torch.cuda.synchronize()
    assert binding.read_status(status) == binding.STATUS_INDEX_RANGE
    fixed = bad.copy()
    fixed[1, 2] = 0
    fixed[3, 0] = 0
    cu_o, tok_o, _, _ = oracle.compact(fixed, w.n, lengths, src)
    np.testing.assert_array_equal(cu.cpu().numpy(), cu_o)
    np.testing.assert_array_equal(toks[: int(cu_o[-1])].cpu().numpy(), tok_o)


def test_seq_weights_with_and_without_mask():
    rng = np.random.default_rng(3)
    lens = rng.integers(0, 70, 50)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    mask = (rng.uniform(size=int(cu[-1])) < 0.6).astype(np.uint8)
    mask[cu[7]:cu[8]] = 0
    got = binding.grpo_seq_weights(torch.from_numpy(mask).cuda(), torch.from_numpy(cu).cuda()).cpu().numpy()
    np.testing.assert_array_equal(got, oracle.seq_weights(mask, cu))
    got = binding.grpo_seq_weights(None, torch.from_numpy(cu).cuda()).cpu().numpy()
    np.testing.assert_array_equal(got, oracle.seq_weights(np.ones_like(mask), cu))
