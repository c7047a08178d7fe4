"""grpo_logp_from_hidden (CUDA, tensor cores) against the fp64 oracle: per-token log-prob abs <= 1e-3.

The kernel forms logits = hidden W^T tile by tile in fp32 accumulators and never stores them; the oracle is the
same product in fp64 followed by the two-pass log-softmax.  Shapes span one tile, several tiles with ragged tails
in every dimension (rows not a multiple of 128, vocabulary not a multiple of 256, features not a multiple of
64), several parts of the vocabulary per row, and the Qwen vocabulary at d = 2048 (sampled rows: the oracle
computes them one block at a time)."""
import numpy as np
import pytest
import torch

from oracle import lm_head
from paper_2504_13818_b200 import binding, workloads as wl
from parity import LOGP_ATOL, record

pytestmark = pytest.mark.gpu


def _inputs(T, V, d, seed, sigma=3.0):
    dev = torch.device("cuda:0")
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    hidden = torch.randn((T, d), generator=gen, device=dev).to(torch.bfloat16)
    W = (torch.randn((V, d), generator=gen, device=dev) * (sigma / d ** 0.5)).to(torch.bfloat16)
    tokens = torch.randint(0, V, (T,), generator=gen, device=dev, dtype=torch.int32)
    return hidden, W, tokens


def _run(hidden, W, tokens, want_lse=True):
    status = binding.new_status()
    logp, lse = binding.grpo_logp_from_hidden(hidden, W, tokens, want_lse=want_lse, status=status)
    torch.cuda.synchronize()
    assert binding.read_status(status) == 0
    return logp.cpu().numpy(), None if lse is None else lse.cpu().numpy()


def _oracle(hidden, W, tokens, rows=None):
    h = hidden.view(torch.uint16).cpu().numpy()
    t = tokens.cpu().numpy()
    if rows is not None:
        h, t = h[rows], t[rows]
    return lm_head.logp_from_hidden(h, W.view(torch.uint16).cpu().numpy(), t)


@pytest.mark.parametrize("T,V,d", [(64, 1024, 128),        # one block of rows, four tiles
                                   (128, 256, 64),         # exactly one tile, one k-block
                                   (300, 1000, 72),        # ragged rows, vocabulary and features
                                   (1, 8, 8),              # the smallest legal shape
                                   (512, 32000, 1024),
                                   (700, 50257, 256)])     # many parts per row block
def test_logp_against_the_oracle_on_all_rows(T, V, d):
    hidden, W, tokens = _inputs(T, V, d, seed=T + V + d)
    logp, lse = _run(hidden, W, tokens)
    want = _oracle(hidden, W, tokens)
    err = float(np.abs(logp - want["logp"]).max())
    record("grpo_logp_from_hidden T=%d V=%d d=%d" % (T, V, d), logp_abs=err,
           lse_abs=float(np.abs(lse - want["lse"]).max()))
    assert err <= LOGP_ATOL
    assert np.abs(lse - want["lse"]).max() <= LOGP_ATOL


def test_peaked_rows_and_targets_at_tile_edges():
    """Targets in the first and last column of a tile and of the vocabulary; rows dominated by one logit."""
    T, V, d = 256, 1000, 128
    hidden, W, tokens = _inputs(T, V, d, seed=5)
    tok = tokens.cpu().numpy()
    tok[:8] = [0, 255, 256, 511, 512, 767, 768, 999]
    tokens = torch.from_numpy(tok).cuda()
    # make row r's hidden state point along W[token]: a large target logit
    Wf = W.float()
    h = hidden.float()
    h[16:48] = Wf[tokens[16:48].long()] * 40.0
    hidden = h.to(torch.bfloat16)
    logp, _ = _run(hidden, W, tokens, want_lse=False)
    want = _oracle(hidden, W, tokens)
    assert (want["logp"][16:48] > -1e-2).any()
    assert np.abs(logp - want["logp"]).max() <= LOGP_ATOL


def test_strided_rows_and_token_range():
    T, V, d = 130, 520, 96
    hidden, W, tokens = _inputs(T, V, d, seed=9)
    wide_h = torch.zeros((T, d + 8), dtype=torch.bfloat16, device="cuda")
    wide_w = torch.zeros((V, d + 16), dtype=torch.bfloat16, device="cuda")
    wide_h[:, :d] = hidden
    wide_w[:, :d] = W
    tok = tokens.clone()
    tok[3] = V
    tok[7] = -5
    status = binding.new_status()
    logp, _ = binding.grpo_logp_from_hidden(wide_h[:, :d], wide_w[:, :d], tok, want_lse=False, status=status)
    torch.cuda.synchronize()
    assert binding.read_status(status) == binding.STATUS_TOKEN_RANGE
    want = _oracle(hidden, W, tok)
    assert want["bad_tokens"] == 2
    assert np.abs(logp.cpu().numpy() - want["logp"]).max() <= LOGP_ATOL


def test_repeated_calls_give_the_same_bits():
    hidden, W, tokens = _inputs(384, 5000, 192, seed=11)
    a = _run(hidden, W, tokens)
    b = _run(hidden, W, tokens)
    assert a[0].tobytes() == b[0].tobytes() and a[1].tobytes() == b[1].tobytes()


@pytest.mark.skipif(not torch.cuda.is_available() or torch.cuda.get_device_properties(0).total_memory < 20e9,
                    reason="needs a few GB of device memory")
def test_qwen_vocabulary_at_d_2048_on_sampled_rows():
    T, V, d = 4096, 151936, 2048
    hidden, W, tokens = _inputs(T, V, d, seed=1)
    logp, lse = _run(hidden, W, tokens)
    rng = np.random.default_rng(0)
    rows = np.unique(np.concatenate([[0, 127, 128, T - 1], rng.integers(0, T, 250)]))
    want = _oracle(hidden, W, tokens, rows=rows)
    err = float(np.abs(logp[rows] - want["logp"]).max())
    record("grpo_logp_from_hidden T=%d V=%d d=%d (%d sampled rows)" % (T, V, d, len(rows)), logp_abs=err,
           lse_abs=float(np.abs(lse[rows] - want["lse"]).max()))
    assert err <= LOGP_ATOL
    assert np.isfinite(logp).all() and (logp <= 0).all()
