"""Seeded synthetic inputs for the PODS hot path.

This module only *draws inputs*: rewards, rollout lengths, token ids, logits and
the behaviour/reference log-probs that a training step would be handed.  It holds
none of the method's arithmetic (no selection, no advantages, no loss) and is the
one module that both the CUDA library's callers and the CPU checker's callers
may share.  The inputs stand in for the rollouts of the paper's GSM8K / MATH /
SciKnowEval runs (Table 1, Table 2): group shapes n -> m follow Table 2
(64 -> 16, 32 -> 8, 512 -> 128) and the reward structure follows Appendix A.1
(a 0/1 accuracy reward plus fractional format credit).
"""
from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    G: int                 # prompt groups
    n: int                 # rollouts per group
    m: int                 # kept rollouts per group
    rewards: str           # "bernoulli_uniform" | "bernoulli_beta" | "mixed" | "ternary"
    seed: int
    V: int = 0             # vocabulary (0: selection-only workload)
    len_kind: str = ""     # "uniform" | "lognormal"
    len_lo: int = 0
    len_hi: int = 0
    len_mu: float = 0.0
    len_sigma: float = 0.0
    logit_sigma: float = 0.0
    spike: float = 0.0     # added to the target logit ...
    spike_frac: float = 0.0  # ... at this fraction of positions
    old_sigma: float = 0.05
    ref_sigma: float = 0.05
    eps: float = 0.2
    beta: float = 0.04
    chunk_rows: int = 16384


WORKLOADS = {
    "c1_tiny": Workload("c1_tiny", G=4, n=16, m=4, rewards="bernoulli_uniform", seed=0, V=1024,
                        len_kind="uniform", len_lo=8, len_hi=64, logit_sigma=2.0),
    "c2_qwen_vocab": Workload("c2_qwen_vocab", G=8, n=64, m=16, rewards="bernoulli_beta", seed=1, V=151936,
                              len_kind="uniform", len_lo=64, len_hi=512, logit_sigma=3.0,
                              spike=8.0, spike_frac=0.3),
    # one prompt group of config 2 (about 4.6k kept tokens, 1.4 GB of logits): small enough for a
    # many-pass profiler capture, still far larger than L2
    "c2_profile": Workload("c2_profile", G=1, n=64, m=16, rewards="bernoulli_beta", seed=1, V=151936,
                           len_kind="uniform", len_lo=64, len_hi=512, logit_sigma=3.0,
                           spike=8.0, spike_frac=0.3),
    "c3_select_mixed": Workload("c3_select_mixed", G=65536, n=32, m=8, rewards="mixed", seed=2),
    "c4_select_ties": Workload("c4_select_ties", G=16384, n=512, m=128, rewards="ternary", seed=3),
    "c5_large_loss": Workload("c5_large_loss", G=16, n=64, m=16, rewards="bernoulli_beta", seed=4, V=151936,
                              len_kind="lognormal", len_mu=6.5, len_sigma=0.6, len_lo=32, len_hi=2048,
                              logit_sigma=3.0, ref_sigma=0.1),
}


def _rng(w: Workload, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([w.seed, stream]))


def make_rewards(w: Workload) -> np.ndarray:
    """fp32 rewards [G,n]."""
    rng = _rng(w, 0)
    G, n = w.G, w.n
    if w.rewards == "bernoulli_uniform":
        p = rng.uniform(0.0, 1.0, size=(G, 1))
        r = (rng.uniform(size=(G, n)) < p).astype(np.float32)
    elif w.rewards == "bernoulli_beta":
        p = rng.beta(0.5, 0.5, size=(G, 1))
        r = (rng.uniform(size=(G, n)) < p).astype(np.float32)
    elif w.rewards == "mixed":
        # correctness + 0.1 * format flag + small continuous noise
        p = rng.beta(1.0, 1.0, size=(G, 1))
        correct = (rng.uniform(size=(G, n)) < p).astype(np.float32)
        fmt = (rng.uniform(size=(G, n)) < 0.8).astype(np.float32)
        noise = rng.normal(0.0, 0.05, size=(G, n)).astype(np.float32)
        r = (correct + np.float32(0.1) * fmt + noise).astype(np.float32)
    elif w.rewards == "ternary":
        # values in {0, 0.5, 1} with per-group Dirichlet(1,1,1) probabilities; 5% of groups all equal
        probs = rng.dirichlet([1.0, 1.0, 1.0], size=G)
        u = rng.uniform(size=(G, n))
        c = np.cumsum(probs, axis=1)
        cat = (u > c[:, [0]]).astype(np.int64) + (u > c[:, [1]]).astype(np.int64)
        r = (0.5 * cat).astype(np.float32)
        flat = rng.uniform(size=G) < 0.05
        val = (0.5 * rng.integers(0, 3, size=G)).astype(np.float32)
        r[flat, :] = val[flat, None]
    else:
        raise ValueError(w.rewards)
    return np.ascontiguousarray(r, dtype=np.float32)


def make_rollouts(w: Workload):
    """Lengths [G*n] int32 and padded token ids [G*n, Lmax] int32 of ALL rollouts."""
    rng = _rng(w, 1)
    R = w.G * w.n
    if w.len_kind == "uniform":
        lengths = rng.integers(w.len_lo, w.len_hi + 1, size=R)
    elif w.len_kind == "lognormal":
        lengths = np.clip(np.rint(np.exp(rng.normal(w.len_mu, w.len_sigma, size=R))), w.len_lo, w.len_hi)
    else:
        raise ValueError(w.len_kind)
    lengths = lengths.astype(np.int32)
    Lmax = int(lengths.max())
    Lmax += (-Lmax) % 4
    tokens = rng.integers(0, w.V, size=(R, Lmax), dtype=np.int32)
    tokens[np.arange(Lmax)[None, :] >= lengths[:, None]] = -1     # padding is never a valid id
    return lengths, tokens


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even) and return the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    return ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def make_logits_host(w: Workload, tokens: np.ndarray) -> np.ndarray:
    """bf16 bit patterns [T,V] for packed target ids ``tokens`` [T] (small workloads)."""
    rng = _rng(w, 2)
    T = tokens.shape[0]
    x = (rng.standard_normal(size=(T, w.V)) * w.logit_sigma).astype(np.float32)
    if w.spike_frac > 0.0:
        rows = np.nonzero(rng.uniform(size=T) < w.spike_frac)[0]
        x[rows, tokens[rows]] += np.float32(w.spike)
    return f32_to_bf16_bits(x)


def make_logits_device(w: Workload, tokens_dev, row0: int = 0, rows_per_fill: int = 2048):
    """bf16 logits [T,V] drawn on the current CUDA device (large workloads).

    ``tokens_dev`` is the packed int32 target-id tensor on the device.  Rows are
    filled in blocks, each block from its own seeded generator state, so that a
    block (hence a chunk starting at ``row0``, a multiple of ``rows_per_fill``)
    is reproducible without drawing the rest.
    """
    import torch
    T = tokens_dev.shape[0]
    dev = tokens_dev.device
    out = torch.empty((T, w.V), dtype=torch.bfloat16, device=dev)
    gen = torch.Generator(device=dev)
    for lo in range(0, T, rows_per_fill):
        hi = min(T, lo + rows_per_fill)
        gen.manual_seed((w.seed << 32) + 7919 * ((row0 + lo) // rows_per_fill) + 17)
        x = torch.randn((hi - lo, w.V), generator=gen, dtype=torch.float32, device=dev) * w.logit_sigma
        if w.spike_frac > 0.0:
            pick = torch.rand((hi - lo,), generator=gen, device=dev) < w.spike_frac
            rows = torch.nonzero(pick).squeeze(1)
            x[rows, tokens_dev[lo:hi][rows].long()] += w.spike
        out[lo:hi] = x.to(torch.bfloat16)
    return out


def library_logp(logits, tokens):
    """A stand-in for the log-probs a frozen policy would report for ``tokens``.

    In training, old/ref log-probs come from separate forward passes of frozen
    models.  Here they are "current log-prob + noise" (see make_old_ref), and the
    current log-prob is taken from the framework's stock ``log_softmax`` on a
    torch tensor of logits [T,V] (any device), in row blocks.  It only shapes the
    inputs: both the library under test and its checker receive the result as data.
    """
    import torch
    T = logits.shape[0]
    out = torch.empty(T, dtype=torch.float32, device=logits.device)
    step = 1024
    for lo in range(0, T, step):
        hi = min(T, lo + step)
        ls = torch.log_softmax(logits[lo:hi].float(), dim=-1)
        out[lo:hi] = ls.gather(1, tokens[lo:hi].long().unsqueeze(1)).squeeze(1)
    return out


def make_old_ref(w: Workload, logp_tilde: np.ndarray):
    """old_logp, ref_logp [T] fp32 = logp_tilde + N(0, sigma^2)."""
    rng = _rng(w, 3)
    T = logp_tilde.shape[0]
    lt = np.asarray(logp_tilde, dtype=np.float64)
    old = (lt + rng.normal(0.0, w.old_sigma, size=T)).astype(np.float32)
    ref = (lt + rng.normal(0.0, w.ref_sigma, size=T)).astype(np.float32)
    return old, ref


def host_logp_tilde(logits_bits: np.ndarray, tokens: np.ndarray) -> np.ndarray:
    """library_logp for host bf16 bit patterns (small workloads)."""
    import torch
    lg = torch.from_numpy(bf16_bits_to_f32(logits_bits))
    return library_logp(lg, torch.from_numpy(np.ascontiguousarray(tokens, dtype=np.int32))).numpy()
