"""Gradient-accumulation batching of GRPO-PODS (Appendix A.2, the note under Table 2).

In the paper's full-parameter settings a prompt's n rollouts do not fit one update batch: they are produced and
down-sampled per ROLLOUT BATCH (128 -> 32), and `steps` accumulation steps (4) make up the effective 512 -> 128.
Down-sampling is applied inside each rollout batch, not across the n rollouts of the prompt, so the kept set is
in general NOT the one a single n -> m selection would keep; everything after the selection is one batch:

  * selection: the rewards [G, n] are regrouped step-major into [steps * G, n / steps] and handed to ONE
    `pods_select` call with m / steps kept per rollout batch (advantages are normalised within each rollout
    batch's kept subset, as Section 3.2 does per group);
  * objective: L_PODS over all M = G m kept rollouts (Section 3.2, mean over rollouts of per-rollout token means).
    Accumulation step a holds the kept rollouts [a G m/steps, (a+1) G m/steps), a contiguous range of rows of the
    packed batch, so it is `grpo_loss_chunk` over that range with the batch-wide cu_seqlens, weights 1/(M |o_i|)
    and advantages (`row0` = the range's first row): the gradient rows of a step already carry the batch-wide
    factor, and the steps' loss terms add up in the one fp64 accumulator.  No 1/steps factor is needed anywhere.

Host logic only (index arithmetic and calls of the binding); the kernels are the single-batch ones."""
from dataclasses import dataclass

import torch

from . import binding


@dataclass(frozen=True)
class AccumulationPlan:
    G: int          # prompts
    n: int          # rollouts per prompt over all accumulation steps (effective n)
    m: int          # kept per prompt over all accumulation steps (effective m)
    steps: int      # accumulation steps = rollout batches per prompt

    @property
    def n_step(self):
        return self.n // self.steps

    @property
    def m_step(self):
        return self.m // self.steps

    @property
    def groups(self):
        """Groups the selection sees: one per (step, prompt), step-major."""
        return self.steps * self.G


def make_plan(G, n, m, steps):
    if G < 1 or steps < 1 or n < 1 or m < 1 or n % steps or m % steps or m > n:
        raise ValueError("make_plan(G=%r, n=%r, m=%r, steps=%r): n and m must be multiples of steps, 1 <= m <= n"
                         % (G, n, m, steps))
    return AccumulationPlan(G, n, m, steps)


def step_major(x, plan):
    """[G, n, ...] -> [steps * G, n / steps, ...]: rollout batch a of prompt g becomes group a * G + g.

    Works on torch tensors and numpy arrays alike (a reshape, a transpose and a copy)."""
    shape = tuple(x.shape)
    if shape[0] != plan.G or shape[1] != plan.n:
        raise ValueError("expected [G=%d, n=%d, ...], got %s" % (plan.G, plan.n, shape))
    y = x.reshape((plan.G, plan.steps, plan.n_step) + shape[2:])
    y = y.transpose(0, 1) if isinstance(y, torch.Tensor) else y.swapaxes(0, 1)
    y = y.reshape((plan.groups, plan.n_step) + shape[2:])
    return y.contiguous() if isinstance(y, torch.Tensor) else y.copy()


def original_rollout(plan, group, j):
    """(prompt, rollout index within the prompt's n) of rollout j of step-major group `group`."""
    a, g = divmod(group, plan.G)
    return g, a * plan.n_step + j


def select(rewards, plan, rule=binding.RULE_MAXVAR, seed=0, flags=0, status=None):
    """Per-rollout-batch down-sampling of rewards [G, n]: returns (idx, adv, k) of `pods_select` on the step-major
    groups, i.e. idx [steps * G, m / steps] holds indices WITHIN the rollout batch (see original_rollout)."""
    return binding.pods_select(step_major(rewards, plan), plan.m_step, rule=rule, seed=seed, flags=flags, status=status)


def step_ranges(cu_seqlens, plan):
    """[(first kept rollout, one past the last, first row, one past the last row)] per accumulation step, from the
    batch-wide cu_seqlens [M + 1] of the step-major packed batch (a host list or a tensor; read on the host)."""
    cu = cu_seqlens.tolist() if hasattr(cu_seqlens, "tolist") else list(cu_seqlens)
    per = plan.G * plan.m_step
    if len(cu) != plan.steps * per + 1:
        raise ValueError("cu_seqlens must hold M + 1 = %d entries, got %d" % (plan.steps * per + 1, len(cu)))
    return [(a * per, (a + 1) * per, int(cu[a * per]), int(cu[(a + 1) * per])) for a in range(plan.steps)]


def loss_step(step, ranges, logits_step, tokens, old_logp, ref_logp, adv, seq_weight, cu_seqlens, mask, eps, beta,
              loss_acc, logp, dlogits_step, workspace, chunk_rows=16384, status=None):
    """Accumulation step `step`: `grpo_loss_chunk` over the step's rows in chunks of chunk_rows.

    ``logits_step`` / ``dlogits_step`` hold the step's rows only (the forward pass of that step produced them);
    tokens, old_logp, ref_logp, mask and logp are the batch-wide packed arrays [T]; adv [M], seq_weight [M] and
    cu_seqlens [M+1] are batch-wide.  ``loss_acc`` is zeroed by the caller before step 0 and finalised after the
    last step with `grpo_loss_finalize`."""
    _, _, row_lo, row_hi = ranges[step]
    if logits_step.shape[0] != row_hi - row_lo:
        raise ValueError("step %d has %d rows, logits_step has %d" % (step, row_hi - row_lo, logits_step.shape[0]))
    for lo in range(row_lo, row_hi, chunk_rows):
        hi = min(row_hi, lo + chunk_rows)
        binding.grpo_loss_chunk(logits_step[lo - row_lo:hi - row_lo], tokens[lo:hi], old_logp[lo:hi],
                                None if ref_logp is None else ref_logp[lo:hi], adv, seq_weight, cu_seqlens, lo,
                                None if mask is None else mask[lo:hi], eps, beta, loss_acc, logp[lo:hi],
                                dlogits_step[lo - row_lo:hi - row_lo], workspace, status=status)
