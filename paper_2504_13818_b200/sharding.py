"""Row sharding of one GRPO-PODS batch over several GPUs (one process per GPU).

The rows of the packed logits [T, V] are independent once the batch-wide per-rollout weights 1/(M |o_i|) and
the advantages are known (L_PODS, Section 3.2: a sum over rollouts of sums over tokens).  So each rank runs
`grpo_loss_chunk` over its own contiguous range of rows with the batch-wide cu_seqlens, weights and advantages
(`row0` is the range's first row); gradient rows need no exchange at all, and the loss is the sum of the ranks'
fp64 accumulators: one all-reduce of one double, after which every rank calls `grpo_loss_finalize`.  A range
may cut a rollout in two; the rollout's weight is batch-wide, so nothing changes.

Host logic only: the partition and the one collective.  The kernels are the single-GPU ones."""
import torch
import torch.distributed as dist


def row_range(T, world_size, rank, multiple=1):
    """Rows [lo, hi) of rank `rank` out of `world_size`: contiguous, disjoint, covering [0, T), sizes differing
    by at most `multiple`; every boundary but T is a multiple of `multiple` (e.g. the chunk size, so that no
    rank's last chunk is ragged but the last rank's).  Ranks beyond the work get an empty range."""
    if T < 0 or world_size < 1 or not 0 <= rank < world_size or multiple < 1:
        raise ValueError("row_range(T=%r, world_size=%r, rank=%r, multiple=%r)" % (T, world_size, rank, multiple))
    units = (T + multiple - 1) // multiple
    base, extra = divmod(units, world_size)
    lo_u = rank * base + min(rank, extra)
    hi_u = lo_u + base + (1 if rank < extra else 0)
    return min(T, lo_u * multiple), min(T, hi_u * multiple)


def all_reduce_loss(loss_acc, group=None):
    """Sums the ranks' fp64 loss accumulators in place (the path's only exchange).  `loss_acc` is the one-element
    float64 tensor `grpo_loss_chunk` accumulates into; call `grpo_loss_finalize` afterwards."""
    if loss_acc.dtype != torch.float64 or loss_acc.numel() != 1:
        raise ValueError("loss_acc must be one float64")
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(loss_acc, op=dist.ReduceOp.SUM, group=group)
    return loss_acc
