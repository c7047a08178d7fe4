"""Row sharding over ranks: the partition, and - with two gloo ranks on CPU - that the per-rank partial losses
(computed here by the oracle on each rank's rows) add up to the batch loss through the one all-reduce."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_row_ranges_are_contiguous_disjoint_and_balanced():
    from paper_2504_13818_b200.sharding import row_range
    for T in (0, 1, 5, 16384, 36853, 198448):
        for world in (1, 2, 3, 8):
            for multiple in (1, 7, 2048):
                edges = [row_range(T, world, r, multiple) for r in range(world)]
                assert edges[0][0] == 0 and edges[-1][1] == T
                for (lo, hi), (lo2, _) in zip(edges, edges[1:]):
                    assert lo <= hi == lo2
                    assert hi == T or hi % multiple == 0
                sizes = [hi - lo for lo, hi in edges]
                full = [s for (lo, hi), s in zip(edges, sizes) if hi < T]
                assert max(sizes) - min(full, default=max(sizes)) <= multiple
    with pytest.raises(ValueError):
        row_range(10, 2, 2)
    with pytest.raises(ValueError):
        row_range(10, 0, 0)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import oracle
    from paper_2504_13818_b200 import workloads as wl
    from paper_2504_13818_b200.sharding import all_reduce_loss, row_range
    from parity import build_batch, shrink
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    w = shrink(wl.WORKLOADS["c1_tiny"], G=3, n=8, m=4, V=96, seed=31)
    b = build_batch(w)                                  # every rank builds the same seeded batch
    T = b["tokens"].shape[0]
    mask = np.ones(T, np.uint8)
    sw = oracle.seq_weights(mask, b["cu"])
    lo, hi = row_range(T, world, rank, multiple=5)      # cuts rollouts in two
    rows = np.arange(lo, hi)
    part = oracle.grpo_rows(b["logits"][rows], b["tokens"][rows], b["old"][rows], b["ref"][rows], b["adv32"], sw,
                            b["seq_of_row"][rows], mask[rows], w.eps, w.beta, want_dlogits=False)
    acc = torch.tensor([float(np.sum(sw[b["seq_of_row"][rows]] * part["ell"]))], dtype=torch.float64)
    all_reduce_loss(acc)
    full = oracle.grpo_rows(b["logits"], b["tokens"], b["old"], b["ref"], b["adv32"], sw, b["seq_of_row"], mask,
                            w.eps, w.beta, want_dlogits=False)
    out[rank] = (lo, hi, T, float(acc.item()), float(oracle.grpo_loss(full["ell"], mask, b["cu"])))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_partial_losses_add_up_to_the_batch_loss():
    world, port = 2, _free_port()
    with mp.get_context("spawn").Manager() as manager:
        out = manager.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        got = dict(out)
    (lo0, hi0, T, acc0, want0), (lo1, hi1, _, acc1, want1) = got[0], got[1]
    assert lo0 == 0 and hi0 == lo1 and hi1 == T and 0 < hi0 < T
    assert acc0 == acc1                                  # every rank holds the same sum after the all-reduce
    assert want0 == want1
    assert abs(acc0 - want0) <= 1e-13 * max(1.0, abs(want0)) + 1e-18


def test_all_reduce_is_a_no_op_without_a_process_group():
    from paper_2504_13818_b200.sharding import all_reduce_loss
    acc = torch.tensor([1.25], dtype=torch.float64)
    assert all_reduce_loss(acc).item() == 1.25
    with pytest.raises(ValueError):
        all_reduce_loss(torch.zeros(1, dtype=torch.float32))
