"""The loss path at the full sizes of configs 2 and 5, in the launch configuration bench.py times
(grpo_loss_chunk over 16384-row chunks at V = 151936), against the oracle:

  * config 2 (36,853 kept tokens, 11.2 GB of logits): every row's log-prob, the loss and every element of
    dlogits against the oracle over ALL rows (the oracle runs in 1024-row blocks of fp64 gradient rows);
  * config 5 (about 2 x 10^5 kept tokens, 61 GB of logits, processed chunk by chunk in place): the first,
    a middle and the last chunk (they hold rollouts that straddle chunk edges): per chunk, every row's
    log-prob and the chunk's contribution to the loss against the oracle over the whole chunk, dlogits
    on sampled rows; the other chunks run too (the accumulated loss is finite and the status word clean).

Rows whose min(rho a, clip(rho) a) is within CLIP_MARGIN of switching branch are compared on logp only
(none is expected; the count is asserted)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_13818_b200 import binding, workloads as wl
from parity import (CLIP_MARGIN, DLOGITS_ULPS, LOGP_ATOL, LOSS_COND, LOSS_RTOL, assert_dlogits_close, dlogits_report,
                    gradient_slack, record)

pytestmark = pytest.mark.gpu

needs_big_gpu = pytest.mark.skipif(
    not torch.cuda.is_available() or torch.cuda.get_device_properties(0).total_memory < 60e9,
    reason="needs tens of GB of device memory")


def _selection_and_layout(w):
    rewards = wl.make_rewards(w)
    lengths, src_tokens = wl.make_rollouts(w)
    sel = oracle.select(rewards, w.m)
    cu, tokens, _, seq_of_row = oracle.compact(sel["idx"], w.n, lengths, src_tokens)
    return sel, cu, tokens, seq_of_row


def _sample_rows(lo, hi, cu, count, rng):
    """Rows of [lo, hi): the first and last, rows on both sides of rollout boundaries, and random ones."""
    picks = {lo, hi - 1}
    edges = cu[(cu > lo) & (cu < hi)]
    for e in edges[:6]:
        picks.update((int(e) - 1, int(e)))
    picks.update(int(x) for x in rng.integers(lo, hi, size=count))
    return np.array(sorted(picks), np.int64)


def _check_rows(b, rows, gpu_logp_rows, gpu_dl_bits):
    """Oracle on the given global rows; compares log-probs and gradient rows.  Returns the oracle's output."""
    want = oracle.grpo_rows(b["logits_rows"], b["tokens"][rows], b["old"][rows], b["ref"][rows], b["adv32"], b["sw"],
                            b["seq_of_row"][rows], b["mask"][rows], b["w"].eps, b["w"].beta, want_dlogits=True)
    assert want["bad_tokens"] == 0
    assert np.abs(gpu_logp_rows - want["logp"]).max() <= LOGP_ATOL
    fragile = (want["margin"] < CLIP_MARGIN) & (want["margin"] > 0)
    assert int(fragile.sum()) == 0
    slack = gradient_slack({"w": b["w"], "mask": b["mask"], "cu": b["cu"], "seq_of_row": b["seq_of_row"],
                            "adv32": b["adv32"], "old": b["old"], "ref": b["ref"]}, want, rows=rows)
    rep = dlogits_report(gpu_dl_bits, want["dlogits"], slack)
    assert_dlogits_close(rep)
    rep["logp_abs"] = float(np.abs(gpu_logp_rows - want["logp"]).max())
    want["report"] = rep
    return want


def _merge(total, rep):
    for k in ("literal_ulps", "allowance_ulps", "logp_abs"):
        total[k] = max(total.get(k, 0.0), rep[k])
    for k in ("allowance_rows", "rows"):
        total[k] = total.get(k, 0) + rep[k]


@needs_big_gpu
def test_config2_at_bench_size_and_launch_configuration():
    w = wl.WORKLOADS["c2_qwen_vocab"]
    sel, cu, tokens, seq_of_row = _selection_and_layout(w)
    T = int(cu[-1])
    assert T == 36853
    dev = torch.device("cuda:0")
    tok_d = torch.from_numpy(tokens).to(dev)
    logits = wl.make_logits_device(w, tok_d)
    old, ref = wl.make_old_ref(w, wl.library_logp(logits, tok_d).cpu().numpy())
    adv32 = sel["adv"].astype(np.float32).reshape(-1)
    mask = np.ones(T, np.uint8)
    sw = oracle.seq_weights(mask, cu)

    # the CUDA path exactly as bench.py launches it
    cu_d = torch.from_numpy(cu).to(dev)
    sw_d = binding.grpo_seq_weights(None, cu_d)
    old_d, ref_d, adv_d = torch.from_numpy(old).to(dev), torch.from_numpy(ref).to(dev), torch.from_numpy(adv32).to(dev)
    dl = torch.empty_like(logits)
    logp = torch.empty(T, dtype=torch.float32, device=dev)
    acc = torch.zeros(1, dtype=torch.float64, device=dev)
    loss = torch.empty(1, dtype=torch.float32, device=dev)
    status = binding.new_status(dev)
    chunk = w.chunk_rows
    ws = torch.empty(binding.grpo_loss_chunk_workspace_bytes(chunk), dtype=torch.uint8, device=dev)
    for lo in range(0, T, chunk):
        hi = min(T, lo + chunk)
        binding.grpo_loss_chunk(logits[lo:hi], tok_d[lo:hi], old_d[lo:hi], ref_d[lo:hi], adv_d, sw_d, cu_d, lo, None,
                                w.eps, w.beta, acc, logp[lo:hi], dl[lo:hi], ws, status=status)
    binding.grpo_loss_finalize(acc, loss)
    torch.cuda.synchronize()
    assert binding.read_status(status) == 0
    np.testing.assert_allclose(sw_d.cpu().numpy(), sw, rtol=1e-15)

    # oracle over ALL rows: log-probs, loss terms and every gradient element, in blocks so that the fp64
    # gradient rows of a block (1024 x 151936 x 8 B = 1.2 GB) stay small on the host
    ell = np.empty(T, np.float64)
    logp_o = np.empty(T, np.float64)
    b = {"w": w, "tokens": tokens, "old": old, "ref": ref, "adv32": adv32, "sw": sw, "seq_of_row": seq_of_row,
         "mask": mask, "cu": cu}
    total = {}
    block = 1024
    for lo in range(0, T, block):
        hi = min(T, lo + block)
        rows = np.arange(lo, hi, dtype=np.int64)
        b["logits_rows"] = logits[lo:hi].view(torch.uint16).cpu().numpy()
        out = _check_rows(b, rows, logp[lo:hi].cpu().numpy(), dl[lo:hi].view(torch.uint16).cpu().numpy())
        ell[lo:hi], logp_o[lo:hi] = out["ell"], out["logp"]
        _merge(total, out["report"])
        del out
    assert total["rows"] == T
    loss_o = oracle.grpo_loss(ell, mask, cu)
    scale = np.mean([abs(ell[cu[i]:cu[i + 1]].mean()) for i in range(len(cu) - 1)])
    d = abs(float(loss.item()) - loss_o)
    record("c2_qwen_vocab, all %d rows, 16384-row chunk launches" % T, V=w.V, loss=loss_o,
           loss_rel_literal=d / abs(loss_o), loss_rel_conditioned=d / max(abs(loss_o), scale / LOSS_COND), **total)
    assert d <= LOSS_RTOL * max(abs(loss_o), scale / LOSS_COND)
    assert d <= LOSS_RTOL * abs(loss_o)       # this batch meets the literal bound too


@needs_big_gpu
def test_config5_chunked_in_place_first_middle_and_last_chunk():
    w = wl.WORKLOADS["c5_large_loss"]
    sel, cu, tokens, seq_of_row = _selection_and_layout(w)
    T = int(cu[-1])
    chunk = w.chunk_rows
    n_chunks = (T + chunk - 1) // chunk
    assert n_chunks >= 8 and chunk % 2048 == 0
    dev = torch.device("cuda:0")
    adv32 = sel["adv"].astype(np.float32).reshape(-1)
    mask = np.ones(T, np.uint8)
    sw = oracle.seq_weights(mask, cu)
    cu_d = torch.from_numpy(cu).to(dev)
    sw_d = binding.grpo_seq_weights(None, cu_d)
    adv_d = torch.from_numpy(adv32).to(dev)
    acc = torch.zeros(1, dtype=torch.float64, device=dev)
    status = binding.new_status(dev)
    ws = torch.empty(binding.grpo_loss_chunk_workspace_bytes(chunk), dtype=torch.uint8, device=dev)
    checked = {0, n_chunks // 2, n_chunks - 1}
    rng = np.random.default_rng(1)
    straddling = 0
    for c in range(n_chunks):
        lo, hi = c * chunk, min(T, (c + 1) * chunk)
        tok_d = torch.from_numpy(tokens[lo:hi]).to(dev)
        logits = wl.make_logits_device(w, tok_d, row0=lo)                 # this chunk's rows only
        # old/ref: log-prob + noise, drawn per chunk from the chunk's own stream
        lt = wl.library_logp(logits, tok_d).cpu().numpy()
        noise = np.random.Generator(np.random.PCG64([w.seed, 3, c]))
        old = (lt + noise.normal(0.0, w.old_sigma, size=hi - lo)).astype(np.float32)
        ref = (lt + noise.normal(0.0, w.ref_sigma, size=hi - lo)).astype(np.float32)
        logp = torch.empty(hi - lo, dtype=torch.float32, device=dev)
        keep = None
        if c in checked:
            rows = _sample_rows(lo, hi, cu, 32, rng)
            rows_d = torch.from_numpy(rows - lo).to(dev)
            keep = logits[rows_d].view(torch.uint16).cpu().numpy()        # the inputs, before they are overwritten in place
            host_bits = logits.view(torch.uint16).cpu().numpy()
        before = float(acc.item())
        binding.grpo_loss_chunk(logits, tok_d, torch.from_numpy(old).to(dev), torch.from_numpy(ref).to(dev), adv_d, sw_d,
                                cu_d, lo, None, w.eps, w.beta, acc, logp, logits, ws, status=status)     # in place
        torch.cuda.synchronize()
        if c not in checked:
            continue
        inside = cu[(cu > lo) & (cu < hi)]
        straddling += int(lo not in cu) + int(hi not in cu and hi < T)
        assert len(inside) > 0
        # the whole chunk: log-probs and the chunk's share of the loss
        out = oracle.grpo_rows(host_bits, tokens[lo:hi], old, ref, adv32, sw, seq_of_row[lo:hi], mask[lo:hi],
                               w.eps, w.beta, want_dlogits=False)
        assert np.abs(logp.cpu().numpy() - out["logp"]).max() <= LOGP_ATOL
        share_o = float(np.sum(sw[seq_of_row[lo:hi]] * out["ell"]))
        share = float(acc.item()) - before
        size = float(np.sum(np.abs(sw[seq_of_row[lo:hi]] * out["ell"])))
        assert abs(share - share_o) <= LOSS_RTOL * max(abs(share_o), size / LOSS_COND)
        # sampled rows: the gradient, element by element
        full_old = np.zeros(T, np.float32)
        full_ref = np.zeros(T, np.float32)
        full_old[lo:hi], full_ref[lo:hi] = old, ref
        b = {"w": w, "tokens": tokens, "old": full_old, "ref": full_ref, "adv32": adv32, "sw": sw,
             "seq_of_row": seq_of_row, "mask": mask, "cu": cu, "logits_rows": keep}
        rep = _check_rows(b, rows, logp[rows_d].cpu().numpy(), logits[rows_d].view(torch.uint16).cpu().numpy())["report"]
        record("c5_large_loss, chunk %d of %d in place" % (c, n_chunks), V=w.V, rows_logp=hi - lo,
               logp_abs_all_rows=float(np.abs(logp.cpu().numpy() - out["logp"]).max()), chunk_loss_share=share_o,
               share_rel_literal=abs(share - share_o) / abs(share_o),
               share_rel_conditioned=abs(share - share_o) / max(abs(share_o), size / LOSS_COND), **rep)
        del host_bits
    assert straddling >= 2                                   # the checked chunks did cut rollouts in two
    assert binding.read_status(status) == 0 and np.isfinite(float(acc.item()))
