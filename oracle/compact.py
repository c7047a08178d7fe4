"""Concatenation of the kept rollouts across prompts.  TEST INFRASTRUCTURE ONLY.

The text after Algorithm 1 says that for a batch of prompts the procedure is
applied per prompt and the down-sampled rollouts are concatenated.  Rollout j of
group g is row g*n + j of the padded storage; kept sequence number g*m + j is
rollout idx[g, j].
"""
import numpy as np


def compact(idx, n, lengths, src_tokens, src_streams=()):
    """Pack the kept rollouts.

    idx [G,m] int; lengths [G*n]; src_tokens [G*n, Lmax]; src_streams: sequence
    of [G*n, Lmax] arrays gathered the same way.  Returns (cu_seqlens int64
    [G*m+1], tokens [T], list of packed streams, seq_of_row int32 [T]).
    """
    idx = np.asarray(idx)
    G, m = idx.shape
    cu = [0]
    toks, streams, seq = [], [[] for _ in src_streams], []
    for g in range(G):
        for j in range(m):
            row = g * n + int(idx[g, j])
            L = int(lengths[row])
            toks.append(np.asarray(src_tokens[row, :L]))
            for s, src in zip(streams, src_streams):
                s.append(np.asarray(src[row, :L]))
            seq.append(np.full(L, g * m + j, np.int32))
            cu.append(cu[-1] + L)
    cat = lambda parts, dt: np.concatenate(parts).astype(dt) if parts else np.zeros(0, dt)
    return (np.asarray(cu, np.int64), cat(toks, np.int32),
            [cat(s, src.dtype) for s, src in zip(streams, src_streams)], cat(seq, np.int32))
