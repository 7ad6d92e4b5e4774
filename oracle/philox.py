"""Counter-based random numbers for the CPU oracle (test infrastructure only).

Philox4x32-10 as published by Salmon, Moraes, Dror and Shaw, "Parallel random
numbers: as easy as 1, 2, 3" (SC'11): a 128-bit counter and a 64-bit key are
mixed by ten rounds of two 32x32->64 multiplications, with the key bumped by
the Weyl constants between rounds.  The paper that defines G-CADA only says
that a minibatch is "randomly selected" (Section II-A) and that computing
times are i.i.d. exponential (Section II-B); the mapping of (seed, iteration,
group / worker, position) onto counters below is this library's convention.

This file is written with numpy uint64 arithmetic only and shares nothing with
the CUDA implementation.
"""
import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = np.uint64(0x9E3779B9)
_W1 = np.uint64(0xBB67AE85)
_MASK = np.uint64(0xFFFFFFFF)
_SH = np.uint64(32)

STREAM_BATCH = 0   # counter word 3 for minibatch indices
STREAM_DELAY = 1   # counter word 3 for straggler delays


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Ten-round Philox-4x32.  All arguments broadcastable integer arrays
    (values < 2**32).  Returns four uint64 arrays holding 32-bit words."""
    c0, c1, c2, c3, k0, k1 = (np.asarray(a, dtype=np.uint64) & _MASK
                              for a in (c0, c1, c2, c3, k0, k1))
    c0, c1, c2, c3, k0, k1 = np.broadcast_arrays(c0, c1, c2, c3, k0, k1)
    for _ in range(10):
        p0 = _M0 * c0          # fits in 64 bits: both factors < 2**32
        p1 = _M1 * c2
        hi0, lo0 = p0 >> _SH, p0 & _MASK
        hi1, lo1 = p1 >> _SH, p1 & _MASK
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0), lo1, (hi0 ^ c3 ^ k1), lo0
        k0 = (k0 + _W0) & _MASK
        k1 = (k1 + _W1) & _MASK
    return c0, c1, c2, c3


def _word(seed, a, b, k, stream):
    """32-bit word number `a` of the stream (b, k, stream): counter
    (a // 4, b, k, stream), key (seed low, seed high), output word a % 4."""
    a = np.asarray(a, dtype=np.uint64)
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    out = philox4x32_10(a >> np.uint64(2), b, k, stream,
                        seed & 0xFFFFFFFF, seed >> 32)
    sel = (a & np.uint64(3)).astype(np.int64)
    stacked = np.stack(np.broadcast_arrays(*out), axis=0)
    return np.take_along_axis(stacked, sel[None, ...], axis=0)[0]


def batch_indices(seed, k, g, batch, n_g):
    """Row numbers (global, int64) of minibatch xi_g^k: `batch` draws, uniform
    with replacement, from the n_g rows of shard g (rows g*n_g .. (g+1)*n_g-1).
    Draw j uses word j of stream (g, k, STREAM_BATCH); a 32-bit word w maps to
    floor(w * n_g / 2**32)."""
    j = np.arange(batch, dtype=np.uint64)
    w = _word(seed, j, g, k, STREAM_BATCH)
    local = (w * np.uint64(n_g)) >> _SH
    return (local + np.uint64(g) * np.uint64(n_g)).astype(np.int64)


def uniform01(seed, k, m):
    """u in (0,1) for worker(s) m at iteration k: (w + 0.5) / 2**32 with w word
    m of stream (0, k, STREAM_DELAY)."""
    w = _word(seed, np.asarray(m, dtype=np.uint64), 0, k, STREAM_DELAY)
    return (w.astype(np.float64) + 0.5) * 2.0 ** -32
