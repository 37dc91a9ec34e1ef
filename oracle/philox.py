"""Counter-based random numbers (oracle; test infrastructure).

Philox-4x32 with 10 rounds as published by Salmon, Moraes, Dror and Shaw,
"Parallel random numbers: as easy as 1, 2, 3" (SC 2011): per round
    (hi0, lo0) = M0 * c0,  (hi1, lo1) = M1 * c2
    c <- (hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0),   k <- k + (W0, W1)
with the multipliers and Weyl constants of that paper.

Streams used by the sampler and the verifier (row = b * N + node):
    counter = (block, row, step_lo, step_hi << 2 | stream), key = seed (lo, hi)
    stream 0: Gumbel uniforms, element j uses word j % 4 of block j // 4
    stream 1: accept uniform of child node `node` (block 0, word 0)
    stream 2: resample uniform of node `node`     (block 0, word 0)
"""

import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = 0x9E3779B9
_W1 = 0xBB67AE85
_MASK = np.uint64(0xFFFFFFFF)
_S32 = np.uint64(32)

STREAM_GUMBEL, STREAM_ACCEPT, STREAM_RESAMPLE = 0, 1, 2


def philox4x32_10(counter, key):
    """counter: [..., 4] uint32 array, key: (k0, k1).  Returns [..., 4] uint32."""
    c = np.asarray(counter, dtype=np.uint64)
    c0, c1, c2, c3 = c[..., 0], c[..., 1], c[..., 2], c[..., 3]
    k0, k1 = int(key[0]) & 0xFFFFFFFF, int(key[1]) & 0xFFFFFFFF
    for _ in range(10):
        p0 = _M0 * c0
        p1 = _M1 * c2
        hi0, lo0 = p0 >> _S32, p0 & _MASK
        hi1, lo1 = p1 >> _S32, p1 & _MASK
        c0, c1, c2, c3 = hi1 ^ c1 ^ np.uint64(k0), lo1, hi0 ^ c3 ^ np.uint64(k1), lo0
        k0 = (k0 + _W0) & 0xFFFFFFFF
        k1 = (k1 + _W1) & 0xFFFFFFFF
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def uniform_open(x):
    """32 random bits -> float32 in (0,1): ((x >> 9) + 0.5) * 2^-23 (exact in float32)."""
    return ((np.asarray(x, dtype=np.uint32) >> 9).astype(np.float64) + 0.5) * 2.0 ** -23


def uniform_halfopen(x):
    """32 random bits -> float32 in [0,1): (x >> 8) * 2^-24."""
    return (np.asarray(x, dtype=np.uint32) >> 8).astype(np.float64) * 2.0 ** -24


def _counters(blocks, row, step, stream):
    blocks = np.asarray(blocks, dtype=np.uint64)
    c = np.empty(blocks.shape + (4,), dtype=np.uint64)
    c[..., 0] = blocks
    c[..., 1] = row
    c[..., 2] = step & 0xFFFFFFFF
    c[..., 3] = (((step >> 32) << 2) | stream) & 0xFFFFFFFF
    return c


def stream_uniforms(seed, step, row, stream, count=1):
    """Uniforms of one (row, stream): Gumbel stream -> `count` values in (0,1)
    for elements 0..count-1; accept / resample streams -> one value in [0,1)."""
    key = (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    if stream == STREAM_GUMBEL:
        nblk = (count + 3) // 4
        words = philox4x32_10(_counters(np.arange(nblk), row, step, stream), key).reshape(-1)
        return uniform_open(words[:count]).astype(np.float32)
    words = philox4x32_10(_counters(np.zeros(1), row, step, stream), key)
    return uniform_halfopen(words[0, 0]).astype(np.float32)
