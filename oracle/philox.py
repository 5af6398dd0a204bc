"""Philox4x32-10 counter-based generator (Salmon, Moraes, Dror, Shaw, SC'11), numpy.

The rollout draws one uniform per (sequence, step) for the sampler of Eq. 3's
pi_theta(. | q_k, prefix) and four normals per counter for the seeded weight
initialisation; both are keyed by a 64-bit seed.  Counter layout used by this
project (stated once here, restated independently in the CUDA library):

  sampler draw : counter = (step, seq_lo, seq_hi, 0)        key = (seed_lo, seed_hi)
  weight init  : counter = (blk_lo, blk_hi, tensor_id, 1)   key = (seed_lo, seed_hi)

where blk = element_index // 4 and the four output words serve elements 4*blk..4*blk+3.
"""
import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = 0x9E3779B9
_W1 = 0xBB67AE85
_MASK = np.uint64(0xFFFFFFFF)
_S32 = np.uint64(32)


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Vectorised Philox4x32 with 10 rounds.

    c0..c3: array-likes of counters (broadcast together, any shape, values < 2**32).
    k0, k1: python ints, the two 32-bit key words.
    Returns four uint32 arrays (x0, x1, x2, x3).
    """
    c0, c1, c2, c3 = np.broadcast_arrays(*(np.asarray(c, dtype=np.uint64) for c in (c0, c1, c2, c3)))
    c0 = c0.copy(); c1 = c1.copy(); c2 = c2.copy(); c3 = c3.copy()
    k0 = int(k0) & 0xFFFFFFFF
    k1 = int(k1) & 0xFFFFFFFF
    for _ in range(10):
        p0 = _M0 * c0            # 64-bit product of two 32-bit values: exact in uint64
        p1 = _M1 * c2
        hi0 = p0 >> _S32; lo0 = p0 & _MASK
        hi1 = p1 >> _S32; lo1 = p1 & _MASK
        n0 = hi1 ^ c1 ^ np.uint64(k0)
        n2 = hi0 ^ c3 ^ np.uint64(k1)
        c0, c1, c2, c3 = n0, lo1, n2, lo0
        k0 = (k0 + _W0) & 0xFFFFFFFF   # Weyl key schedule, bumped after every round
        k1 = (k1 + _W1) & 0xFFFFFFFF
    return tuple(c.astype(np.uint32) for c in (c0, c1, c2, c3))


def split_seed(seed):
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    return seed & 0xFFFFFFFF, seed >> 32


def sampler_u24(seed, seq, step):
    """24-bit uniform integer for the draw of sequence `seq` at suffix step `step`."""
    k0, k1 = split_seed(seed)
    seq = np.asarray(seq, dtype=np.uint64)
    x0, _, _, _ = philox4x32_10(np.asarray(step, dtype=np.uint64), seq & _MASK, seq >> _S32, 0, k0, k1)
    return (x0 >> np.uint32(8)).astype(np.uint32)
