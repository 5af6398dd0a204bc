"""Seeded weight initialisation: matrices ~ N(0, std^2), RMSNorm gains = 1.

The paper names the policy models only (Section 4, experimental setup); the decoder
shape and "random init N(0, 0.02)" come from the benchmark configurations.  Every
matrix element is a pure function of (seed, tensor id, element index): Philox block
blk = index // 4 yields four words; (x0, x1) and (x2, x3) each feed one Box-Muller
pair built from the reproducible float32 ln / sin / cos of `exactmath`, so the GPU
library must reproduce these values bit for bit.
"""
from concurrent.futures import ThreadPoolExecutor
import os
import numpy as np
from . import philox, exactmath as em

F = np.float32
STREAM_INIT = 1
TENSOR_EMBED = 0
TENSOR_LM_HEAD = 1
LAYER_TENSORS = ("wq", "wk", "wv", "wo", "wg", "wu", "wd")


def layer_tensor_id(layer, name):
    return 16 + 8 * layer + LAYER_TENSORS.index(name)


def _normals_for_blocks(blk, k0, k1, tensor_id):
    """Four standard normals per Philox block index (uint64 array)."""
    x0, x1, x2, x3 = philox.philox4x32_10(blk & np.uint64(0xFFFFFFFF), blk >> np.uint64(32),
                                          tensor_id, STREAM_INIT, k0, k1)
    out = np.empty((blk.size, 4), dtype=F)
    for j, (xa, xb) in enumerate(((x0, x1), (x2, x3))):
        u1 = (((xa >> np.uint32(9)).astype(F) + F(0.5)).astype(F) * F(2.0 ** -23)).astype(F)
        rad = np.sqrt((F(-2.0) * em.ln_unit(u1)).astype(F)).astype(F)
        sin, cos = em.sincos_turn24(xb >> np.uint32(8))
        out[:, 2 * j] = (rad * cos).astype(F)
        out[:, 2 * j + 1] = (rad * sin).astype(F)
    return out


def normal_tensor(seed, tensor_id, n_elems, std, chunk_blocks=1 << 18, threads=None):
    """float32 vector of n_elems draws, value = float32(std) * z, one rounding."""
    k0, k1 = philox.split_seed(seed)
    n_blocks = (n_elems + 3) // 4
    out = np.empty(n_blocks * 4, dtype=F)
    std = F(std)

    def work(lo):
        hi = min(lo + chunk_blocks, n_blocks)
        blk = np.arange(lo, hi, dtype=np.uint64)
        z = _normals_for_blocks(blk, k0, k1, tensor_id)
        out[4 * lo:4 * hi] = (z.reshape(-1) * std).astype(F)

    starts = list(range(0, n_blocks, chunk_blocks))
    threads = threads or min(len(starts), os.cpu_count() or 1)
    if threads <= 1:
        for s in starts:
            work(s)
    else:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(work, starts))
    return out[:n_elems]


def tensor_shapes(shape):
    """name -> (rows, cols); every matrix is stored [out_features, in_features]."""
    d, dh = shape.d_model, shape.head_dim
    hq, hkv, f, v = shape.n_q_heads, shape.n_kv_heads, shape.d_ffn, shape.vocab
    per_layer = {"wq": (hq * dh, d), "wk": (hkv * dh, d), "wv": (hkv * dh, d), "wo": (d, hq * dh),
                 "wg": (f, d), "wu": (f, d), "wd": (d, f)}
    out = {"embed": (v, d), "lm_head": (v, d)}
    for l in range(shape.n_layers):
        for n, s in per_layer.items():
            out[f"layers.{l}.{n}"] = s
    return out


def tensor_id_of(name):
    if name == "embed":
        return TENSOR_EMBED
    if name == "lm_head":
        return TENSOR_LM_HEAD
    _, l, n = name.split(".")
    return layer_tensor_id(int(l), n)


def init_tensor(shape, name, seed, std):
    """One named matrix with the values the model computes with, as float32.

    For a bf16 model these are the float32 draws rounded to bfloat16 (nearest even)
    and widened again.
    """
    rows, cols = tensor_shapes(shape)[name]
    w = normal_tensor(seed, tensor_id_of(name), rows * cols, std).reshape(rows, cols)
    if shape.dtype == "bf16":
        w = em.round_bf16(w)
    return w


def init_weights(shape, seed, std=0.02, compact_bf16=False):
    """All weights of the decoder.  Gains g1, g2 (per layer) and gf are ones.

    compact_bf16=True keeps bf16 models as uint16 bit patterns (half the memory);
    `decoder.mat` widens them on use.
    """
    w = {}
    for name in tensor_shapes(shape):
        t = init_tensor(shape, name, seed, std)
        if compact_bf16 and shape.dtype == "bf16":
            t = em.to_bf16_bits(t)
        w[name] = t
    for l in range(shape.n_layers):
        w[f"layers.{l}.g1"] = np.ones(shape.d_model, dtype=F)
        w[f"layers.{l}.g2"] = np.ones(shape.d_model, dtype=F)
    w["gf"] = np.ones(shape.d_model, dtype=F)
    return w
