"""Pins for the oracle's bit-level building blocks: Philox, reproducible float32
functions, bf16 rounding and the seeded normal initialisation."""
import math
import os
import subprocess
import sys
import numpy as np
import pytest
import torch
from oracle import philox, exactmath as em, init, decoder

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_TRITON_SNIPPET = r'''
import os, sys
os.environ["TRITON_INTERPRET"] = "1"
import numpy as np, torch, triton, triton.language as tl
@triton.jit
def k(out_ptr, c_ptr, k0, k1, N: tl.constexpr):
    i = tl.arange(0, N)
    c0 = tl.load(c_ptr + i).to(tl.uint32); c1 = tl.load(c_ptr + N + i).to(tl.uint32)
    c2 = tl.load(c_ptr + 2 * N + i).to(tl.uint32); c3 = tl.load(c_ptr + 3 * N + i).to(tl.uint32)
    z = c0 * 0
    a, b, c, d = tl.philox_impl(c0, c1, c2, c3, (z + k0).to(tl.uint32), (z + k1).to(tl.uint32), 10)
    tl.store(out_ptr + i, a); tl.store(out_ptr + N + i, b)
    tl.store(out_ptr + 2 * N + i, c); tl.store(out_ptr + 3 * N + i, d)
N = 64
ctr = np.load(sys.argv[1]); k0, k1 = int(sys.argv[2]), int(sys.argv[3])
out = torch.zeros(4 * N, dtype=torch.int32)
k[(1,)](out, torch.from_numpy(ctr.view(np.int32).reshape(-1).copy()), k0, k1, N)
np.save(sys.argv[4], out.numpy().view(np.uint32).reshape(4, N))
'''


def test_philox_matches_library_implementation(tmp_path):
    """Re-derive the words with an unrelated Philox (Triton's, run by its CPU interpreter)."""
    rng = np.random.default_rng(5)
    ctr = rng.integers(0, 2 ** 32, size=(4, 64), dtype=np.uint64).astype(np.uint32)
    ctr[:, 0] = 0
    ctr[:, 1] = 0xFFFFFFFF
    k0, k1 = 0x7FFFFFF1, 0x12345678 & 0x7FFFFFFF
    src = tmp_path / "tri.py"; src.write_text(_TRITON_SNIPPET)
    cin, cout = tmp_path / "c.npy", tmp_path / "o.npy"
    np.save(cin, ctr)
    r = subprocess.run([sys.executable, str(src), str(cin), str(k0), str(k1), str(cout)],
                       capture_output=True, text=True, timeout=600)
    # no skip: without this run the Philox words would be pinned by statistics only
    assert r.returncode == 0, "the independent Philox (Triton's CPU interpreter) did not run: " + r.stderr[-500:]
    got = np.stack(philox.philox4x32_10(ctr[0], ctr[1], ctr[2], ctr[3], k0, k1))
    assert np.array_equal(got, np.load(cout))


def test_philox_round_is_a_bijection_and_uses_every_input_word():
    base = np.stack(philox.philox4x32_10(1, 2, 3, 4, 5, 6)).ravel()
    for args in [(0, 2, 3, 4, 5, 6), (1, 0, 3, 4, 5, 6), (1, 2, 0, 4, 5, 6), (1, 2, 3, 0, 5, 6),
                 (1, 2, 3, 4, 0, 6), (1, 2, 3, 4, 5, 0)]:
        other = np.stack(philox.philox4x32_10(*args)).ravel()
        flipped = sum(bin(int(a) ^ int(b)).count("1") for a, b in zip(base, other))
        assert 40 < flipped < 88          # avalanche: ~64 of 128 bits change
    n = 1 << 16
    x = philox.philox4x32_10(np.arange(n), 0, 0, 0, 9, 9)
    words = set(zip(*[w.tolist() for w in x]))
    assert len(words) == n                 # distinct counters -> distinct outputs
    bits = np.unpackbits(np.stack(x).view(np.uint8))
    assert abs(bits.mean() - 0.5) < 2e-3


def test_sampler_draw_counter_layout():
    u = philox.sampler_u24(seed=(7 << 32) | 9, seq=np.array([3, (1 << 33) + 5]), step=11)
    a = philox.philox4x32_10(11, 3, 0, 0, 9, 7)[0] >> 8
    b = philox.philox4x32_10(11, 5, 2, 0, 9, 7)[0] >> 8
    assert u.tolist() == [int(a), int(b)]


def test_ln_exp_sincos_accuracy_and_special_values():
    rng = np.random.default_rng(1)
    u = ((rng.integers(0, 2 ** 23, 200000).astype(np.float32) + np.float32(0.5)) * np.float32(2.0 ** -23))
    ref = np.log(u.astype(np.float64))
    assert np.max(np.abs(em.ln_unit(u) - ref)) < 2e-6
    assert em.ln_unit(np.float32(1.0)) == 0.0
    assert abs(float(em.ln_unit(np.float32(0.5))) + math.log(2)) < 1e-7
    x = -rng.random(200000).astype(np.float32) * np.float32(24.0)
    e = em.exp_nonpos(x)
    assert np.max(np.abs(e / np.exp(x.astype(np.float64)) - 1)) < 4e-7
    assert em.exp_nonpos(np.float32(0.0)) == np.float32(1.0)
    assert em.exp_nonpos(np.float32(-24.0001)) == 0.0 and em.exp_nonpos(np.float32(-1e30)) == 0.0
    assert np.all(np.diff(em.exp_nonpos(np.sort(x))) >= -1e-9)          # monotone up to rounding
    k = rng.integers(0, 2 ** 24, 200000).astype(np.uint32)
    s, c = em.sincos_turn24(k)
    a = 2 * np.pi * k.astype(np.float64) / 2 ** 24
    assert np.max(np.abs(s - np.sin(a))) < 4e-7 and np.max(np.abs(c - np.cos(a))) < 4e-7
    s0, c0 = em.sincos_turn24(np.array([0, 1 << 22, 1 << 23, 3 << 22], dtype=np.uint32))
    assert s0.tolist() == [0.0, 1.0, -0.0, -1.0] or s0.tolist() == [0.0, 1.0, 0.0, -1.0]
    assert c0.tolist() in ([1.0, -0.0, -1.0, 0.0], [1.0, 0.0, -1.0, 0.0], [1.0, -0.0, -1.0, -0.0])
    assert all(v.dtype == np.float32 for v in (e, s, c, em.ln_unit(u)))


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(2)
    x = (rng.standard_normal(100000) * 0.02).astype(np.float32)
    x[:4] = [1.00390625, 1.01171875, -1.00390625, 0.0]        # exact ties: round to even
    ours = em.round_bf16(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(ours.view(np.uint32), ref.view(np.uint32))


def test_normal_init_statistics_and_determinism():
    from scipy import stats
    z = init.normal_tensor(seed=0, tensor_id=3, n_elems=1_000_003, std=1.0)
    assert z.dtype == np.float32 and z.size == 1_000_003
    assert abs(z.mean()) < 4e-3 and abs(z.std() - 1) < 3e-3
    assert abs((z ** 4).mean() - 3) < 0.03 and abs((z ** 3).mean()) < 0.02
    assert stats.kstest(z[:200000].astype(np.float64), "norm").pvalue > 1e-3
    assert abs(np.corrcoef(z[:-1], z[1:])[0, 1]) < 4e-3          # pair partners uncorrelated
    # chunking / threading must not change a single bit; element e depends only on (seed, id, e)
    z2 = init.normal_tensor(0, 3, 1_000_003, 1.0, chunk_blocks=777, threads=1)
    assert np.array_equal(z.view(np.uint32), z2.view(np.uint32))
    assert not np.array_equal(z[:100], init.normal_tensor(1, 3, 100, 1.0))
    assert not np.array_equal(z[:100], init.normal_tensor(0, 4, 100, 1.0))
    w = init.normal_tensor(0, 3, 1000, 0.02)
    assert np.array_equal(w, (z[:1000] * np.float32(0.02)).astype(np.float32))


def test_box_muller_against_direct_formula():
    """Element values re-derived from the Philox words with libm in float64."""
    k0, k1 = philox.split_seed(42)
    blk = np.arange(50, dtype=np.uint64)
    x = philox.philox4x32_10(blk, 0, 9, 1, k0, k1)
    z = init.normal_tensor(42, 9, 200, 1.0).reshape(50, 4)
    for j, (a, b) in enumerate(((0, 1), (2, 3))):
        u1 = ((x[a] >> 9).astype(np.float64) + 0.5) / 2 ** 23
        th = 2 * np.pi * (x[b] >> 8).astype(np.float64) / 2 ** 24
        r = np.sqrt(-2 * np.log(u1))
        assert np.max(np.abs(z[:, 2 * j] - r * np.cos(th))) < 3e-6
        assert np.max(np.abs(z[:, 2 * j + 1] - r * np.sin(th))) < 3e-6


def test_init_weights_layout_and_bf16():
    sh = decoder.Shape(2, 64, 4, 2, 16, 96, 128, dtype="bf16")
    w = init.init_weights(sh, seed=3, std=0.02)
    assert w["layers.1.wq"].shape == (64, 64) and w["layers.0.wk"].shape == (32, 64)
    assert w["layers.0.wo"].shape == (64, 64) and w["layers.0.wg"].shape == (96, 64)
    assert w["layers.0.wd"].shape == (64, 96) and w["embed"].shape == (128, 64) == w["lm_head"].shape
    assert np.all(w["gf"] == 1) and np.all(w["layers.0.g1"] == 1) and np.all(w["layers.1.g2"] == 1)
    for t in ("embed", "layers.1.wd"):
        assert np.array_equal(w[t], em.round_bf16(w[t]))       # representable in bf16
    raw = init.normal_tensor(3, init.layer_tensor_id(1, "wd"), 64 * 96, 0.02).reshape(64, 96)
    assert np.array_equal(w["layers.1.wd"], em.round_bf16(raw))
    assert not np.array_equal(w["embed"], w["lm_head"])         # untied, separately drawn
    wc = init.init_weights(sh, seed=3, std=0.02, compact_bf16=True)
    assert wc["embed"].dtype == np.uint16
    assert np.array_equal(decoder.mat(wc, "embed", np.float32), w["embed"])
