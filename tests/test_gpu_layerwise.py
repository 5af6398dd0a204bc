"""Full-depth parity, layer by layer.

A bf16 decoder rounds its GEMM inputs, K/V and attention output in every layer, and the 28 layers'
roundings add up in the residual stream: against the float64 oracle run end to end, the logits of
ANY 16-bit implementation sit ~0.08 away at depth 28 (a float32 CUDA-core path with the same storage
lands in the same place), which says nothing about whether a kernel is right.  Just as the tokens are
teacher-forced so that sampled trajectories cannot diverge, the hidden state is teacher-forced here:
the library records the input and output of every layer (rpo_debug_tap) and the oracle - the plain
float64 definition, no rounding model - computes each layer from the library's own input of that
layer.  What is compared is then one layer's worth of rounding, for every layer of the full model
over the full prefix, and the stated tolerances (logits 3e-2, log-probs 2e-2, greedy arg max where the
oracle's top-2 gap exceeds 0.05) apply to the oracle's head on the library's last hidden state.

Per-layer bounds.  A layer rounds five tensors to bf16 (relative error <= 2^-9, rms 2^-9/sqrt(3) =
1.1e-3 each): its output deviates by ~2.5e-3 of the rms of the layer's increment, with the largest of
millions of elements up to ~10x that (5 sigma, on elements above the row's rms): measured <= 0.05.
(Layer 0 starts from the embedding rows, whose entries are ~0.02: its attention increment is as large
as the row it is added to, so the second RMSNorm amplifies that increment's rounding; rms bound 1.5e-2.)
The attention output alone: rms deviation 4-6e-3 of its rms; its largest element deviates by up to
0.1 row-rms at the 7B widths, where the scores have std 1.6 and a handful of keys carry a row (the
float32 CUDA-core path shows the same element and value).  A dropped key tile or a wrong block id
moves these quantities by O(1)."""
import numpy as np
import pytest

import workloads
from gpu_util import oracle_shape, make_ctx, layerwise_errors

pytestmark = pytest.mark.gpu


def _run(shape, P, G, S, seed):
    sh = oracle_shape(shape)
    with make_ctx(shape, 1, G, P, S, chunk=max(1024, P)) as ctx:
        ctx.init_weights(0, 0.02)
        toks, _ = workloads.prefix_tokens(np.array([P], dtype=np.int32), sh.vocab, seed=seed)
        forced = workloads.teacher_tokens(G, S, sh.vocab, seed=seed + 1)
        r = layerwise_errors(ctx, shape, sh, toks, G, S, forced)
        assert ctx.device_status() == 0
    return r


def _assert_layerwise(r, attn_max):
    assert max(r["x_prefill"]) <= 0.08 and max(r["x_decode"]) <= 0.08, (r["x_prefill"], r["x_decode"])
    assert max(r["attn_prefill"]) <= attn_max and max(r["attn_decode"]) <= attn_max, (r["attn_prefill"], r["attn_decode"])
    assert max(r["x_rms"][1:]) <= 8e-3 and r["x_rms"][0] <= 1.5e-2 and max(r["attn_rms"]) <= 1.2e-2, (r["x_rms"], r["attn_rms"])
    # the stated tolerances, on the last hidden state the library itself produced
    assert r["logits_err"] <= 3e-2 and r["logprob_err"] <= 2e-2 and r["argmax_ok"], r


def test_config2_slice_full_depth_full_prefix():
    """1.5B-class decoder, all 28 layers, one prompt group with the configuration's 2048-token prefix
    (8 prefix splits in the decode attention), G = 8, four suffix positions."""
    r = _run(workloads.shape_with("qwen1.5b-class"), 2048, 8, 4, seed=40)
    _assert_layerwise(r, attn_max=0.05)
    assert r["clear_steps"] >= 8


def test_7b_slice_full_depth():
    """7B-class decoder, all 28 layers, a 650-token prefix with a partial last KV block, G = 8 (56 query
    rows per KV head in the decode attention)."""
    r = _run(workloads.shape_with("qwen7b-class"), 650, 8, 3, seed=42)
    _assert_layerwise(r, attn_max=0.15)


def test_7b_widths_config4_prefix_length():
    """7B-class widths with the 4096-token prefix of configurations 4 and 5 (two 2048-key prefix splits
    per group and KV head), two layers."""
    r = _run(workloads.shape_with("qwen7b-class", n_layers=2), 4096, 8, 3, seed=44)
    _assert_layerwise(r, attn_max=0.15)
