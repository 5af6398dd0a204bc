"""Seeded synthetic workloads shaped like the paper's rollout stage.

Holds data only: decoder shapes, the five benchmark configurations and generators
for prefix lengths / prefix tokens / teacher tokens.  None of the method's arithmetic
lives here (no Philox, no decoder maths), so the CPU oracle and the CUDA library can
both take their inputs from this module without sharing any implementation.

The paper samples G = 6..16 responses per question, caps generation at 4096 tokens,
and reports ~2.5k generated tokens per full-path sample against ~150-400 for RPO
(Section 4 and the token-count table); hence long shared prefixes (1k-6k tokens) and
short suffixes (128-256).  The open-rs prompts, cached reasoning paths and the
DeepSeek-R1-Distill-Qwen weights are not available offline: prefix tokens are i.i.d.
uniform over the vocabulary and weights are seeded N(0, 0.02).
"""
import numpy as np

SHAPES = {
    "tiny": dict(n_layers=2, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=64, d_ffn=688, vocab=1024,
                 rope_base=10000.0, rms_eps=1e-6, dtype="fp32"),
    "qwen1.5b-class": dict(n_layers=28, d_model=1536, n_q_heads=12, n_kv_heads=2, head_dim=128, d_ffn=8960,
                           vocab=151936, rope_base=1e6, rms_eps=1e-6, dtype="bf16"),
    "qwen7b-class": dict(n_layers=28, d_model=3584, n_q_heads=28, n_kv_heads=4, head_dim=128, d_ffn=18944,
                         vocab=152064, rope_base=1e6, rms_eps=1e-6, dtype="bf16"),
}

KV_BLOCK_TOKENS = 16

CONFIGS = {
    "cfg1_tiny": dict(shape="tiny", n_groups=2, G=4, prefix=("fixed", 128), suffix=32,
                      sampler=dict(temperature=1.0, top_p=0.9, greedy=False, eos_id=-1)),
    "cfg2_1p5b_16x8": dict(shape="qwen1.5b-class", n_groups=16, G=8, prefix=("fixed", 2048), suffix=128,
                           sampler=dict(temperature=1.0, top_p=0.95, greedy=False, eos_id=-1)),
    "cfg3_1p5b_64x8_ragged": dict(shape="qwen1.5b-class", n_groups=64, G=8, prefix=("uniform", 1024, 6144),
                                  suffix=256, sampler=dict(temperature=1.0, top_p=0.95, greedy=False, eos_id=2)),
    "cfg4_7b_32x8": dict(shape="qwen7b-class", n_groups=32, G=8, prefix=("fixed", 4096), suffix=256,
                         sampler=dict(temperature=1.0, top_p=0.95, greedy=False, eos_id=-1), logprobs=True),
    "cfg5_7b_partial": dict(shape="qwen7b-class", n_groups=32, G=8, prefix=("fixed", 4096), suffix=256,
                            sampler=dict(temperature=1.0, top_p=0.95, greedy=False, eos_id=-1)),
    "cfg5_7b_full": dict(shape="qwen7b-class", n_groups=32, G=8, prefix=("fixed", 256), suffix=4352,
                         sampler=dict(temperature=1.0, top_p=0.95, greedy=False, eos_id=-1)),
}


def shape_with(name, **over):
    s = dict(SHAPES[name]); s.update(over); return s


def prefix_lengths(cfg, seed=0, n_groups=None):
    n = cfg["n_groups"] if n_groups is None else n_groups
    spec = cfg["prefix"]
    if spec[0] == "fixed":
        return np.full(n, spec[1], dtype=np.int32)
    rng = np.random.Generator(np.random.PCG64([seed, 101]))
    return rng.integers(spec[1], spec[2] + 1, size=n).astype(np.int32)


def rank_group_ids(n_groups, rank):
    """Group ids of a rank when prompt groups are sharded over ranks (each rank its own groups,
    ids disjoint so that the samples' random streams differ)."""
    return np.arange(n_groups, dtype=np.int32) + np.int32(rank * n_groups)


def prefix_tokens(lengths, vocab, seed=0):
    """Concatenated uniform token ids and the offsets array [n_groups + 1]."""
    rng = np.random.Generator(np.random.PCG64([seed, 202]))
    offsets = np.zeros(len(lengths) + 1, dtype=np.int32)
    offsets[1:] = np.cumsum(lengths)
    return rng.integers(0, vocab, size=int(offsets[-1])).astype(np.int32), offsets


def teacher_tokens(n_seq, n_steps, vocab, seed=0):
    """Uniform suffix tokens used to teacher-force both implementations identically."""
    rng = np.random.Generator(np.random.PCG64([seed, 303]))
    return rng.integers(0, vocab, size=(n_seq, n_steps)).astype(np.int32)


def logits_rows(n_rows, vocab, sigma, seed=0, bf16_like=False):
    """Synthetic float32 logits rows ~ N(0, sigma^2) for sampler tests.

    bf16_like rounds the values to 8 significant bits so that many exact ties occur,
    as they do for logits born from low-precision arithmetic.
    """
    rng = np.random.Generator(np.random.PCG64([seed, 404]))
    x = (rng.standard_normal((n_rows, vocab)) * sigma).astype(np.float32)
    if bf16_like:
        b = x.view(np.uint32) & np.uint32(0xFFFF0000)
        x = b.view(np.float32)
    return x
