"""CPU oracle for the RPO suffix-rollout path (test infrastructure, not product code).

This package is a plain, slow, obviously-correct restatement of what the rollout path
computes: seeded weight initialisation, the decoder forward over a cached reasoning
prefix, batched suffix generation for the G samples of a sampling group (Eq. 3,
Algorithm 1 rollout loop) and the per-token log-probabilities pi(o_j | q, o_<j) that
the probability ratio of Eq. 7 consumes.

It shares no code with the CUDA library and must never be imported by the product
package; only the test-suite, the smoke check and the benchmark's CPU-baseline leg
use it.  Floating point runs in float64 by default (float32 on request for large
slices); integer/bit work (Philox words, quantised sampler weights, token ids) is
exact.

Parity status: every routine here is pinned by the not-gpu tests (closed forms,
invariants, brute force on tiny inputs, torch CPU library routines).  The only
unpinned statement is about the *trained* model of the paper (weights, tokenizer and
datasets are not available): "parity unpinned" for that, by necessity.
"""
from . import philox, exactmath, init, decoder, sampler, rollout, objective  # noqa: F401
