"""CPU checker for the draft-tree verification step and the tri-gram store.

TEST INFRASTRUCTURE ONLY.  This package is a slow, plain numpy restatement of what
the verification step of adaptive draft-verification decoding computes ("Draft
Construction and Verification", Eq. 1, Algorithm 2).  It exists so that the CUDA
library can be compared against something written independently of it.  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may import it; the
library never does, and shares no code with it.

Pinned parts (see tests/test_oracle_*.py): bf16 rounding, RMSNorm, RoPE, SwiGLU and
the whole tree forward (against a library Llama run on every root-to-node path as an
ordinary causal sequence), greedy acceptance (against token-by-token autoregressive
decoding), cache append, tri-gram update (against a brute-force window count) and
top-k (against a full sort).

Parity unpinned: the `min_count` filter of `trigram.topk` and the `cap` saturation
value of `trigram.update` (the paper names a threshold t = 12, an increment and a
maximum without defining them); both default to inert values.
"""
