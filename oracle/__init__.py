"""CPU oracle for exact-attention response replay (LongStraw, arxiv 2607.14952).

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this package:
only the test-suite, the smoke check and the benchmark's CPU-baseline leg do.
It is plain numpy in fp64, slow on purpose, and shares no code with the CUDA
library (not a header, not a helper, not a constant table).

Modules
-------
pages      integer page / shard arithmetic (Sec. "From Logical Shards to
           Physical Pages", Eq. qwen-page-owner, Eq. qwen-page-count,
           Eq. glm-tr-zigzag-pages).
attention  unsharded masked softmax attention and its analytic gradients
           (Eq. qwen-local-attn with one partition = the definition), the
           per-shard local attention, the LSE/output merge
           (Eq. qwen-lse-parts, Eq. qwen-global-attn) and the detached-prefix
           backward (Sec. "Lazy Gradient Pages", Eq. qwen-dq-reduce).

Pins (tests/test_oracle_*.py): worked page examples printed in the paper,
closed forms (identical keys, two-key hand example, one-hot limit), central
finite differences for every gradient, merge = unsharded for every split,
page-permutation bit-identity, and the P = 0 case against a library causal
attention.  Parity with the paper authors' own implementation is unpinned:
the paper prints no numeric output of this operator.
"""
