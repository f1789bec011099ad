"""CPU oracle (test infrastructure, not the product).

Plain fp64 restatement of the blockwise verification step, written from the
paper's definitions in ``tsd_oracle.c`` and loaded here through ctypes.  Only
tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library never does, and the two share no code.

``theorem1`` holds the toy-model harness for the exactness theorem; ``interblock`` the joint
mask, trigger and two-tree acceptance of inter-block speculation (Section 3.4); ``commit`` the
bookkeeping that turns an accepted path into the next root and its sequential step indices;
``fp8`` the e4m3 decode and dequantisation of the FP8 K/V cache variant.
"""
from .binding import (  # noqa: F401
    BUILD_FLAGS,
    build,
    num_threads,
    dense_mask,
    masked_attention,
    confidence_topk,
    decode_rule,
    accept,
    draft_token_prob,
    build_draft_tree,
)
