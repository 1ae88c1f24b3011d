"""CPU oracle for the DAF prefill-attention path.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the product path never does.  It imports nothing from the CUDA
package.
"""
from .daf_oracle import (  # noqa: F401
    build,
    num_important,
    aggregate,
    select,
    gather_rows,
    hybrid_kv,
    important_attn,
    qd_attn,
    full_causal_attn,
    fuse,
    deviation_scores,
    blend_attn,
    e4m3_decode,
    dequant_fp8,
    daf_layer,
    num_threads,
)
