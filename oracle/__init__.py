"""FP64 CPU oracle for the attention forward / backward path (test infrastructure only).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It shares no code with the CUDA path and is never tuned.

Two tiers:

* :mod:`oracle.exact` -- the exact softmax-attention forward and VJP in FP64 at
  the represented BF16 inputs (Eq. "row-attention", Eq. "row-gradients"); this
  is the parity target.  The arithmetic is the plain C in ``gproj_oracle.c``.
* :mod:`oracle.emulation` -- Algorithm 1 restated untiled in numpy with BF16 /
  FP32 roundings placed where the paper's Appendix "Implemented Arithmetic"
  places them; it pins the GProj semantics (for example the -24 witness).
"""
from .exact import (  # noqa: F401
    attn_fwd_bwd_f64,
    attn_rect_f64,
    head_rows_f64,
    head_keys_f64,
    num_threads,
    rel_l2_percent,
)
