"""CPU oracle for the segment training step with synthetic intermediate labels.

This package is TEST INFRASTRUCTURE, not product code.  It is a plain, slow,
fp64-accumulating NumPy restatement of what one training step of a network
segment computes (label generation, forward, loss, backward, optimizer).  It
shares no code with the CUDA library and never imports it; only the tests, the
smoke check and the CPU-baseline leg of the benchmark may import it.
"""
