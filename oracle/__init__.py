"""CPU oracle for the swizzled tiled GEMM (TEST INFRASTRUCTURE, not product code).

Everything under this package is a plain, slow, obviously-correct CPU statement of
what the GPU path computes:

* ``oracle.remap``   -- tile-order permutations ("swizzles"), written by enumeration.
* ``oracle.gemm``    -- fp64-accumulated GEMM of bf16 inputs (plain C loops, see
  ``gemm_oracle.c``) and the element-wise comparison metric.
* ``oracle.l2model`` -- an LRU model of operand-panel reuse (a model, not parity).

Only the tests, the smoke check and the CPU-baseline leg of the benchmark may import
this package.  It shares no code, header, table or helper with the CUDA library and
never imports it; the CUDA library never imports this package.
"""
