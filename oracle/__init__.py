"""CPU oracle for the sensitive-sparse zeroth-order fine-tuning step.

TEST INFRASTRUCTURE ONLY.  Plain, slow, obviously-correct restatements of what the
paper's method computes, used to check the CUDA library.  Nothing here is part of
the product: only the tests, the smoke check and the benchmark's CPU-baseline leg
import it, and it shares no code with the CUDA path.

Modules
-------
szo_oracle    Philox4x32-10, Gaussian draw, group-wise int4 quantizer, sensitive-mask
              selection, sparse perturb / update, decomposed linear forward.
model_oracle  fp64 decoder forward (Llama-, Mistral-, OPT-shaped), losses, first-order
              gradients for the mask, SPSA estimate and the ZO-SGD step.

Parity status
-------------
The paper prints no worked numeric example of a step, a mask or a quantized tensor,
so absolute end-to-end values are "parity unpinned"; every function is pinned by
closed forms, invariants, brute force or library routines in tests/test_oracle_*.py.
The int4 rounding convention (uniform asymmetric, zero = group minimum, round half
to even) is the reading taken here: the paper allows any post-training quantizer, so
that convention is "parity unpinned" by the paper and pinned only by its invariants.
"""
