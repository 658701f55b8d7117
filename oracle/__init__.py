"""CPU oracle for the complete-expert sparse-MoE layer forward (ExactMoE).

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, numpy restatement of
what the hot path computes.  It shares no code with the CUDA library, imports
nothing from it, and nothing on the product path may import it: only the test
suite, the smoke check and the benchmark's CPU-baseline leg call it.

Modules (each function cites the passage of the paper it follows):

  bf16.py    BF16 <-> float helpers (exact widening, round-to-nearest-even).
  quant.py   Symmetric group-128 int4 quantiser and its dequantiser (Eq. 3).
  layout.py  Packed byte layout of one expert (Eq. 4 size model, Section 3.2/3.3
             "same representation in host pool and GPU slot").
  moe.py     Sparse block output, per token over its selected experts (Eq. 2).
  cache.py   Slot cache: global-expert -> slot map, LRU, waves, expert map with
             sentinel, token grouping (Sections 3.3 and 3.4).
  router.py  Router logits, softmax over all experts, top-k with ties to the lower id (Eq. 1).

Pins (tests/test_oracle_*.py, run without a GPU) hold every function to
something other than itself: closed forms, invariants, brute force on tiny
inputs, reductions to library routines, and the paper's own printed numbers.
Parity unpinned: the paper's measured hit rates, tokens/s and accuracies need
its checkpoint, prompts and datasets; they are context, not pins.
"""
