"""CPU oracle for the weight-remap path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, element-by-element statement of what the transfer computes, written
from the paper's definition of layout correspondence (Section 3.1: two in-GPU
elements correspond iff the same checkpoint element supplies both).  It shares no
code with the CUDA library or its planner and must never be imported by the product
path; only the tests, the smoke check and the benchmark's CPU-baseline leg use it.

Pins (see tests marked "not gpu"):
  cast.f32_to_bf16_bits   exact-rational nearest/ties-to-even check, torch CPU cast on
                          all non-NaN inputs sampled, special-value table.
                          NaN -> 0x7FFF is a reading of ours (the paper assumes equal
                          precisions): parity unpinned for NaN inputs.
  remap.remap_oracle      brute-force join on materialised element ids of both sides,
                          torch cat/stack/chunk statements of the fused rollout tensors,
                          hand-worked 4x6 micro case, exactly-once counters, inverse
                          remap identity.
  remap.checkpoint_view   equality with the seeded checkpoint tensors the trainer
                          buffers were loaded from.
  quant.e4m3_encode / e4m3_decode / quantize / dequantize
                          (Section 5 sketches pre-transfer quantisation and fixes no rule: the
                          rule is a reading of ours, parity unpinned by the paper) format definition
                          in exact rationals, torch's CPU float8_e4m3fn table and cast inside the
                          finite range, brute-force nearest-even over all codes incl. every
                          midpoint, saturation and NaN table, scale rule and round-trip bound.
  The order of payloads inside a transfer bucket and the rule that picks which trainer
  replica supplies a replicated element are planner choices the paper does not fix:
  parity unpinned by the paper, checked only against the directory the library reports
  and against replica-independence of the result.
"""
from .cast import f32_to_bf16_bits, bf16_to_f32_bits, cast_bits
from .remap import (remap_oracle, checkpoint_view, OracleResult, UncoveredError,
                    ReplicaMismatchError, DoubleWriteError, source_of_rollout_element,
                    SampleIndex)

__all__ = ["f32_to_bf16_bits", "bf16_to_f32_bits", "cast_bits", "remap_oracle",
           "checkpoint_view", "OracleResult", "UncoveredError", "ReplicaMismatchError",
           "DoubleWriteError", "source_of_rollout_element", "SampleIndex"]
