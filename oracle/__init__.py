"""CPU oracle for the MXAttention hot path (UOS-scaled MXFP4 quantization + PNQ attention forward).

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, float64 restatement of what the
paper defines; it exists to check the CUDA path and to serve as the timed CPU baseline.
Only ``tests/``, ``__graft_entry__.smoke()`` and ``bench.py``'s CPU-baseline / reference legs
may import it.  It shares no code with, and never imports, the CUDA package.

Modules
-------
``mxfp4``      E2M1 grid, E8M0 shared-scale rules (OCP floor rule, ceiling family, UOS), block
               quantizer (Section 2 "MXFP4 Block Quantization", Algorithm 1), canonical packing.
``nvfp4``      the comparison format of Section 5.2: 16-element blocks, E4M3 block scales, one fp32 tensor-level
               scale (the two-level recipe, every step in IEEE fp32: a reading, the paper only names the format).
``attention``  tiled online-softmax forward with direct or pre-normalization placement of the
               P-tilde quantizer (Section 2 recurrence, Eq. 12, Eq. 22, Algorithm 2), and the
               float64 dense softmax attention.
``rowsum``     the row-sum diagnostic of Section 5.3: quantize materialized probabilities, split the row-sum
               error into zeroing / saturation / downward / upward rounding, and the row entropy.
``uos_theory`` the quantization-error objective E, D, Delta, J of Section 4.1 / Appendices B-C,
               evaluated numerically; used to pin the 7.25 boundary independently of the quantizer.

Parity pins: every function here is pinned by ``tests/test_oracle_*.py`` against values the
paper prints, closed forms, exact rational brute force, or textbook special cases.  Not pinned
("parity unpinned"): nothing in these modules; the paper's model-level quality tables are not
reproduced at all (they need model weights and prompts).
"""
