"""TileMix hot path for NVIDIA B200 (sm_100a): blockwise INT8 quantiser, routing-mask packer
and the fused mixed-precision causal prefill attention kernel, behind a C-ABI library.

``paper_2608_17336_b200.binding`` is the thin ctypes layer over that library (it raises if
the library has not been built); ``paper_2608_17336_b200.synth`` holds the seeded synthetic
input generators and needs neither a GPU nor the library.
"""
