"""B200-native forward pass of an MoE layer with zero-output experts (ZEDA, Section 2.1, Eq. 1).

``paper_2605_18643_b200.zeda``   - Python binding over the C-ABI CUDA library (loads the .so, fails
                                   loudly if it is missing).
``paper_2605_18643_b200.inputs`` - seeded synthetic workloads (no layer arithmetic).
``paper_2605_18643_b200.flops``  - the paper's FLOP model (Appendix D) and the roofline bounds.
"""
