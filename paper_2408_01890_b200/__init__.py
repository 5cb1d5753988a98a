"""LiSA shared-layer attention forward for B200 (sm_100a): Python binding of the C-ABI library.

The CUDA library is loaded on first use (`paper_2408_01890_b200.binding`); the
input generators in `paper_2408_01890_b200.synth` need no GPU.
"""
