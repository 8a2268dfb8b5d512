"""SparseLoCo outer synchronisation step (paper §2.1, Eq. 2) for NVIDIA B200.

`paper_2601_02360_b200.api` is the thin binding over the C-ABI CUDA library;
`paper_2601_02360_b200.synth` draws the seeded synthetic parameter sets.
Nothing is imported eagerly, so `synth` can be used without the CUDA library.
"""
__all__ = ["api", "synth", "build"]
