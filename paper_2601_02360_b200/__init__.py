"""SparseLoCo outer synchronisation step (paper §2.1, Eq. 2) for NVIDIA B200.

`paper_2601_02360_b200.api` is the thin binding over the C-ABI CUDA library (the outer step, the
12-bit wire form of the positions, the embedding re-projection of §2.4, the activation subspace
compression of §2.3);
`paper_2601_02360_b200.exchange` is the replica-per-GPU form of the step (torch.distributed);
`paper_2601_02360_b200.synth` draws the seeded synthetic inputs; `paper_2601_02360_b200.build`
compiles the library in-tree.  Nothing is imported eagerly, so `synth` can be used without the
CUDA library.
"""
__all__ = ["api", "exchange", "synth", "build"]
