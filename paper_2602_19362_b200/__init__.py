"""B200-native OAPL LM-head hot path: fused log-prob pass, Eq. 2 / Eq. 3 and
their backward, as a C-ABI CUDA library with a thin ctypes binding.

`paper_2602_19362_b200.binding` loads the compiled library on first use and
raises if it is missing; there is no CPU fallback.  `synth` builds seeded
synthetic batches and needs only torch.
"""
__all__ = ["binding", "synth", "build"]
