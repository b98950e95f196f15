"""B200-native NVFP4 MoE rollout forward (online activation quantize, top-k
routing, grouped W4A4 expert GEMMs with SwiGLU, Residual Activation
Compensation) and the trainer-side weight fake-quant, behind a C-ABI library.

`paper_2607_15810_b200.binding` is the thin ctypes layer over libquads.so (it
raises at import when the library has not been built); `synth` draws the
seeded synthetic inputs and needs no GPU."""
__all__ = ["synth"]
