"""B200-native masked-block denoising path for threshold-based diffusion-LLM decoding.

``binding`` exposes the C ABI of ``libd3.so`` (CUDA kernels for sm_100a); ``synth_inputs`` holds the
seeded synthetic model shapes, weights and prompts; ``build`` compiles the library in-tree.
Importing the package does not load the library; the first call does, and raises if it is missing.
"""
__all__ = ["binding", "synth_inputs", "build"]
