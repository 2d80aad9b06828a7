"""B200-native hot path of ScaleBITS' bitwidth search (arxiv 2602.17698).

`binding` holds the thin ctypes layer over the C-ABI CUDA library, `pipeline`
sequences its calls for a Llama-shaped decoder layer, `synth` draws the seeded
synthetic inputs.  Importing the package does not load the CUDA library; the
first use of `binding.lib()` does, and fails loudly if it is missing.
"""
__all__ = ["binding", "pipeline", "synth", "build"]
