"""AdaComp residual gradient compression for one B200: compress / decompress-accumulate.

The CUDA library is loaded on first use of `paper_1712_02679_b200.binding`;
importing this package (or `synth`) needs neither a GPU nor the built library.
"""
__all__ = ["synth"]
