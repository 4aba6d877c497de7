"""Tree-verify hot path for online-compressed (CSA/HCA/window) attention on B200.

`synth` (seeded inputs) imports without a GPU.  The product path lives in
`binding` (ctypes over the C-ABI library built from `csrc/`); importing it raises
if the library has not been built -- there is no CPU fallback.
"""
__all__ = ["synth"]
