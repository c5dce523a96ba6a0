"""R-TOSS hot path for NVIDIA B200 (sm_100a): pattern selection, packing and
pattern-sparse 3x3 / 1x1 inference convolution behind a C-ABI library
(``librtoss.so``, declared in ``include/rtoss.h``) with a thin ctypes binding.

``import paper_2303_02191_b200.binding`` loads the CUDA library and raises if
it is missing: there is no CPU fallback.  ``synth`` holds the seeded synthetic
inputs and the layer-shape tables and needs no GPU.
"""
__all__ = ["synth"]
