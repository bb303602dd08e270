"""B200-native hot path of FVAttn's adaptive sparse attention for video DiTs.

reorder -> route (Top-p with a Top-k floor) -> block-sparse attention -> inverse reorder,
hand-written CUDA for sm_100a behind the C-ABI library ``libfvattn.so``.  ``binding`` is the
ctypes front end (argument marshalling only); ``synth`` draws the seeded synthetic inputs.
There is no CPU fallback: using the ops without the built library raises.
"""
__all__ = ["binding", "synth", "build"]
