"""libsdllm: B200-native cache refresh and sparse block attention for diffusion LLMs.

`paper_2508_02558_b200.binding` is the thin ctypes layer over the C-ABI library `libsdllm.so`
(hand-written CUDA for sm_100a); `paper_2508_02558_b200.workloads` draws the seeded synthetic inputs.
Nothing is imported eagerly so that the input generators stay usable without CUDA.
"""
__all__ = ["binding", "workloads", "build"]
