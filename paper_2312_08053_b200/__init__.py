"""B200-native worker-side compression pass of Kimad+ (EF21 difference, Top-K error curves,
knapsack DP, Top-K select, sparse pack, EF21 update) behind a C ABI.

``binding`` is the ctypes front end of the CUDA library; ``workloads`` produces synthetic inputs.
Nothing is imported eagerly so that input generation works without the compiled library.
"""
__all__ = ["binding", "workloads", "build"]
