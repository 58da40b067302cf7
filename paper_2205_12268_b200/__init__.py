"""B200-native forward pass of the Wavelet Compressed Convolution (WCC) layer.

``paper_2205_12268_b200.wcc`` is the thin binding over the C-ABI CUDA library
(loaded on first use); ``paper_2205_12268_b200.inputs`` builds the seeded
synthetic workloads.  Importing the package itself loads nothing.
"""
