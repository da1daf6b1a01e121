"""B200-native convolution merging and merged-network inference (arXiv 2301.12187 hot path).

`paper_2301_12187_b200.dc`      ctypes binding of the C-ABI CUDA library (fails loudly if it is missing)
`paper_2301_12187_b200.inputs`  seeded synthetic inputs (data only; no method arithmetic)
"""
