"""B200-native LoQT quantized low-rank linear layer (arXiv 2405.16528).

The CUDA library is loaded on first use by `paper_2405_16528_b200.binding`;
importing the package itself touches no GPU.
"""
