"""B200-native eviction step of Lookahead Q-Cache (LAQ, Section 4.3): a thin Python binding over
the C-ABI library ``liblaq`` (hand-written sm_100a CUDA kernels). PyTorch is used only for device
memory and streams."""
__version__ = "0.1.0"
