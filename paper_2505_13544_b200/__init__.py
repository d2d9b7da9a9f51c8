"""B200-native MTLA decode/prefill library: Python binding over the C-ABI in csrc/."""
