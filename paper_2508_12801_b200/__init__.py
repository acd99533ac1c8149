"""MaxScore router for B200: thin Python binding over the C-ABI CUDA library."""
