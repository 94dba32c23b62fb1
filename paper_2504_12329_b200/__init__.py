"""B200-native Speculative Thinking decode: thin Python binding over the C-ABI CUDA library."""
