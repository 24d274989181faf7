"""KVSink quantized-KV-cache hot path for NVIDIA B200: Python binding over the C-ABI CUDA library."""
