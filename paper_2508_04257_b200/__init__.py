"""KVSink quantized-KV-cache hot path for NVIDIA B200: Python binding over the C-ABI CUDA library."""
from .binding import (Config, KVCache, KvsinkError, SinkSet, StaticParams, calibrate, quantize_append_calibrated, decode_attention_calibrated, quantize_append_pertoken, decode_attention_pertoken, prefill_attention, cache_sizes, channel_absmax, quant_error, decode_attention, decode_attention_static, predict_sinks,  # noqa: F401
                      launch_count, quantize_append, read_status, strerror)
