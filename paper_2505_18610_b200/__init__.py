"""B200-native PM-KVQ decode hot path: quantize-on-append, progressive bit-width reduction
and fused dequantize + GQA decode attention over a packed mixed-precision KV cache.

The compute lives in a C-ABI CUDA library (``csrc/``, built in-tree as ``libpmkvq.so``);
``binding`` is a thin ctypes layer with the same call names.
"""
