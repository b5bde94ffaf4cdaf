"""FreqDepthKV hot path for one B200: prefill compression, routing probe and decode attention over the
depth-factorised KV cache, as hand-written sm_100a CUDA behind a C ABI (include/fdkv.h).

`synth` (seeded inputs) imports without the compiled library; `binding` loads libfdkv.so and raises if it is
missing -- there is no CPU fallback.
"""
