"""B200-native WUSH-KV serving hot path: quantize-on-append and decode attention over a packed
2/4-bit paged KV cache, as a C-ABI CUDA library (``libwushkv.so``) with a thin ctypes binding.

``paper_2609_38121_b200.binding`` loads the library and raises if it is missing;
``paper_2609_38121_b200.workloads`` only makes seeded synthetic inputs and needs no library.
"""
