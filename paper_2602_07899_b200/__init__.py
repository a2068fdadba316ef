"""B200-native hot path of TLQ's layer-wise scale search (hand-written sm_100a CUDA behind a C ABI).

`workloads` (seeded synthetic inputs) imports without the CUDA library; the binding in `tlq`
loads `libtlq.so` on first use and raises if it is missing (there is no CPU fallback).
"""
