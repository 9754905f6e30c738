"""B200-native (sm_100a) selected-KV decode attention and full-context verification attention
for KAP / GraphSpec runtime access plans.

``paper_2607_24260_b200.kap`` is the thin binding over the C ABI declared in ``include/kap.h``
(argument marshalling only; every step runs in the library's own kernels / host C++);
``paper_2607_24260_b200.synth`` draws the seeded synthetic workloads.  Nothing is imported eagerly
so that the input generators can be used without loading the CUDA library.
"""
__all__ = ["kap", "synth", "build"]
