"""B200-native random-gossip BMUF synchronisation round (Algorithm 1 of "A Random Gossip BMUF
Process for Neural Language Modeling").

``paper_1909_09010_b200.binding`` is the thin ctypes layer over the C-ABI library
``libgbmuf.so`` (CUDA, sm_100a); ``paper_1909_09010_b200.workloads`` describes the synthetic
parameter sets.  There is no CPU or other fallback: if the CUDA library is missing, loading it
raises.
"""
