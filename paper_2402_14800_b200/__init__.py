"""Top-2 MoE layer forward with expert pruning and dynamic expert skipping, and
the layer-wise pruning search, as CUDA kernels for sm_100a behind a C ABI.

``synth`` (input generators) imports without the CUDA library; ``binding``
loads ``libmoe.so`` and fails loudly when it is missing.
"""
