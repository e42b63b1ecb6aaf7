"""B200-native phase-owned MoE layer (route -> dispatch layout -> grouped SwiGLU FFN -> combine).

The compute lives in ``csrc/`` (CUDA for sm_100a behind a C ABI, ``include/moe_pd.h``);
``binding`` is argument marshalling only and raises if the built library is missing.
``workloads`` holds the seeded synthetic-input generators and imports nothing else from here.
"""
__all__ = ["binding", "workloads", "build"]
