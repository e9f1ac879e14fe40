"""MatQuant's nested int8 -> int4 -> int2 weight path as hand-written sm_100a CUDA kernels.

``binding`` wraps the C ABI of ``libmatq.so`` (declared in ``include/matq.h``);
``synth`` holds the seeded synthetic inputs; ``build`` compiles the library.
"""
__all__ = ["binding", "synth", "build", "shard"]
