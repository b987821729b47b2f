"""B200 (sm_100a) library for the branch-isolated attention step of ASPD's Hybrid Decoding Engine.

``binding`` wraps the C ABI declared in ``include/aspd.h``; ``workloads`` draws the seeded
synthetic inputs; ``build`` compiles the CUDA sources in-tree.  Importing the package loads
nothing; the first call into ``binding`` loads (and if needed builds) ``libaspd.so`` and raises
if that fails -- there is no CPU fallback.
"""
