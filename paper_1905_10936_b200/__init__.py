"""B200-native hot path of dist-EF-blockSGDM (Algorithm 4 of arXiv 1905.10936).

``binding`` mirrors the C ABI of ``include/ef.h`` one to one; ``engine.EFEngine`` owns the
torch workspace around a context; ``workloads`` holds the benchmark layouts and the seeded
synthetic gradients.  Nothing is imported eagerly so that ``workloads`` can be used on a
machine without the compiled library.
"""
__all__ = ["binding", "engine", "workloads", "build"]
