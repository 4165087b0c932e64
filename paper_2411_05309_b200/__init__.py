"""GPU-thread-driven demand paging for oversubscribed memory on B200 (sm_100a).

``paper_2411_05309_b200.binding`` is the Python face of the C-ABI library
(``libgpuvm.so``, built from ``csrc/``); ``paper_2411_05309_b200.inputs`` holds the
seeded input generators.  Nothing is imported eagerly so that the generators can
be used on a machine without the CUDA library.
"""
__all__ = ["binding", "inputs"]
