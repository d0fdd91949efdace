"""B200-native KV-block swapping + paged decode attention (the hot path of Pie, arXiv 2411.09317).

``paper_2411_09317_b200.binding`` is the ctypes binding of the C-ABI library ``libpie.so``;
``paper_2411_09317_b200.synth`` is the seeded input generator.  Nothing is imported eagerly so that
the generator can be used without the CUDA library.
"""
__all__ = ["binding", "synth"]
