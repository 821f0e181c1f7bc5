"""B200-native SparQ decode attention: a C-ABI CUDA library plus this thin binding.

``from paper_2312_04985_b200 import sparq`` gives the binding (loads the shared library on
first use and raises if it is missing); ``synth`` draws the seeded synthetic workloads.
"""
__all__ = ["sparq", "synth"]
