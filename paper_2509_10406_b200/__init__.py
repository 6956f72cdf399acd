"""B200-native MuSe (Multipole Semantic Attention) layer: C-ABI CUDA library + thin binding.

Importing the package has no side effects; the CUDA library is loaded on first
use of `paper_2509_10406_b200.binding` and a missing library raises.
"""
