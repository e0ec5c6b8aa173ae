"""Moonwalk gradient step for B200 (sm_100a): Python binding over the C-ABI library.

Importing the package loads nothing; `paper_2402_14212_b200.binding` loads the CUDA
library on first use and raises if it is missing (there is no CPU fallback).
"""
