"""Writes tests/golden/uniform_T8.txt from exact rational arithmetic.

Under uniform causal attention (all logits equal) query j spreads 1/(j+1) over
keys 0..j, so Eq. 2 gives S_k = sum_{j=k}^{T-1} 1/(j+1) = H_T - H_k and Eq. 3
with the last w = 3 queries gives sum_{j=max(T-w,k)}^{T-1} 1/(j+1).  Nothing
here imports the oracle or the CUDA library; run `python make_golden.py`.
"""
import os
from fractions import Fraction

T, W = 8, 3
here = os.path.dirname(os.path.abspath(__file__))
with open(os.path.join(here, "uniform_T8.txt"), "w") as f:
    f.write("# uniform causal attention, T=8: k, Eq.2 S_k = H_8 - H_k, Eq.3 S_k with last w=3 queries (exact rationals)\n")
    for k in range(T):
        s2 = sum(Fraction(1, j + 1) for j in range(k, T))
        s3 = sum(Fraction(1, j + 1) for j in range(max(T - W, k), T))
        f.write(f"{k} {s2} {s3}\n")
