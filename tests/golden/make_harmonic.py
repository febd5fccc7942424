"""Writes harmonic_scores_S12.txt: the aggregated causal attention scores for
all-equal logits (Eq. 1 with Q = 0), where every row i of the attention map is
uniform over its i+1 visible keys, so a_j = sum_{i=j}^{S-1} 1/(i+1) = H_S - H_j
(H_n the n-th harmonic number, H_0 = 0).  Exact rational arithmetic; no
implementation of the method is called."""
from fractions import Fraction
import os

S = 12
H = [Fraction(0)]
for n in range(1, S + 1):
    H.append(H[-1] + Fraction(1, n))
path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "harmonic_scores_S12.txt")
with open(path, "w") as f:
    f.write("# a_j = H_12 - H_j, j = 0..11 (Eq. 1 with uniform rows; column sums as in Algorithm 2 / Eq. 6)\n")
    for j in range(S):
        v = H[S] - H[j]
        f.write(f"{j} {v.numerator}/{v.denominator} {float(v):.17g}\n")
