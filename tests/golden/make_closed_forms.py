"""Writes closed_forms.json from the formulas printed in the paper (no oracle, no GPU).

Section 2.3, Example 2: P[coordinate empty] = (1 - K/N)^M.
Section 3.2, Lemma 3:   P[M_n = u] = C(M, u) gamma^u (1 - gamma)^(M - u).
Section 3.2, Theorem 1: alpha(M, gamma) = 1 - (1 - gamma)^M.
"""
import json
import os
from fractions import Fraction
from math import comb

CASES = [  # (N, K, M)
    (65536, 655, 5),
    (4096, 256, 8),
    (200000, 2000, 16),
]

out = {"citation": "Section 2.3 Example 2; Section 3.2 Lemma 3 and Theorem 1", "cases": []}
for N, K, M in CASES:
    g = Fraction(K, N)
    pmf = [float(comb(M, u) * g**u * (1 - g) ** (M - u)) for u in range(M + 1)]
    out["cases"].append({"N": N, "K": K, "M": M, "p_empty": float((1 - g) ** M),
                         "alpha": float(1 - (1 - g) ** M), "voter_count_pmf": pmf})
with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "closed_forms.json"), "w") as f:
    json.dump(out, f, indent=1)
    f.write("\n")
