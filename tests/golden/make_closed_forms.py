"""Writes closed_forms.txt: entropies of two-level logit vectors from their closed form, evaluated
with 50-digit arithmetic (mpmath).  Calls neither the oracle nor the CUDA library."""
import os

import mpmath as mp

HEADER = """\
# Closed-form entropy values (nats) that pin the oracle's softmax statistics (paper section 3.4.1:
# the confidence metric is the entropy of the predicted distribution over the vocabulary).
# name ; V ; n_high ; a ; entropy ; max_prob     (n_high logits equal to a >= 0, the other V - n_high equal to 0)
# entropy = ln(Z) - a*n*e^a/Z with Z = n*e^a + V - n ; max_prob = e^a / Z.  The first row is ln(50304).
# Written by make_closed_forms.py with 50-digit decimal arithmetic.
"""
ROWS = [("uniform_pythia", 50304, 0, 0), ("one_hot_a10", 50304, 1, 10), ("one_hot_a40", 50304, 1, 40),
        ("two_level_n3_a12", 50304, 3, 12), ("two_level_n100_a5", 50304, 100, 5),
        ("tiny_v2_a1", 2, 1, 1), ("tiny_v5_n2_a3", 5, 2, 3)]

if __name__ == "__main__":
    mp.mp.dps = 50
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "closed_forms.txt")
    with open(path, "w") as f:
        f.write(HEADER)
        for name, V, n, a in ROWS:
            Z = n * mp.e ** a + (V - n)
            H = mp.log(Z) - a * n * mp.e ** a / Z
            p = mp.e ** a / Z
            f.write(f"{name} ; {V} ; {n} ; {a} ; {mp.nstr(H, 17)} ; {mp.nstr(p, 17)}\n")
