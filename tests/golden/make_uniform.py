"""Writes uniform_attention_L16_w4.txt: the closed form of Eq. 1's window sum when every key is
identical, so that each causal softmax row is flat: query position t gives 1/(t+1) to each of keys
0..t, and A[i] = sum over window positions t >= i of 1/(t+1).  Exact rationals; no oracle, no GPU."""
from fractions import Fraction
import os

L, w = 16, 4
with open(os.path.join(os.path.dirname(__file__), "uniform_attention_L16_w4.txt"), "w") as f:
    f.write("# Eq. 1 (window sum of causal softmax rows), all keys equal, L=16, w=4: i  A[i]\n")
    for i in range(L):
        a = sum(Fraction(1, t + 1) for t in range(L - w, L) if t >= i)
        f.write("%d %s\n" % (i, a))
