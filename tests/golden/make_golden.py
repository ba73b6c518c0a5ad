"""Writes the text fixtures in this folder.  Independent of the CUDA path and of the oracle:
closed forms evaluated with 50-digit arithmetic (mpmath).

rope_delta1000_d8_theta1e6.txt -- the paper's worked example (Rotary Positional Embeddings
section): a key cached at position 50 and reused at position 1050 needs the correction
R_theta^{1000}.  For head_dim 8 and base 1e6 the four plane angles are 1000 * 1e6^(-2j/8);
each line holds angle, cos, sin.
"""
import os

import mpmath as mp

mp.mp.dps = 50
here = os.path.dirname(os.path.abspath(__file__))
with open(os.path.join(here, "rope_delta1000_d8_theta1e6.txt"), "w") as f:
    f.write("# Rotary Positional Embeddings, worked example t=50 -> t=1050: angle cos sin per plane j (d=8, theta=1e6)\n")
    for j in range(4):
        a = mp.mpf(1000) * mp.power(mp.mpf(10) ** 6, -mp.mpf(2 * j) / 8)
        f.write("%s %s %s\n" % (mp.nstr(a, 25), mp.nstr(mp.cos(a), 25), mp.nstr(mp.sin(a), 25)))
