"""Re-derives tests/golden/worked_example.json with exact rational arithmetic (fractions.Fraction).

This is the hand calculation of the fixture, mechanised: it imports neither the oracle nor the CUDA
library.  Every norm is an integer or a quarter-integer Pythagorean triple, so Algorithm 1's warm-up
branch (Eq. 2, min-seeding of gamma) and AdaGC branch (Eq. 3, EMA of the clipped norm) can be followed
without rounding.  Run it to print the table; the test suite checks that the stored fixture equals it.
"""
import json
import os
from fractions import Fraction as F
from math import isqrt


def exact_norm(vec):
    """Norm of a vector whose squared norm is a perfect square of a rational (Pythagorean triples)."""
    s = sum(F(x) * F(x) for x in vec)
    num, den = isqrt(s.numerator), isqrt(s.denominator)
    assert num * num == s.numerator and den * den == s.denominator, "not an exact norm"
    return F(num, den)


def derive():
    lam_abs, lam_rel, beta, warmup = F(13, 2), F(3, 2), F(1, 2), 2
    grads = [([3, 4], [0, 0, 12]), ([F(3, 4), 1], [0, 3, 4]), ([3, 4], [0, 6, 0]), ([3, 4], [0, 0, 0])]
    gamma = [None, None]
    rows = []
    for t, (ga, gb) in enumerate(grads, start=1):
        n = [exact_norm(ga), exact_norm(gb)]
        g2 = sum(F(x) * F(x) for x in list(ga) + list(gb))           # squared global norm
        if t <= warmup:
            clip = g2 > lam_abs * lam_abs
            if clip:
                G = exact_norm(list(ga) + list(gb))
                h = [lam_abs / G] * 2
            else:
                h = [F(1)] * 2
            c = [h[i] * n[i] for i in range(2)]
            gamma = c if t == 1 else [min(gamma[i], c[i]) for i in range(2)]
            flag = [int(clip)] * 2
        else:
            thr = [lam_rel * gamma[i] for i in range(2)]
            flag = [int(n[i] > thr[i]) for i in range(2)]
            h = [thr[i] / n[i] if flag[i] else F(1) for i in range(2)]
            c = [thr[i] if flag[i] else n[i] for i in range(2)]
            gamma = [beta * gamma[i] + (1 - beta) * c[i] for i in range(2)]
        rows.append(dict(t=t, norm=[float(x) for x in n], h=[float(x) for x in h], flag=flag,
                         gamma=[float(x) for x in gamma], global_norm_sq=float(g2)))
    return rows


if __name__ == "__main__":
    rows = derive()
    for r in rows:
        print(json.dumps(r))
    stored = json.load(open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "worked_example.json")))
    for r, s in zip(rows, stored["steps"]):
        assert r["norm"] == s["norm"] and r["h"] == s["h"] and r["flag"] == s["flag"] and r["gamma"] == s["gamma"], r
    print("stored fixture matches the exact derivation")
