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


GRADS_BINARY = [([3, 4], [0, 0, 12]), ([F(3, 4), 1], [0, 3, 4]), ([3, 4], [0, 6, 0]), ([3, 4], [0, 0, 0])]
# the second example differs at t = 2 only: decimal gradients (0.6, 0.8), still an exact norm (0.36 + 0.64 = 1)
GRADS_DECIMAL = [([3, 4], [0, 0, 12]), ([F(3, 5), F(4, 5)], [0, 3, 4]), ([3, 4], [0, 6, 0]), ([3, 4], [0, 0, 0])]


def derive(grads=None, exact=False):
    lam_abs, lam_rel, beta, warmup = F(13, 2), F(3, 2), F(1, 2), 2
    grads = GRADS_BINARY if grads is None else grads
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
        if exact:
            rows.append(dict(t=t, norm=n, h=h, flag=flag, gamma=list(gamma), g=(ga, gb)))
        else:
            rows.append(dict(t=t, norm=[float(x) for x in n], h=[float(x) for x in h], flag=flag,
                             gamma=[float(x) for x in gamma], global_norm_sq=float(g2)))
    return rows


def derive_theta(grads, theta0, lr="0.1", wd="0.1", beta1="0.9", beta2="0.999", eps="1e-8", digits=50):
    """theta after every step: the AdamW lines of Algorithm 1 on hat(g) = h g with the exact clip factors from derive(),
    in 50-digit decimal arithmetic (the square root is the only irrational operation)."""
    from decimal import Decimal as D, getcontext
    getcontext().prec = digits
    lr, wd, b1, b2, eps = D(lr), D(wd), D(beta1), D(beta2), D(eps)
    to_d = lambda x: D(F(x).numerator) / D(F(x).denominator)
    theta = [[D(str(x)) for x in ten] for ten in theta0]
    m = [[D(0)] * len(ten) for ten in theta0]
    v = [[D(0)] * len(ten) for ten in theta0]
    out = []
    for row in derive(grads, exact=True):
        t = row["t"]
        for i, g_i in enumerate(row["g"]):
            h = to_d(row["h"][i])
            for j, g in enumerate(g_i):
                gh = h * to_d(g)
                m[i][j] = b1 * m[i][j] + (1 - b1) * gh
                v[i][j] = b2 * v[i][j] + (1 - b2) * gh * gh
                m_hat, v_hat = m[i][j] / (1 - b1 ** t), v[i][j] / (1 - b2 ** t)
                theta[i][j] = theta[i][j] - lr * wd * theta[i][j] - lr * m_hat / (v_hat.sqrt() + eps)
        out.append([[float(x) for x in ten] for ten in theta])
    return out


if __name__ == "__main__":
    rows = derive()
    for r in rows:
        print(json.dumps(r))
    stored = json.load(open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "worked_example.json")))
    for r, s in zip(rows, stored["steps"]):
        assert r["norm"] == s["norm"] and r["h"] == s["h"] and r["flag"] == s["flag"] and r["gamma"] == s["gamma"], r
    print("stored fixture matches the exact derivation")
    second = json.load(open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "worked_example_decimal.json")))
    rows = derive(GRADS_DECIMAL)
    thetas = derive_theta(GRADS_DECIMAL, [second["theta0"]["A"], second["theta0"]["B"]])
    for r, th, sdict in zip(rows, thetas, second["steps"]):
        assert r["norm"] == sdict["norm"] and r["h"] == sdict["h"] and r["flag"] == sdict["flag"] and r["gamma"] == sdict["gamma"], r
        for got, want in zip(th, (sdict["theta_A"], sdict["theta_B"])):
            assert all(abs(a - b) <= 1e-9 for a, b in zip(got, want)), (r["t"], got, want)
    print("the printed values of the decimal example match the derivation to 1e-9")
