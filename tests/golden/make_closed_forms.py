"""Writes closed_forms.json: values of the freshness score of Eq. 11,
f = exp(-alpha*sqrt(D_roll) - beta*sqrt(D_sup)) / (tau + 1), the ReLU gate of
Eq. 13 and the alignment ratio of Algorithm 1, evaluated with 50-digit decimal
arithmetic for hand-picked arguments.  The paper prints no numeric example, so
these closed-form evaluations stand in for one.  D_sup values are exactly
representable in fp32 because the interface takes them as fp32.  Calls neither the oracle nor
the CUDA library.  Run:  python tests/golden/make_closed_forms.py
"""
import json
import os
from decimal import Decimal, getcontext

getcontext().prec = 50

CASES = [
    # tau, D_roll, D_sup, alpha, beta, xi, cnt, H
    (3, "0.04", "0.0625", "1", "2", "0.05", 10, 20),
    (0, "0", "0", "1", "1", "0.15", 7, 7),
    (8, "0.0225", "0", "1", "1", "0.15", 100, 250),
    (2, "1.44", "0.25", "0.5", "0.25", "0.1", 3, 4),
    (5, "0.01", "0.000244140625", "1", "1", "0.15", 64, 64),
    (1, "0.36", "0.140625", "2", "3", "0", 9, 12),
]


def main():
    out = []
    for tau, dr, ds, a, b, xi, cnt, H in CASES:
        dr, ds, a, b, xi = map(Decimal, (dr, ds, a, b, xi))
        f = (-(a * dr.sqrt() + b * ds.sqrt())).exp() / Decimal(tau + 1)
        w = max(f - xi, Decimal(0))
        out.append(dict(tau=tau, D_roll=float(dr), D_sup=float(ds), alpha=float(a), beta=float(b),
                        xi=float(xi), cnt=cnt, H=H, f=float(f), w=float(w), m=cnt / H))
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "closed_forms.json")
    with open(path, "w") as fh:
        json.dump({"cite": "Eq. 11 (freshness), Eq. 13 (ReLU gate), Algorithm 1 (alignment ratio)",
                   "freshness": out}, fh, indent=1)


if __name__ == "__main__":
    main()
