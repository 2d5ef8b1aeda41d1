"""Rewrites the derived fixtures in this folder from first principles.

Uses only the Python standard library: no project code, no oracle, no CUDA path.
"""
import os
from decimal import Decimal, getcontext

HERE = os.path.dirname(os.path.abspath(__file__))


def trinomial_rows(kmax):
    rows, poly = [], [1]
    for _ in range(kmax):
        nxt = [0] * (len(poly) + 2)
        for i, a in enumerate(poly):
            for s in range(3):
                nxt[i + s] += a
        poly = nxt
        rows.append(poly)
    return rows


def path3():
    getcontext().prec = 40
    x = [Decimal(1), Decimal(2), Decimal(3)]
    dt = [Decimal(2), Decimal(3), Decimal(2)]  # D~ = D + 1 on the path 0-1-2
    adj = {0: [0, 1], 1: [0, 1, 2], 2: [1, 2]}  # support of A~
    gcn = [sum(x[j] / (dt[i].sqrt() * dt[j].sqrt()) for j in adj[i]) for i in range(3)]
    nb = {0: [1], 1: [0, 2], 2: [1]}
    sage = [sum(x[j] for j in nb[i]) / len(nb[i]) for i in range(3)]
    eps = Decimal("0.1")
    gin = [sum(x[j] for j in nb[i]) + (1 + eps) * x[i] for i in range(3)]
    return gcn, sage, gin


if __name__ == "__main__":
    with open(os.path.join(HERE, "trinomial.txt"), "w") as f:
        f.write("# row k: coefficients of (1 + x + x^2)^k, k = 1..5\n")
        for r in trinomial_rows(5):
            f.write(" ".join(str(v) for v in r) + "\n")
    gcn, sage, gin = path3()
    with open(os.path.join(HERE, "path3_worked.txt"), "w") as f:
        f.write("# path 0-1-2, x = (1, 2, 3); one hop of each operator (GIN eps = 0.1)\n")
        for name, v in (("gcn", gcn), ("sage", sage), ("gin", gin)):
            f.write(name + " " + " ".join(f"{t:.18f}" for t in v) + "\n")
