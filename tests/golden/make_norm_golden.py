"""Writes norm_mpmath.txt: fixed small inputs and their layer_norm / group_norm values evaluated
from the operators' definitions with mpmath at 60 digits, rounded once to fp64. The paper
(Sec. IV-C, Stable Diffusion 3.5 Medium results) names the two operators but prints no worked
example, so these values come from the definitions alone:
    mu = mean x,  var = mean (x - mu)^2,  y = (x - mu) / sqrt(var + eps) * gamma + beta
This script calls neither the oracle nor the CUDA library.

Line format:  kind | groups | n, channels, spatial | eps (C float, hex) | x | gamma or '-' | beta or '-' | y
(values as hex floats; layer_norm uses n = rows, channels = 1... see the reader in the pin test)
Run:  python tests/golden/make_norm_golden.py
"""
import os

import mpmath
import numpy as np

CASES = [
    # kind, groups, shape (n, channels, spatial), eps, x, gamma, beta
    ("layer", 1, (1, 1, 4), 1e-5, [0.0, 1.0, 2.0, 3.0], None, None),
    ("layer", 1, (2, 1, 5), 1e-5, [-1.5, 2.25, 0.0, -8.0, 3.0, 100.0, 100.5, 99.5, 100.25, 99.75],
     [1.0, 0.5, -2.0, 0.25, 3.0], [0.0, 1.0, -1.0, 0.5, 0.125]),
    ("layer", 1, (1, 1, 3), 1e-12, [1e-3, 2e-3, 4e-3], [2.0, 2.0, 2.0], None),
    ("layer", 1, (1, 1, 6), 0.5, [7.0, 7.0, 7.0, 7.0, 7.0, 7.0], [1.5, -1.5, 0.0, 2.0, 3.0, 4.0], [0.25, 0.5, 0.75, 1.0, 1.25, 1.5]),
    ("layer", 1, (1, 1, 2), 1e-5, [3.0e4, -3.0e4], None, [1.0, -1.0]),
    ("group", 2, (1, 4, 3), 1e-5, [0.5, -1.0, 2.0, 4.0, 0.0, -3.0, 1.0, 1.5, 2.5, -0.5, 0.25, 8.0],
     [1.0, 2.0, -1.0, 0.5], [0.0, 0.5, 1.0, -2.0]),
    ("group", 3, (2, 6, 2), 1e-3, [float(v) for v in np.linspace(-3.0, 4.0, 24) ** 3 / 7.0],
     [0.5, 1.0, 1.5, 2.0, 2.5, 3.0], [-1.0, -0.5, 0.0, 0.5, 1.0, 1.5]),
    ("group", 1, (1, 2, 4), 1e-5, [1.0, 2.0, 3.0, 4.0, 5.0, 6.0, 7.0, 9.0], None, None),
]


def main():
    mpmath.mp.dps = 60
    out = ["# kind | groups | n,channels,spatial | eps | x | gamma | beta | y   (written by make_norm_golden.py; mpmath, 60 digits; fp32 inputs)"]
    for kind, groups, (n, ch, sp), eps, x, gamma, beta in CASES:
        xs = np.array(x, dtype=np.float32).astype(np.float64)
        assert xs.size == n * ch * sp
        g = None if gamma is None else np.array(gamma, dtype=np.float32).astype(np.float64)
        b = None if beta is None else np.array(beta, dtype=np.float32).astype(np.float64)
        e32 = float(np.float32(eps))
        ys = []
        if kind == "layer":
            rows, cols = n, sp
            assert ch == 1
            for r in range(rows):
                row = [mpmath.mpf(float(v)) for v in xs[r * cols:(r + 1) * cols]]
                mu = sum(row) / cols
                var = sum((v - mu) ** 2 for v in row) / cols
                rstd = 1 / mpmath.sqrt(var + mpmath.mpf(e32))
                for j, v in enumerate(row):
                    y = (v - mu) * rstd
                    if g is not None:
                        y *= mpmath.mpf(float(g[j]))
                    if b is not None:
                        y += mpmath.mpf(float(b[j]))
                    ys.append(float(y))
        else:
            cpg = ch // groups
            ys = [0.0] * xs.size
            for s in range(n):
                for gi in range(groups):
                    idx = [(s * ch + c) * sp + k for c in range(gi * cpg, (gi + 1) * cpg) for k in range(sp)]
                    vals = [mpmath.mpf(float(xs[i])) for i in idx]
                    mu = sum(vals) / len(vals)
                    var = sum((v - mu) ** 2 for v in vals) / len(vals)
                    rstd = 1 / mpmath.sqrt(var + mpmath.mpf(e32))
                    for i, v in zip(idx, vals):
                        c = (i // sp) % ch
                        y = (v - mu) * rstd
                        if g is not None:
                            y *= mpmath.mpf(float(g[c]))
                        if b is not None:
                            y += mpmath.mpf(float(b[c]))
                        ys[i] = float(y)
        hx = lambda a: " ".join(float(v).hex() for v in a)
        out.append(" | ".join([kind, str(groups), f"{n},{ch},{sp}", e32.hex(), hx(xs), "-" if g is None else hx(g),
                               "-" if b is None else hx(b), hx(ys)]))
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "norm_mpmath.txt")
    with open(path, "w") as f:
        f.write("\n".join(out) + "\n")
    print("wrote", path, len(out) - 1, "cases")


if __name__ == "__main__":
    main()
