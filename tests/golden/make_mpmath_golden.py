"""Writes softmax_mpmath.txt: fixed input rows and their softmax evaluated from the definition
y_j = exp(z_j - max z) / sum_k exp(z_k - max z), z = scale * x, with mpmath at 100 digits and
rounded once to fp64. The paper (abstract, Sec. IV-C) names the operator but prints no worked
example, so these values come from the definition alone. This script calls neither the oracle
nor the CUDA library.

Line format:  dtype | scale (C float, hex) | inputs (hex floats, exact in dtype) | outputs (hex fp64)
Run:  python tests/golden/make_mpmath_golden.py
"""
import os

import mpmath
import numpy as np

ROWS = [
    ("fp32", 1.0, [0.0, 1.0, 2.0, 3.0]),
    ("fp32", 1.0, [-1.5, 2.25, 0.0, -8.0, 3.0, 3.0, 0.125]),
    ("fp32", 0.5, [10.0, -10.0, 0.0, 4.0, 4.5]),
    ("fp32", -1.0, [1.0, 2.0, 3.0, -4.0]),
    ("fp32", 1.0, [float("-inf"), 0.0, 1.0, float("-inf"), -1.0]),
    ("fp32", 1.0, [88.0, 87.0, -88.0, 0.0]),
    ("fp32", float(np.float32(1.0 / np.sqrt(128.0))), [12.0, -7.0, 3.5, 0.0, 9.25, -15.0, 1.0, 2.0]),
    ("fp32", 1.0, [3.0e38, 2.9e38, -3.0e38]),
    ("bf16", 1.0, [0.5, 1.0, -2.0, 3.0, 30.0, 30.0]),
    ("bf16", float(np.float32(1.0 / np.sqrt(128.0))), [9.0, -3.0, 0.75, 6.0, -12.0]),
    ("bf16", 1.0, [float("-inf"), -0.25, 0.25]),
    ("fp16", 1.0, [65504.0, 65472.0, 0.0, -65504.0]),
    ("fp16", 0.25, [1.0, 2.0, 3.0, 4.0, 5.0, 6.0, 7.0, 8.0, 9.0]),
    ("fp16", 1.0, [6.103515625e-05, 5.9604644775390625e-08, 0.0]),
]


def to_dtype(v, dtype):
    a = np.array(v, dtype=np.float64)
    if dtype == "fp32":
        return a.astype(np.float32).astype(np.float64)
    if dtype == "fp16":
        return a.astype(np.float16).astype(np.float64)
    import ml_dtypes
    return a.astype(np.float32).astype(ml_dtypes.bfloat16).astype(np.float64)


def main():
    out = ["# dtype | scale | inputs | outputs   (written by make_mpmath_golden.py; mpmath, 100 digits)"]
    mpmath.mp.dps = 100
    for dtype, scale, row in ROWS:
        xs = to_dtype(row, dtype)
        s32 = float(np.float32(scale))
        z = [mpmath.mpf(s32) * mpmath.mpf(float(v)) if np.isfinite(v) else None for v in xs]
        m = max(v for v in z if v is not None)
        e = [mpmath.exp(v - m) if v is not None else mpmath.mpf(0) for v in z]
        total = mpmath.fsum(e)
        ys = [float(v / total) for v in e]
        out.append(" | ".join([dtype, float(s32).hex(),
                               " ".join(float(v).hex() for v in xs),
                               " ".join(float(v).hex() for v in ys)]))
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "softmax_mpmath.txt")
    with open(path, "w") as f:
        f.write("\n".join(out) + "\n")


if __name__ == "__main__":
    main()
