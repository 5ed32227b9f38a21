"""GPU parity on randomly drawn shapes: every entry point against its fp64 oracle, through the C ABI,
on a seeded sequence of (operation, dtype, rows, cols, scale) draws. The fixed-shape parity tests pick
the sizes where the dispatcher changes kernels; this one covers the sizes nobody thought of. The bars
are the ones the per-operation tests state."""
import numpy as np
import pytest
import torch

import paper_2607_24762_b200 as fs
from oracle import fno, fso
from paper_2607_24762_b200 import workloads as W
from tests.gpu_util import np_to_torch_bits, torch_bits_to_np

pytestmark = pytest.mark.gpu
CASES_PER_SEED = 120


@pytest.fixture(scope="module", autouse=True)
def built_library():
    from paper_2607_24762_b200 import _build
    _build.build_library()
    yield
    assert fs.fs_device_status() == fs.FS_OK


def dev(a):
    return np_to_torch_bits(a).cuda()


def rand_cols(rng):
    k = rng.integers(0, 6)
    if k == 0:
        return int(rng.integers(1, 64))
    if k == 1:
        return int(rng.integers(1, 600)) * 8
    if k == 2:
        return int(rng.integers(1, 5000))
    if k == 3:
        return int(rng.integers(64, 4096)) * 8
    if k == 4:
        return int(rng.integers(4096, 40000)) * 8
    return int(2 ** rng.integers(3, 19))


def one_case(rng, S):
    """Draws one case, runs it, returns (ok, description)."""
    dtype = int(rng.integers(0, 3)); cols = rand_cols(rng)
    rows = int(max(1, min(rng.integers(1, 400), (1 << 22) // cols)))
    scale = float(rng.choice([1.0, 0.5, -1.0, 0.125, 2.0, 0.0, -0.3]))
    x = W.random_case(rows, cols, dtype, seed=int(rng.integers(1 << 30)), sigma=float(rng.choice([0.5, 2.0, 6.0])), neg_inf_frac=0.02 if scale > 0 else 0.0)
    op = int(rng.integers(0, 7))
    if op == 0:
        yd = torch.zeros_like(dev(x)); xd = dev(x)
        fs.fs_softmax(xd, yd, rows, cols, dtype, scale, S); torch.cuda.synchronize()
        ok = fso.compare(torch_bits_to_np(yd, dtype).reshape(rows, cols), dtype, fso.softmax_f64(x, dtype, scale)).ok(dtype); tag = 'softmax'
    elif op == 1:
        xd = dev(x); yd = torch.zeros_like(xd)
        fs.fs_log_softmax(xd, yd, rows, cols, dtype, scale, S); torch.cuda.synchronize()
        want = fso.log_softmax_f64(x, dtype, scale)
        ok = fno.compare(torch_bits_to_np(yd, dtype).reshape(rows, cols), dtype, want, fno.log_softmax_bound(want), rel_tol=1.0).ok(dtype, rel_tol=1.0); tag = 'log_softmax'
    elif op == 2:
        q = int(rng.integers(0, cols + 3)) - 2
        xd = dev(x); yd = torch.zeros_like(xd)
        fs.fs_softmax_causal(xd, yd, rows, cols, q, dtype, scale, S); torch.cuda.synchronize()
        ok = fso.compare(torch_bits_to_np(yd, dtype).reshape(rows, cols), dtype, fso.softmax_causal_f64(x, dtype, q, scale)).ok(dtype); tag = f'causal q={q}'
    elif op == 3:
        y = fso.round_from_f64(fso.softmax_f64(W.random_case(rows, cols, dtype, seed=3, sigma=2.0), dtype, 1.0), dtype)
        dy = fso.round_from_f64(rng.standard_normal((rows, cols)), dtype)
        gd, yd2 = dev(dy), dev(y); dd = torch.zeros_like(gd)
        fs.fs_softmax_backward(gd, yd2, dd, rows, cols, dtype, scale, S); torch.cuda.synchronize()
        es = fno.backward_error_scale(dy, y, dtype, scale)
        ok = fno.compare(torch_bits_to_np(dd, dtype).reshape(rows, cols), dtype, fso.softmax_backward_f64(dy, y, dtype, scale), es).ok(dtype); tag = 'backward'
    elif op == 4:
        xs = fso.round_from_f64(rng.standard_normal((rows, cols)) * rng.choice([0.5, 3.0]) + rng.choice([0.0, 5.0]), dtype)
        aff = int(rng.integers(0, 3))
        g = fso.round_from_f64(rng.standard_normal(cols) * 0.3 + 1, dtype) if aff >= 1 else None
        b = fso.round_from_f64(rng.standard_normal(cols) * 0.2, dtype) if aff == 2 else None
        xd = dev(xs); yd = torch.zeros_like(xd)
        fs.fs_layer_norm(xd, None if g is None else dev(g), None if b is None else dev(b), yd, rows, cols, dtype, 1e-5, S); torch.cuda.synchronize()
        scl = fno.error_scale(xs, dtype, xs.shape, None if g is None else fso.widen(g, dtype)[None, :], None if b is None else fso.widen(b, dtype)[None, :], 1e-5)
        ok = fno.compare(torch_bits_to_np(yd, dtype).reshape(rows, cols), dtype, fno.layer_norm_f64(xs, dtype, g, b, 1e-5), scl).ok(dtype); tag = f'layer_norm aff={aff}'
    elif op == 5:
        if dtype == 0:
            dtype = 1 + int(rng.integers(0, 2))
            x = W.random_case(rows, cols, dtype, seed=11, sigma=2.0)
        xd = dev(x); yd = torch.zeros((rows, cols), dtype=torch.float32, device='cuda')
        fs.fs_softmax_f32out(xd, yd, rows, cols, dtype, scale, S); torch.cuda.synchronize()
        ok = fso.compare(yd.cpu().numpy(), 0, fso.softmax_f64(x, dtype, scale)).ok(0); tag = 'f32out'
    else:
        heads = int(rng.choice([1, 2, 4])); q = max(1, rows // heads); rows2 = q * heads
        x2 = x[:rows2] if rows2 <= rows else np.tile(x, (heads, 1))[:rows2]
        x2 = np.ascontiguousarray(x2)
        m = np.where(rng.random((q, cols)) < 0.2, -np.inf, rng.standard_normal((q, cols)) * 0.5); m[:, 0] = 0.0
        m = fso.round_from_f64(m, dtype)
        xd, md = dev(x2), dev(m); yd = torch.zeros_like(xd)
        fs.fs_softmax_masked(xd, md, yd, rows2, cols, q, heads, dtype, scale, S); torch.cuda.synchronize()
        want = fso.softmax_masked_f64(x2, m, dtype, q, heads, scale)
        bound = fno.masked_softmax_bound(x2, m, dtype, q, heads, scale, want)
        ok = fno.compare(torch_bits_to_np(yd, dtype).reshape(rows2, cols), dtype, want, bound, rel_tol=1.0).ok(dtype, rel_tol=1.0); tag = f'masked h={heads}'
    return ok, f"{tag} dtype={dtype} rows={rows} cols={cols} scale={scale}"


@pytest.mark.parametrize("seed", [101, 202, 303])
def test_random_shapes_match_the_oracles(seed):
    rng = np.random.default_rng(seed)
    S = torch.cuda.current_stream()
    bad = []
    for _ in range(CASES_PER_SEED):
        ok, what = one_case(rng, S)
        if not ok:
            bad.append(what)
    assert not bad, bad
