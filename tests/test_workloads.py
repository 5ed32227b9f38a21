"""The seeded input generators: shapes, dtypes, moments, structure and block-wise reproducibility.
These inputs stand in for the operator captures of the paper's Table I workloads. CPU only."""
import numpy as np
import pytest

from paper_2607_24762_b200 import workloads as W


def test_shapes_and_min_bytes():
    expect = {"cfg1": (64, 1000, 512_000), "cfg2": (16384, 2048, 134_217_728),
              "cfg3": (131072, 128, 67_108_864), "cfg4": (256, 262144, 268_435_456),
              "cfg5": (32768, 32768, 8_589_934_592)}
    for name, (rows, cols, nbytes) in expect.items():
        w = W.WORKLOADS[name]
        assert (w.rows, w.cols, w.min_bytes) == (rows, cols, nbytes)
    assert abs(W.WORKLOADS["cfg2"].scale_f32 - 128 ** -0.5) < 1e-8


@pytest.mark.parametrize("name,r0,r1", [("cfg1", 0, 64), ("cfg2", 500, 1030), ("cfg3", 8000, 16500),
                                        ("cfg4", 3, 9), ("cfg5", 31, 66)])
def test_any_row_range_reproduces_the_same_rows(name, r0, r1):
    w = W.WORKLOADS[name]
    a = W.generate_rows(w, r0, r1)
    b = W.generate_rows(w, r0, r1, threads=4)
    assert a.dtype == W.NP_STORE[w.dtype] and a.shape == (r1 - r0, w.cols)
    assert np.array_equal(a.view(np.uint8), b.view(np.uint8))
    mid = (r0 + r1) // 2
    c = W.generate_rows(w, mid, mid + 1)
    assert np.array_equal(c.view(np.uint8), a[mid - r0:mid - r0 + 1].view(np.uint8))
    assert W.checksum(a) == W.checksum(b) != W.checksum(a[::-1])


def test_moments():
    x = W.generate(W.WORKLOADS["cfg1"]).astype(np.float64)
    n = x.size
    assert abs(x.mean()) < 4 / np.sqrt(n) and abs(x.var() - 1) < 4 * np.sqrt(2 / n)
    w = W.WORKLOADS["cfg2"]
    x = W.stored_to_f32(W.generate_rows(w, 0, 1024), w.dtype).astype(np.float64)
    n = x.size
    assert abs(x.mean()) < 4 * 3 / np.sqrt(n) and abs(x.var() / 9 - 1) < 0.01
    w = W.WORKLOADS["cfg3"]
    x = W.stored_to_f32(W.generate_rows(w, 0, 16384), w.dtype).astype(np.float64)
    row_mean = x.mean(axis=1)
    # row means carry the bias: variance 0.25 + 1/128
    assert abs(row_mean.var() - (0.25 + 1 / 128)) < 0.02
    assert abs((x - row_mean[:, None]).var() - 1) < 0.02


def test_vocabulary_spikes():
    w = W.WORKLOADS["cfg4"]
    x = W.stored_to_f32(W.generate_rows(w, 8, 12), w.dtype)
    for r in range(4):
        assert np.count_nonzero(x[r] == 30.0) == 8
        rest = x[r][x[r] != 30.0].astype(np.float64)
        assert abs(rest.var() / 16 - 1) < 0.02 and rest.max() < 30.0


def test_causal_mask():
    w = W.WORKLOADS["cfg5"]
    x = W.generate_rows(w, 100, 104)
    for k, i in enumerate(range(100, 104)):
        assert np.all(np.isneginf(x[k, i + 1:])) and np.all(np.isfinite(x[k, :i + 1]))
    x = W.generate_rows(w, w.rows - 1, w.rows)
    assert np.all(np.isfinite(x)) and abs(x.astype(np.float64).var() / 4 - 1) < 0.05


def test_bf16_rounding_is_single_rounding():
    # 1 + 2^-8 + 2^-40 lies just above the midpoint of two bf16 neighbours: must round up, although
    # narrowing to fp32 first (nearest-even) would land on the midpoint and then tie to even (down).
    v = np.array([1.0 + 2.0 ** -8 + 2.0 ** -40, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8])
    assert list(W.f64_to_bf16_bits(v)) == [0x3F81, 0x3F80, 0x3F82]
    assert list(W.f32_to_bf16_bits(v.astype(np.float32))) == [0x3F80, 0x3F80, 0x3F82]
    assert list(W.bf16_bits_to_f32(np.array([0x3F80, 0xC000], dtype=np.uint16))) == [1.0, -2.0]


def test_streaming_checksum_equals_the_whole_buffer_checksum():
    """Checksum taken slab by slab (what the benchmark records for the 4 GiB workload) is the checksum of the whole."""
    w = W.WORKLOADS["cfg2"]
    x = W.generate_rows(w, 0, 700)
    whole = W.checksum(x)
    for slab in (1, 128, 699, 700):
        c = W.Checksum()
        for r0 in range(0, 700, slab):
            c.update(x[r0:r0 + slab], threads=1 if slab == 1 else 4)
        assert c.value() == whole
    y = x.copy()
    y[350, 7] ^= 1
    assert W.Checksum().update(y).value() != whole
    a, b = x[:300].copy(), x[300:].copy()
    assert W.Checksum().update(b).update(a).value() != whole          # order-sensitive
