"""The library only enqueues work: its launches can be captured into a CUDA graph (after a first
call outside the capture, which does the per-device set-up) and replayed, and calls on different
streams can overlap. Results are checked against the oracle."""
import numpy as np
import pytest
import torch

import paper_2607_24762_b200 as fs
from paper_2607_24762_b200 import workloads as W

from gpu_util import check, np_to_torch_bits, torch_bits_to_np

pytestmark = pytest.mark.gpu

CASES = [(W.BF16, 512, 128, 1.0), (W.BF16, 300, 2048, 0.25), (W.FP32, 64, 8192, 1.0), (W.FP16, 40, 65536, 0.5),
         (W.FP32, 37, 1001, 1.0)]


def test_capture_into_a_cuda_graph_and_replay():
    xs, ys, hosts = [], [], []
    for dtype, rows, cols, scale in CASES:
        x = W.random_case(rows, cols, dtype, seed=rows, sigma=2.0, neg_inf_frac=0.02)
        hosts.append(x)
        xs.append(np_to_torch_bits(x).cuda())
        ys.append(torch.zeros_like(xs[-1]))
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for (dtype, rows, cols, scale), xd, yd in zip(CASES, xs, ys):        # set-up outside the capture
            fs.fs_softmax(xd, yd, rows, cols, dtype, scale, side)
        fs.fs_softmax_causal(xs[1], ys[1], CASES[1][1], CASES[1][2], 5, CASES[1][0], CASES[1][3], side)
    side.synchronize()
    for yd in ys:
        yd.zero_()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for (dtype, rows, cols, scale), xd, yd in zip(CASES, xs, ys):
            fs.fs_softmax(xd, yd, rows, cols, dtype, scale, torch.cuda.current_stream())
    torch.cuda.synchronize()
    assert all(int(yd.view(torch.uint8).max()) == 0 for yd in ys)            # capture ran nothing
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    assert fs.fs_device_status() == fs.FS_OK
    for (dtype, rows, cols, scale), x, yd in zip(CASES, hosts, ys):
        check(x, dtype, scale, torch_bits_to_np(yd, dtype))


def test_calls_on_two_streams_overlap_safely():
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    w = W.WORKLOADS["cfg2"]
    x = W.generate_rows(w, 0, 4096)
    xd = np_to_torch_bits(x).cuda()
    outs = [torch.empty_like(xd) for _ in range(8)]
    torch.cuda.synchronize()
    for i, yd in enumerate(outs):
        fs.fs_softmax(xd, yd, 4096, w.cols, w.dtype, w.scale_f32, s1 if i % 2 == 0 else s2)
    torch.cuda.synchronize()
    ref = torch_bits_to_np(outs[0], w.dtype)
    check(x, w.dtype, w.scale_f32, ref)
    for yd in outs[1:]:
        assert np.array_equal(torch_bits_to_np(yd, w.dtype), ref)


def test_added_entry_points_capture_and_replay():
    """log_softmax, backward, masked softmax and layer_norm only enqueue kernels too."""
    from oracle import fno, fso
    rows, cols, dtype = 96, 8192, W.BF16
    x = W.random_case(rows, cols, dtype, seed=5, sigma=2.0)
    gamma = fso.round_from_f64(np.random.default_rng(1).standard_normal(cols) * 0.2 + 1, dtype)
    mask = fso.round_from_f64(np.where(np.arange(cols)[None, :] > np.arange(rows)[:, None] + cols - rows, -np.inf, 0.0), dtype)
    xd, gd, md = np_to_torch_bits(x).cuda(), np_to_torch_bits(gamma).cuda(), np_to_torch_bits(mask).cuda()
    y = [torch.zeros_like(xd) for _ in range(5)]
    side = torch.cuda.Stream()

    def enqueue(s):
        fs.fs_softmax(xd, y[0], rows, cols, dtype, 1.0, s)
        fs.fs_log_softmax(xd, y[1], rows, cols, dtype, 0.5, s)
        fs.fs_softmax_masked(xd, md, y[2], rows, cols, rows, 1, dtype, 0.25, s)
        fs.fs_layer_norm(xd, gd, None, y[3], rows, cols, dtype, 1e-5, s)
        fs.fs_softmax_backward(xd, y[0], y[4], rows, cols, dtype, 1.0, s)          # dy = x, y = the softmax above

    with torch.cuda.stream(side):
        enqueue(side)                                        # set-up outside the capture
    side.synchronize()
    for t in y:
        t.zero_()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        enqueue(torch.cuda.current_stream())
    torch.cuda.synchronize()
    assert all(int(t.view(torch.uint8).max()) == 0 for t in y)
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert fs.fs_device_status() == fs.FS_OK
    got = [torch_bits_to_np(t, dtype) for t in y]
    check(x, dtype, 1.0, got[0])
    want = fso.log_softmax_f64(x, dtype, 0.5)
    assert fno.compare(got[1], dtype, want, np.maximum(1.0, np.abs(want)), rel_tol=1e-6).ok(dtype, rel_tol=1e-6)
    want = fso.softmax_masked_f64(x, mask, dtype, rows, 1, 0.25)
    assert fno.compare(got[2], dtype, want, 1e-6 + 1e-5 * want, rel_tol=1.0).ok(dtype, rel_tol=1.0)
    want = fno.layer_norm_f64(x, dtype, gamma, None, 1e-5)
    assert fno.compare(got[3], dtype, want, fno.error_scale(x, dtype, x.shape, fso.widen(gamma, dtype)[None, :], None, 1e-5)).ok(dtype)
    want = fso.softmax_backward_f64(x, got[0], dtype, 1.0)
    g64, y64 = fso.widen(x, dtype), fso.widen(got[0], dtype)
    es = np.abs(y64) * (np.abs(g64) + np.abs(g64 * y64).sum(axis=1, keepdims=True))
    assert fno.compare(got[4], dtype, want, es).ok(dtype)


def test_two_kernel_paths_on_two_streams_do_not_share_scratch():
    """Rows beyond a cluster's shared memory exchange partial results through a buffer allocated in stream
    order per call: concurrent calls on different streams cannot see each other's."""
    from oracle import fno
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    cols = (1 << 20) + 16
    xs = [W.random_case(2, cols, W.FP32, seed=40 + i, sigma=2.0) for i in range(4)]
    xd = [np_to_torch_bits(x).cuda() for x in xs]
    yd = [torch.empty_like(t) for t in xd]
    nd = [torch.empty_like(t) for t in xd]
    torch.cuda.synchronize()
    for rep in range(3):
        for i in range(4):
            s = s1 if i % 2 == 0 else s2
            fs.fs_softmax(xd[i], yd[i], 2, cols, W.FP32, 1.0, s)
            fs.fs_layer_norm(xd[i], None, None, nd[i], 2, cols, W.FP32, 1e-5, s)
    torch.cuda.synchronize()
    assert fs.fs_device_status() == fs.FS_OK
    for i in range(4):
        check(xs[i], W.FP32, 1.0, torch_bits_to_np(yd[i], W.FP32))
        rep = fno.compare(torch_bits_to_np(nd[i], W.FP32), W.FP32, fno.layer_norm_f64(xs[i], W.FP32), fno.error_scale(xs[i], W.FP32, xs[i].shape))
        assert rep.ok(W.FP32), rep


def test_a_launch_reads_what_the_previous_launch_of_the_stream_wrote():
    """Kernels start under programmatic dependent launch while the previous kernel of the stream drains, and the
    long-row kernels ask L2 for their input before they wait for it. The input of each launch here IS the output
    of the launch before it, written into a buffer that held NaN until then: a chain run back to back must give,
    bit for bit, what the same launches give with a synchronisation between them."""
    cases = [(W.BF16, 256, 262144), (W.BF16, 2048, 32768), (W.FP32, 4096, 8192), (W.BF16, 16384, 2048), (W.FP32, 300, 50000),
             (W.BF16, 16384, 5120)]
    s = torch.cuda.current_stream()
    for dtype, rows, cols in cases:
        x = np_to_torch_bits(W.random_case(rows, cols, dtype, seed=rows + cols, sigma=3.0)).cuda()
        bufs = [torch.empty_like(x) for _ in range(4)]
        want = []
        src = x
        for b in bufs:                                                       # one at a time
            fs.fs_softmax(src, b, rows, cols, dtype, 4.0, s)
            torch.cuda.synchronize()
            want.append(b.clone())
            src = b
        for rep in range(3):
            for b in bufs:
                b.view(torch.int16 if dtype != W.FP32 else torch.int32).fill_(-1)      # NaN patterns
            src = x
            for b in bufs:                                                   # back to back
                fs.fs_softmax(src, b, rows, cols, dtype, 4.0, s)
                src = b
            torch.cuda.synchronize()
            for b, w in zip(bufs, want):
                assert torch.equal(b.view(torch.uint8), w.view(torch.uint8)), (dtype, rows, cols, rep)
    assert fs.fs_device_status() == fs.FS_OK
