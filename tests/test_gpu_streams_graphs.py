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
