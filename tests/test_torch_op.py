"""The guarded PyTorch front end (the analogue of the paper's guarded dispatch, Sec. III-E): calls
the library only when the guard admits them, else eager. CPU part: the guard's reasons, the eager
route, patch/restore. GPU part: admitted calls against the oracle, a small attention block under
the patch against its eager self."""
import numpy as np
import pytest
import torch

from paper_2607_24762_b200 import torch_op


def test_guard_reasons_and_eager_route_on_cpu():
    torch_op.stats(reset=True)
    x = torch.randn(4, 9)
    assert torch_op.why_not(x, -1) == "not on a CUDA device"
    y = torch_op.softmax(x, -1)
    assert torch.equal(y, torch.softmax(x, -1))
    y = torch_op.softmax(x, -1, scale=0.5)
    assert torch.allclose(y, torch.softmax(x * 0.5, -1))
    out = torch.empty_like(x)
    assert torch_op.softmax(x, -1, out=out) is out and torch.equal(out, torch.softmax(x, -1))
    assert torch_op.stats()["eager:not on a CUDA device"] == 3
    assert torch_op.why_not(torch.zeros(3, dtype=torch.float64), -1) is not None
    assert torch_op.why_not("x", -1) == "not a tensor"


def test_patch_routes_and_restores():
    before = (torch.softmax, torch.nn.functional.softmax, torch.Tensor.softmax)
    x = torch.randn(3, 5)
    torch_op.stats(reset=True)
    with torch_op.patched():
        a = torch.softmax(x, -1)
        b = torch.nn.functional.softmax(x, dim=1)
        c = x.softmax(-1)
        d = torch.softmax(x, 0, dtype=torch.float64)
    assert (torch.softmax, torch.nn.functional.softmax, torch.Tensor.softmax) == before
    ref = before[0](x, -1)
    assert torch.equal(a, ref) and torch.equal(b, ref) and torch.equal(c, ref)
    assert d.dtype == torch.float64
    assert sum(torch_op.stats().values()) == 4


@pytest.mark.gpu
def test_admitted_calls_match_the_oracle_and_others_fall_back():
    from oracle import fso
    from paper_2607_24762_b200 import workloads as W
    torch_op.stats(reset=True)
    for tdt, dt in ((torch.float32, W.FP32), (torch.bfloat16, W.BF16), (torch.float16, W.FP16)):
        x = (torch.randn(2, 4, 33, 2048, device="cuda") * 2).to(tdt)
        y = torch_op.softmax(x, -1, scale=0.25)
        assert y.shape == x.shape and y.dtype == x.dtype
        bits = (lambda t: t.view(torch.int16).cpu().numpy().view(np.uint16)) if dt != W.FP32 else (lambda t: t.cpu().numpy())
        rep = fso.compare(bits(y).reshape(-1, 2048), dt, fso.softmax_f64(bits(x).reshape(-1, 2048), dt, 0.25))
        assert rep.ok(dt), rep
    assert torch_op.stats()["library"] == 3
    x = torch.randn(8, 64, device="cuda")
    assert torch_op.why_not(x, 0) == "softmax dimension is not the last one"
    assert torch.equal(torch_op.softmax(x, 0), torch.softmax(x, 0))
    xt = x.t()
    assert torch_op.why_not(xt, -1) == "not contiguous"
    assert torch.allclose(torch_op.softmax(xt, -1), torch.softmax(xt, -1))
    xg = x.clone().requires_grad_(True)
    assert torch_op.why_not(xg, -1) == "autograd is recording" and torch_op.why_not(xg, -1, grad_ok=True) is None
    with torch.no_grad():
        assert torch_op.why_not(xg, -1) is None
    # log_softmax has no backward kernel: while autograd records, the guard sends it to eager, and autograd works
    lg = torch_op.log_softmax(xg, -1)
    lg.sum().backward()
    assert xg.grad is not None
    assert torch_op.why_not(x, -1, dtype=torch.float64) == "output dtype conversion requested"
    # eager attention's upcast: 16-bit scores, float32 probabilities, through the mixed-dtype kernel
    xb = (torch.randn(4, 8, 96, 1024, device="cuda") * 2).to(torch.bfloat16)
    before = torch_op.stats().get("library", 0)
    yb = torch_op.softmax(xb, -1, dtype=torch.float32)
    assert yb.dtype == torch.float32 and torch_op.stats()["library"] == before + 1
    assert torch.allclose(yb, torch.softmax(xb, -1, dtype=torch.float32), atol=2e-6, rtol=0)
    assert torch_op.log_softmax(xb, -1, dtype=torch.float32).dtype == torch.float32          # eager route


@pytest.mark.gpu
def test_attention_block_under_the_patch_matches_eager():
    torch.manual_seed(0)

    def attention(q, k, v):                               # eager attention as in the paper's LLM workloads
        s = torch.matmul(q, k.transpose(-1, -2)) / q.shape[-1] ** 0.5
        mask = torch.full(s.shape[-2:], float("-inf"), device=s.device, dtype=s.dtype).triu(1)
        p = torch.nn.functional.softmax(s + mask, dim=-1)
        return torch.matmul(p, v)

    q, k, v = (torch.randn(1, 8, 256, 64, device="cuda", dtype=torch.bfloat16) for _ in range(3))
    with torch.no_grad():
        ref = attention(q, k, v)
        torch_op.stats(reset=True)
        with torch_op.patched():
            got = attention(q, k, v)
    assert torch_op.stats().get("library", 0) == 1
    assert torch.allclose(got.float(), ref.float(), atol=2e-2, rtol=2e-2)


def test_patch_covers_log_softmax_and_norms_on_cpu():
    F = torch.nn.functional
    before = (torch.log_softmax, F.log_softmax, F.layer_norm, F.group_norm)
    x = torch.randn(4, 6, 10)
    w, b = torch.randn(10), torch.randn(10)
    torch_op.stats(reset=True)
    with torch_op.patched():
        a = F.log_softmax(x, dim=-1)
        c = torch.log_softmax(x, -1)
        d = F.layer_norm(x, (10,), w, b, 1e-5)
        e = F.group_norm(x, 3, None, None, 1e-5)
        m = torch.nn.LayerNorm(10)(x)                     # modules call F.layer_norm at run time
    assert (torch.log_softmax, F.log_softmax, F.layer_norm, F.group_norm) == before
    assert torch.equal(a, before[0](x, -1)) and torch.equal(c, a)
    assert torch.equal(d, before[2](x, (10,), w, b, 1e-5)) and torch.equal(e, before[3](x, 3, None, None, 1e-5))
    assert m.shape == x.shape
    assert sum(torch_op.stats().values()) == 5 and "library" not in torch_op.stats()


@pytest.mark.gpu
def test_log_softmax_and_norms_through_the_guard_on_gpu():
    F = torch.nn.functional
    torch.manual_seed(1)
    torch_op.stats(reset=True)
    with torch.no_grad():
        x = torch.randn(3, 50, 1536, device="cuda", dtype=torch.bfloat16)
        w = torch.randn(1536, device="cuda", dtype=torch.bfloat16)
        b = torch.randn(1536, device="cuda", dtype=torch.bfloat16)
        logits = torch.randn(7, 32000, device="cuda", dtype=torch.float32) * 3
        img = torch.randn(2, 64, 32, 32, device="cuda", dtype=torch.float16)
        gw = torch.randn(64, device="cuda", dtype=torch.float16)
        ref = (F.layer_norm(x.float(), (1536,), w.float(), b.float(), 1e-5), torch.log_softmax(logits.double(), -1),
               F.group_norm(img.float(), 32, gw.float(), None, 1e-5))
        with torch_op.patched():
            got = (F.layer_norm(x, (1536,), w, b, 1e-5), torch.log_softmax(logits, -1), F.group_norm(img, 32, gw, None, 1e-5),
                   torch.nn.LayerNorm(1536, device="cuda", dtype=torch.bfloat16)(x))
    assert torch_op.stats().get("library", 0) == 4
    assert torch.allclose(got[0].float(), ref[0], atol=3e-2, rtol=2e-2)
    assert torch.allclose(got[1].double(), ref[1], atol=1e-5, rtol=1e-6)
    assert torch.allclose(got[2].float(), ref[2], atol=1e-2, rtol=1e-2)
    assert got[3].shape == x.shape and torch.isfinite(got[3].float()).all()
    # guard: a weight on another dtype goes to eager
    assert torch.allclose(torch_op.layer_norm(x, (1536,), w, b).float(), ref[0], atol=3e-2, rtol=2e-2)
    y = torch_op.layer_norm(x.float(), (1536,), w.float(), b.float())
    assert y.dtype == torch.float32


def test_registered_operators_pass_opcheck_on_cpu():
    """The operators exist under torch.ops.fsoftmax with schema, fake implementation and (softmax) autograd
    registration that torch's own checker accepts; on CPU tensors they compute with eager PyTorch."""
    ops = torch.ops.fsoftmax
    for name in ("softmax", "softmax_backward", "log_softmax", "layer_norm", "group_norm"):
        assert hasattr(ops, name)
    torch.manual_seed(3)
    cases = [(ops.softmax, (torch.randn(3, 5, requires_grad=True), 0.5)),
             (ops.softmax_backward, (torch.randn(3, 5), torch.softmax(torch.randn(3, 5), -1), 0.5)),
             (ops.log_softmax, (torch.randn(3, 5),)),
             (ops.layer_norm, (torch.randn(3, 5), torch.randn(5), None, 1e-5)),
             (ops.group_norm, (torch.randn(2, 4, 5), 2, None, torch.randn(4), 1e-5))]
    for op, args in cases:
        res = torch.library.opcheck(op, args)
        assert all(v == "SUCCESS" for v in res.values()), (op, res)
    x = torch.randn(4, 9, dtype=torch.float64, requires_grad=True)
    g = torch.randn(4, 9, dtype=torch.float64)
    ops.softmax(x, 0.5).backward(g)
    xr = x.detach().clone().requires_grad_(True)
    torch.softmax(xr * 0.5, -1).backward(g)
    assert torch.allclose(x.grad, xr.grad, atol=1e-12)


@pytest.mark.gpu
def test_softmax_operator_forward_and_backward_run_the_library():
    """torch.ops.fsoftmax.softmax on a tensor that requires grad: forward through fs_softmax, x.grad through
    fs_softmax_backward, both against the oracle under the bars of their entry points."""
    from oracle import fno, fso
    from paper_2607_24762_b200 import workloads as W
    torch.manual_seed(5)
    for tdt, dt, rows, cols, scale in ((torch.float32, W.FP32, 48, 4096, 1.0), (torch.bfloat16, W.BF16, 64, 2048, 0.125),
                                       (torch.float16, W.FP16, 6, 65536, 0.5)):
        x = (torch.randn(rows, cols, device="cuda") * 2).to(tdt).requires_grad_(True)
        dy = torch.randn(rows, cols, device="cuda").to(tdt)
        torch_op.stats(reset=True)
        y = torch_op.softmax(x, -1, scale=scale)                    # the guarded front end routes to the operator
        y.backward(dy)
        assert torch_op.stats() == {"library": 2}                   # one forward, one backward kernel; nothing went to eager
        bits = (lambda t: t.detach().view(torch.int16).cpu().numpy().view(np.uint16)) if dt != W.FP32 else (lambda t: t.detach().cpu().numpy())
        assert fso.compare(bits(y), dt, fso.softmax_f64(bits(x), dt, scale)).ok(dt)
        es = fno.backward_error_scale(bits(dy), bits(y), dt, scale)
        rep = fno.compare(bits(x.grad), dt, fso.softmax_backward_f64(bits(dy), bits(y), dt, scale), es)
        assert rep.ok(dt), rep
    # called directly, as a traced graph would: same kernels; a tensor the guard refuses is computed by eager
    xs = torch.randn(8, 512, device="cuda")
    assert torch.allclose(torch.ops.fsoftmax.softmax(xs, 1.0), torch.softmax(xs, -1), atol=1e-6)
    xt = torch.randn(512, 8, device="cuda").t()
    assert torch.allclose(torch.ops.fsoftmax.softmax(xt, 1.0), torch.softmax(xt, -1), atol=1e-6)
    assert torch_op.stats()["eager:operator called on tensors the guard refuses"] == 1
