"""GPU parity of the gradients through mixed attention (Eq. 8) and of the gradients with the ReLU kernel function,
against the oracle.  Tolerances as for linattn_backward: relative L2 <= 5e-3 per gradient tensor and max-abs <=
2e-2 * max|reference|; dL/dr is one number, a sum of signed terms t = dout * (a - lin), and is held to
1e-2 * ||t||_2 (the size of what rounding lin to bf16 can add up to) plus 1e-6 * ||t||_1 for fp32 summation."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2510_08318_b200 import linattn
from util import errors

pytestmark = pytest.mark.gpu

NAMES = ("dq", "dk", "dv", "dWq", "dWk", "d_o_softmax")


def _inputs(B, H, n, d, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    sx = 1.0 / math.sqrt(d)
    q, k, v = (torch.randn(B, H, n, d, generator=g) * sx for _ in range(3))
    Wq, Wk = (torch.randn(H, d, d // 2, generator=g) / (math.sqrt(d) * sx) for _ in range(2))
    dout = torch.randn(B, H, n, d, generator=g)
    a = torch.randn(B, H, n, d, generator=g) * sx
    return {"q": q.to(dtype), "k": k.to(dtype), "v": v.to(dtype), "Wq": Wq.to(dtype), "Wk": Wk.to(dtype),
            "dout": dout.to(dtype), "a": a.to(dtype)}


def _close(name, got, want, what):
    got = got.detach().cpu().double().numpy()
    assert np.isfinite(got).all(), f"{what}: {name} has non-finite entries"
    scale = float(np.abs(want).max())
    if scale == 0.0:
        assert np.abs(got).max() == 0.0, f"{what}: {name} must vanish"
        return
    rel, mx = errors(got, want)
    assert rel <= 5e-3 and mx <= 2e-2 * scale, f"{what}: {name} rel-L2 {rel:.3e}, max-abs {mx:.3e} (largest reference entry {scale:.3e})"


def _check_dr(got_dr, x, r, lin, what):
    t = x["dout"].double().numpy() * (x["a"].double().numpy() - lin)
    want = t.sum() if 0.0 <= r <= 1.0 else 0.0
    tol = 1e-2 * np.sqrt((t ** 2).sum()) + 1e-6 * np.abs(t).sum()
    assert abs(float(got_dr) - want) <= (tol if 0.0 <= r <= 1.0 else 0.0), f"{what}: dr {float(got_dr):.6e} vs {want:.6e} (tolerance {tol:.3e})"


@pytest.mark.parametrize("r", [0.3, 0.0, 1.0, -0.5, 1.5])
@pytest.mark.parametrize("B,H,n,d,dtype,path", [
    (2, 2, 1000, 128, torch.bfloat16, linattn.PATH_AUTO),    # tensor-core kernels
    (1, 5, 700, 128, torch.bfloat16, linattn.PATH_AUTO),     # CTA runs that cross heads
    (2, 2, 1000, 128, torch.bfloat16, linattn.PATH_SIMT),
    (2, 2, 300, 64, torch.float32, linattn.PATH_AUTO),       # CUDA-core kernels, fp32
    (1, 3, 257, 64, torch.bfloat16, linattn.PATH_AUTO),
], ids=["tc", "tc-crossing", "simt-bf16", "simt-f32-d64", "simt-bf16-d64"])
def test_mixed_attention_gradients_match_the_oracle(B, H, n, d, dtype, path, r):
    x = _inputs(B, H, n, d, dtype, seed=300 + n + d)
    want = oracle.ref_backward_mixed(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], x["a"], r, x["dout"])
    lin = oracle.ref_linear(x["q"], x["k"], x["v"], x["Wq"], x["Wk"])
    ctx = linattn.LinAttn(H, d, max_B=B, max_n=n)
    try:
        ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
        ctx.set_option(linattn.OPT_PATH, path)
        args = [x[s].cuda() for s in ("q", "k", "v", "a")]
        got = ctx.backward_mixed(*args, r, x["dout"].cuda())
        again = ctx.backward_mixed(*args, r, x["dout"].cuda())
        ctx.check()
        for g1, g2 in zip(got, again):
            assert torch.equal(g1, g2), "the gradients are not bit-reproducible"
    finally:
        ctx.destroy()
    what = f"B={B} H={H} n={n} d={d} {dtype} r={r}"
    for name, g, w in zip(NAMES, got[:6], want[:6]):
        _close(name, g, w, what)
    _check_dr(got[6].item(), x, r, lin, what)
    np.testing.assert_allclose(want[6], (x["dout"].double().numpy() * (x["a"].double().numpy() - lin)).sum() if 0 <= r <= 1 else 0.0,
                               rtol=1e-9, atol=1e-9)


def test_mixed_gradients_in_the_token_major_layout_and_without_the_softmax_branch_gradient():
    B, H, n, d = 2, 3, 900, 128
    x = _inputs(B, H, n, d, torch.bfloat16, seed=77)
    ctx = linattn.LinAttn(H, d, max_B=B, max_n=n)
    try:
        ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
        dev = {s: x[s].cuda() for s in ("q", "k", "v", "a", "dout")}
        ref = ctx.backward_mixed(dev["q"], dev["k"], dev["v"], dev["a"], 0.4, dev["dout"])
        tm = lambda t: t.permute(0, 2, 1, 3).contiguous().view(B, H, n, d)
        back = lambda t: t.view(B, n, H, d).permute(0, 2, 1, 3)
        ctx.set_option(linattn.OPT_LAYOUT, linattn.LAYOUT_BNHD)
        got = ctx.backward_mixed(tm(dev["q"]), tm(dev["k"]), tm(dev["v"]), tm(dev["a"]), 0.4, tm(dev["dout"]), want_d_o_softmax=False)
        ctx.check()
        assert got[5] is None
        for i in range(3):
            assert torch.equal(back(got[i]), ref[i])
        assert torch.equal(got[3], ref[3]) and torch.equal(got[4], ref[4]) and torch.equal(got[6], ref[6])
    finally:
        ctx.destroy()


def test_mixed_backward_argument_errors():
    lib = linattn.load_library()
    x = _inputs(1, 2, 256, 128, torch.bfloat16, seed=5)
    dev = {s: x[s].cuda() for s in ("q", "k", "v", "a", "dout")}
    outs = [torch.empty_like(dev["q"]) for _ in range(4)]
    dW = [torch.empty(2, 128, 64, device="cuda") for _ in range(2)]
    dr = torch.empty(1, device="cuda")
    ctx = linattn.LinAttn(2, 128, max_B=1, max_n=256)
    try:
        ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())

        def call(a=dev["a"], r=0.5, da=outs[3], drp=dr):
            return lib.linattn_backward_mixed(ctx._h, dev["q"].data_ptr(), dev["k"].data_ptr(), dev["v"].data_ptr(),
                                              a.data_ptr() if a is not None else None, r, dev["dout"].data_ptr(), outs[0].data_ptr(),
                                              outs[1].data_ptr(), outs[2].data_ptr(), dW[0].data_ptr(), dW[1].data_ptr(), 1,
                                              da.data_ptr() if da is not None else None, drp.data_ptr() if drp is not None else None,
                                              1, 2, 256, 128, linattn.BF16, None)
        assert call() == linattn.OK
        assert call(a=None) == linattn.ERR_INVALID_ARG
        assert call(r=float("nan")) == linattn.ERR_INVALID_ARG
        assert call(drp=None) == linattn.ERR_INVALID_ARG
        assert call(da=dev["a"]) == linattn.ERR_INVALID_ARG      # the softmax branch's gradient may not overwrite its output
        assert call(da=None) == linattn.OK
        ctx.check()
    finally:
        ctx.destroy()


@pytest.mark.parametrize("B,H,n,d,dtype", [(2, 2, 300, 64, torch.float32), (1, 3, 1000, 128, torch.bfloat16),
                                           (1, 2, 129, 64, torch.bfloat16), (1, 1, 1, 128, torch.float32)])
def test_relu_gradients_match_the_oracle(B, H, n, d, dtype):
    x = _inputs(B, H, n, d, dtype, seed=400 + n)
    want = oracle.ref_relu_backward(x["q"], x["k"], x["v"], x["dout"])
    ctx = linattn.LinAttn(H, d, max_B=B, max_n=n)
    try:
        ctx.set_option(linattn.OPT_KERNEL_FUNCTION, linattn.PHI_RELU)
        args = [x[s].cuda() for s in ("q", "k", "v", "dout")]
        got = ctx.backward(*args)
        again = ctx.backward(*args)
        ctx.check()
        for g1, g2 in zip(got[:3], again[:3]):
            assert torch.equal(g1, g2)
        # Eq. 8 on top of the ReLU kernel function
        want_m = oracle.ref_relu_backward(x["q"], x["k"], x["v"], (0.75 * x["dout"].double()).float()) if dtype == torch.float32 else None
        got_m = ctx.backward_mixed(x["q"].cuda(), x["k"].cuda(), x["v"].cuda(), x["a"].cuda(), 0.25, x["dout"].cuda())
        ctx.check()
    finally:
        ctx.destroy()
    what = f"ReLU B={B} H={H} n={n} d={d} {dtype}"
    if n == 1:
        assert float(got[0].abs().max()) <= 1e-5 and float(got[1].abs().max()) <= 1e-5
        assert torch.allclose(got[2].cpu().float(), x["dout"].float(), rtol=1e-6, atol=0)
        return
    for name, g, w in zip(("dq", "dk", "dv"), got[:3], want):
        _close(name, g, w, what)
    # the gradients are linear in the incoming one: (1 - r^) = 0.75 of the plain ones
    for name, g, w in zip(("dq", "dk", "dv"), got_m[:3], want):
        _close(name, g, 0.75 * w, what + ", Eq. 8 with r = 0.25")
    lin = oracle.ref_relu_linear(x["q"], x["k"], x["v"])
    _check_dr(got_m[6].item(), x, 0.25, lin, what)
