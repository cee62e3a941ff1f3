"""GPU parity for mixed attention (Eq. 8): linattn_forward_mixed against the oracle's blend of its
softmax-attention term and its linear-attention term.

The softmax branch's output is an INPUT of the entry point; the tests take it from the oracle (small cases) or
from torch's attention kernel (full size), round it to the storage type once, and give the same rounded values
to both sides.  Tolerances as everywhere: relative L2 <= 5e-3, max-abs <= 2e-2.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2510_08318_b200 import linattn, synth
from util import assert_parity

pytestmark = pytest.mark.gpu

MODES = [(linattn.PATH_AUTO, 1), (linattn.PATH_AUTO, 0), (linattn.PATH_SIMT, 0)]
MODE_IDS = ["auto", "unfused", "simt"]


def _inputs(B, H, n, d, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    sx = 1.0 / math.sqrt(d)
    q, k, v = (torch.randn(B, H, n, d, generator=g) * sx for _ in range(3))
    Wq, Wk = (torch.randn(H, d, d // 2, generator=g) / (math.sqrt(d) * sx) for _ in range(2))
    x = {"q": q.to(dtype), "k": k.to(dtype), "v": v.to(dtype), "Wq": Wq.to(dtype), "Wk": Wk.to(dtype)}
    # softmax branch on the rounded inputs; q.k has standard deviation 1/sqrt(d) here, so this scale gives logits of
    # standard deviation 3: a softmax that differs clearly from both the uniform average and the linear branch
    soft = oracle.ref_softmax(x["q"], x["k"], x["v"], scale=3.0 * math.sqrt(d))
    x["soft"] = torch.from_numpy(soft).to(dtype)
    return x


def _ctx(x, mode):
    B, H, n, d = x["q"].shape
    ctx = linattn.LinAttn(H, d, max_B=B, max_n=n)
    ctx.set_option(linattn.OPT_PATH, mode[0])
    ctx.set_option(linattn.OPT_FUSE, mode[1])
    ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
    return ctx


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("n,d,dtype", [(1000, 128, torch.bfloat16), (129, 128, torch.bfloat16), (300, 64, torch.float32),
                                       (257, 128, torch.float32)])
def test_blend_matches_the_oracle(n, d, dtype, mode):
    x = _inputs(2, 2, n, d, dtype, seed=100 + n)
    lin = oracle.ref_linear(x["q"], x["k"], x["v"], x["Wq"], x["Wk"])
    soft = x["soft"].double().numpy()
    ctx = _ctx(x, mode)
    try:
        q, k, v, a = x["q"].cuda(), x["k"].cuda(), x["v"].cuda(), x["soft"].cuda()
        plain = ctx.forward(q, k, v)
        for r in (0.0, 0.3, 0.75, 1.0, 1.7, -0.5):
            got = ctx.forward_mixed(q, k, v, a, r)
            ctx.check()
            assert_parity(got.cpu().double().numpy(), oracle.ref_mix(soft, lin, r), f"r={r} n={n} d={d} {dtype}")
            if r <= 0.0:
                assert torch.equal(got, plain), "a clipped score of 0 must give the plain linear attention"
            if r >= 1.0:
                assert torch.equal(got, a), "a clipped score of 1 must return the softmax branch"
    finally:
        ctx.destroy()


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
def test_in_place_on_the_softmax_buffer(mode):
    x = _inputs(1, 3, 777, 128, torch.bfloat16, seed=7)
    ctx = _ctx(x, mode)
    try:
        q, k, v = x["q"].cuda(), x["k"].cuda(), x["v"].cuda()
        separate = ctx.forward_mixed(q, k, v, x["soft"].cuda(), 0.4)
        buf = x["soft"].cuda().clone()
        ctx.forward_mixed(q, k, v, buf, 0.4, out=buf)
        ctx.check()
        assert torch.equal(buf, separate)
    finally:
        ctx.destroy()


def test_argument_errors():
    lib = linattn.load_library()
    x = _inputs(1, 2, 256, 128, torch.bfloat16, seed=8)
    ctx = _ctx(x, MODES[0])
    try:
        q, k, v, a = x["q"].cuda(), x["k"].cuda(), x["v"].cuda(), x["soft"].cuda()
        big = torch.empty(q.numel() + 64, dtype=q.dtype, device="cuda")
        out = big[:q.numel()].view_as(q)
        shifted = big[64:].view_as(q)   # overlaps `out` without being the same buffer

        def call(ap, r, op):
            return lib.linattn_forward_mixed(ctx._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), ap, r, op, 1, 2, 256, 128,
                                             linattn.BF16, None)
        assert call(a.data_ptr(), 0.5, out.data_ptr()) == linattn.OK
        assert call(None, 0.5, out.data_ptr()) == linattn.ERR_INVALID_ARG
        assert call(a.data_ptr(), float("nan"), out.data_ptr()) == linattn.ERR_INVALID_ARG
        assert call(shifted.data_ptr(), 0.5, out.data_ptr()) == linattn.ERR_INVALID_ARG
        assert call(a.data_ptr() + 2, 0.5, out.data_ptr()) == linattn.ERR_INVALID_ARG
        assert call(a.data_ptr(), 0.5, q.data_ptr()) == linattn.ERR_INVALID_ARG   # out aliases q
        ctx.check()
    finally:
        ctx.destroy()


def test_config2_full_size_with_a_library_softmax_branch():
    """Full size, fused kernel: the softmax branch comes from torch's attention kernel on the GPU (it is only an
    input here); sampled rows against the oracle's blend of those very values with its own linear attention."""
    x = synth.make_inputs(2)
    B, H, n, d = x["q"].shape
    ctx = linattn.LinAttn(H, d, max_B=B, max_n=n)
    try:
        ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
        q, k, v = x["q"].cuda(), x["k"].cuda(), x["v"].cuda()
        a = torch.nn.functional.scaled_dot_product_attention(q, k, v)
        got = ctx.forward_mixed(q, k, v, a, 0.35)
        ctx.check()
        assert ctx.last_launch_count() == 1
        rows = np.sort(np.unique(np.concatenate([np.random.default_rng(9).choice(n, 1500, replace=False), [0, 127, n - 128, n - 1]])))
        lin = oracle.ref_linear(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], rows=rows)
        idx = torch.from_numpy(rows)
        want = oracle.ref_mix(a.cpu()[:, :, idx].double().numpy(), lin, 0.35)
        assert_parity(got.cpu()[:, :, idx].double().numpy(), want, "config 2 mixed, sampled rows")
    finally:
        ctx.destroy()
