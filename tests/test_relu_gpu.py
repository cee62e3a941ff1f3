"""GPU parity for the ReLU kernel function (LINATTN_OPT_KERNEL_FUNCTION = 1), the second row of the paper's
comparison across kernel functions: Eq. 5 with phi(x) = max(x, 0), against the oracle's ref_relu_linear and, on
sampled rows, its O(n^2) form.  Tolerances as for the Hedgehog map: relative L2 <= 5e-3, max-abs <= 2e-2."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2510_08318_b200 import linattn, synth
from util import assert_parity, errors

pytestmark = pytest.mark.gpu

MODES = [(linattn.PATH_AUTO, 1), (linattn.PATH_AUTO, 0), (linattn.PATH_SIMT, 0)]
MODE_IDS = ["auto", "unfused", "simt"]


def _inputs(B, H, n, d, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    q, k, v = (torch.randn(B, H, n, d, generator=g) / math.sqrt(d) for _ in range(3))
    return {"q": q.to(dtype), "k": k.to(dtype), "v": v.to(dtype)}


def _ctx(H, d, B, n, mode):
    ctx = linattn.LinAttn(H, d, max_B=B, max_n=n)
    ctx.set_option(linattn.OPT_PATH, mode[0])
    ctx.set_option(linattn.OPT_FUSE, mode[1])
    ctx.set_option(linattn.OPT_KERNEL_FUNCTION, linattn.PHI_RELU)   # no feature-map weights are set
    return ctx


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("B,H,n,d,dtype", [(2, 3, 1000, 128, torch.bfloat16), (1, 2, 129, 128, torch.bfloat16),
                                           (1, 12, 2048, 128, torch.bfloat16), (1, 1, 1, 128, torch.bfloat16),
                                           (2, 2, 300, 64, torch.float32), (1, 3, 257, 128, torch.float32),
                                           (1, 2, 77, 64, torch.bfloat16)])
def test_relu_matches_the_oracle(B, H, n, d, dtype, mode):
    x = _inputs(B, H, n, d, dtype, seed=300 + n)
    want, S_ref, z_ref = oracle.ref_relu_linear(x["q"], x["k"], x["v"], return_state=True)
    ctx = _ctx(H, d, B, n, mode)
    try:
        q, k, v = x["q"].cuda(), x["k"].cuda(), x["v"].cuda()
        got = ctx.forward(q, k, v)
        again = ctx.forward(q, k, v)
        ctx.check()
        S, z = ctx.read_state(B)
        assert torch.equal(got, again)
        assert_parity(got.cpu().double().numpy(), want, f"relu {mode} n={n} d={d} {dtype}")
        assert errors(S.double().numpy(), S_ref)[0] <= 5e-3 and errors(z.double().numpy(), z_ref)[0] <= 5e-3
        # Eq. 8 with this kernel function, and the token-major layout
        soft = torch.randn_like(q)
        mixed = ctx.forward_mixed(q, k, v, soft, 0.4)
        assert_parity(mixed.cpu().double().numpy(), oracle.ref_mix(soft.cpu().double().numpy(), want, 0.4), "relu, mixed")
        ctx.set_option(linattn.OPT_LAYOUT, linattn.LAYOUT_BNHD)
        tm = lambda t: t.permute(0, 2, 1, 3).contiguous().view(B, H, n, d)
        got_tm = ctx.forward(tm(q), tm(k), tm(v))
        ctx.check()
        assert torch.equal(got_tm.view(B, n, H, d).permute(0, 2, 1, 3), got)
    finally:
        ctx.destroy()


def test_switching_back_to_the_hedgehog_map_on_one_context():
    B, H, n, d = 1, 2, 640, 128
    g = torch.Generator().manual_seed(5)
    q, k, v = (torch.randn(B, H, n, d, generator=g).div(math.sqrt(d)).bfloat16() for _ in range(3))
    Wq, Wk = (torch.randn(H, d, d // 2, generator=g).bfloat16() for _ in range(2))
    ctx = linattn.LinAttn(H, d, max_B=B, max_n=n)
    try:
        with pytest.raises(linattn.LinAttnError) as e:
            ctx.forward(q.cuda(), k.cuda(), v.cuda())
        assert e.value.status == linattn.ERR_NO_FEATURE_MAP
        ctx.set_option(linattn.OPT_KERNEL_FUNCTION, linattn.PHI_RELU)
        relu = ctx.forward(q.cuda(), k.cuda(), v.cuda())
        assert_parity(relu.cpu().double().numpy(), oracle.ref_relu_linear(q, k, v), "relu before the map is set")
        ctx.set_feature_map(Wq.cuda(), Wk.cuda())
        assert torch.equal(ctx.forward(q.cuda(), k.cuda(), v.cuda()), relu), "the weights must not matter to the ReLU kernel function"
        ctx.set_option(linattn.OPT_KERNEL_FUNCTION, linattn.PHI_HEDGEHOG)
        hedge = ctx.forward(q.cuda(), k.cuda(), v.cuda())
        ctx.check()
        assert_parity(hedge.cpu().double().numpy(), oracle.ref_linear(q, k, v, Wq, Wk), "hedgehog after relu")
        with pytest.raises(linattn.LinAttnError):
            ctx.set_option(linattn.OPT_KERNEL_FUNCTION, 2)
        # the gradients exist for the ReLU kernel function too (CUDA-core kernels; tests/test_backward_mixed_gpu.py),
        # but there are no tensor-core kernels for them: asking for those is an error, not a silent detour
        ctx.set_option(linattn.OPT_KERNEL_FUNCTION, linattn.PHI_RELU)
        ctx.set_option(linattn.OPT_PATH, linattn.PATH_TENSOR)
        with pytest.raises(linattn.LinAttnError) as e:
            ctx.backward(q.cuda(), k.cuda(), v.cuda(), q.cuda())
        assert e.value.status == linattn.ERR_UNSUPPORTED
    finally:
        ctx.destroy()


def test_config2_full_size_relu():
    x = synth.make_inputs(2)
    B, H, n, d = x["q"].shape
    ctx = _ctx(H, d, B, n, MODES[0])
    try:
        got = ctx.forward(x["q"].cuda(), x["k"].cuda(), x["v"].cuda())
        ctx.check()
        assert ctx.last_launch_count() == 1, "expected the fused tensor-core kernel"
        want = oracle.ref_relu_linear(x["q"], x["k"], x["v"])
        assert_parity(got.cpu().double().numpy(), want, "config 2, ReLU, whole output")
        rows = np.sort(np.unique(np.concatenate([np.random.default_rng(3).choice(n, 28, replace=False), [0, 127, n - 128, n - 1]])))
        want_q = oracle.ref_relu_quadratic(x["q"], x["k"], x["v"], rows=rows)
        assert_parity(got.cpu()[:, :, torch.from_numpy(rows)].double().numpy(), want_q, "config 2, ReLU, vs the O(n^2) form")
    finally:
        ctx.destroy()
