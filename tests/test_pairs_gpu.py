"""Head dimension 64 on the tensor-core kernels: the heads are taken two at a time (a pair of heads is one 128-feature
unit with block-diagonal feature-map weights, state S and normaliser z), so that the d = 128 kernels' shapes apply.
Checked against the fp64 oracle head by head (an error that mixed the two heads of a pair would show at once), for
even and odd numbers of heads (the last pair may lack its second head), ragged lengths, both memory layouts, mixed
attention and the ReLU kernel function; the single-kernel form must equal the three-launch form bit for bit."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2510_08318_b200 import linattn, synth
from util import assert_parity, errors

pytestmark = pytest.mark.gpu


def _inputs(B, H, n, seed, shared=False):
    d = 64
    g = torch.Generator().manual_seed(seed)
    sx = 1.0 / math.sqrt(d)
    q, k, v = (torch.randn(B, H, n, d, generator=g).mul_(sx).bfloat16() for _ in range(3))
    wshape = (d, d // 2) if shared else (H, d, d // 2)
    Wq, Wk = (torch.randn(*wshape, generator=g).div_(math.sqrt(d) * sx).bfloat16() for _ in range(2))
    return {"q": q, "k": k, "v": v, "Wq": Wq, "Wk": Wk}


def _ctx(x):
    B, H, n, d = x["q"].shape
    ctx = linattn.LinAttn(H, d, max_B=B, max_n=n)
    ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
    return ctx


def test_bf16_d64_takes_the_tensor_core_kernels():
    x = _inputs(1, 4, 700, seed=1)
    ctx = _ctx(x)
    try:
        ctx.set_option(linattn.OPT_PROFILE, 1)
        q, k, v = (x[t].cuda() for t in "qkv")
        ctx.forward(q, k, v)
        ctx.check()
        assert [kt["name"] for kt in ctx.kernel_times()] == ["linattn_fused_tc"] and ctx.last_launch_count() == 1
        ctx.set_option(linattn.OPT_PATH, linattn.PATH_TENSOR)
        ctx.set_option(linattn.OPT_FUSE, 0)
        ctx.forward(q, k, v)
        ctx.check()
        assert [kt["name"] for kt in ctx.kernel_times()] == ["kside_tc", "combine_tc", "qside_tc"]
    finally:
        ctx.destroy()


@pytest.mark.parametrize("fuse", [1, 0], ids=["fused", "unfused"])
@pytest.mark.parametrize("n", [1, 2, 127, 129, 1000, 4097])
@pytest.mark.parametrize("B,H", [(1, 1), (1, 2), (1, 3), (2, 3), (1, 5), (2, 4)])
def test_parity_head_by_head(B, H, n, fuse):
    x = _inputs(B, H, n, seed=100 * H + n + B)
    ctx = _ctx(x)
    try:
        ctx.set_option(linattn.OPT_FUSE, fuse)
        out = ctx.forward(*(x[t].cuda() for t in "qkv"))
        ctx.check()
        assert ctx.last_launch_count() == (1 if fuse else 3)
        S, z = ctx.read_state(B)
    finally:
        ctx.destroy()
    want, S_ref, z_ref = oracle.ref_linear(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], return_state=True)
    got = out.cpu().double().numpy()
    for b in range(B):
        for h in range(H):
            assert_parity(got[b, h], want[b, h], f"B={B} H={H} n={n} head ({b},{h})")
            assert errors(S[b, h].double().numpy(), S_ref[b, h])[0] <= 5e-3, f"S of head ({b},{h})"
            assert errors(z[b, h].double().numpy(), z_ref[b, h])[0] <= 5e-3, f"z of head ({b},{h})"
    assert abs(z.double().numpy().sum(-1) - 2.0 * n).max() <= 2e-3 * 2.0 * n, "sum(z) must be 2n for every head"


def test_shared_weights_and_special_maps():
    x = _inputs(2, 3, 900, seed=7, shared=True)
    ctx = _ctx(x)
    try:
        out = ctx.forward(*(x[t].cuda() for t in "qkv"))
        ctx.check()
        assert ctx.last_launch_count() == 1
        assert_parity(out.cpu().double().numpy(), oracle.ref_linear(x["q"], x["k"], x["v"], x["Wq"], x["Wk"]), "shared W")
        # W = 0: every head returns the mean of its own V (a leak between the heads of a pair would break this)
        zero = torch.zeros(3, 64, 32, dtype=torch.bfloat16, device="cuda")
        ctx.set_feature_map(zero, zero)
        out0 = ctx.forward(*(x[t].cuda() for t in "qkv"))
        ctx.check()
        mean_v = x["v"].double().numpy().mean(axis=2, keepdims=True)
        assert_parity(out0.cpu().double().numpy(), np.broadcast_to(mean_v, out0.shape), "W = 0 -> mean of V per head")
    finally:
        ctx.destroy()


def test_fused_equals_three_launches_bit_for_bit():
    dev = torch.device("cuda", 0)
    g = torch.Generator(device=dev).manual_seed(321)
    checked = 0
    for G in (1, 2, 3, 5, 8, 11, 30, 41, 75, 151, 297):
        for Tn in (1, 2, 3, 5, 8, 13, 21):
            if G * Tn > 3000:
                continue
            n = Tn * 128 - (29 if Tn % 2 else 0)
            q, k, v = (torch.randn(1, G, n, 64, generator=g, device=dev).mul_(0.125).bfloat16() for _ in range(3))
            Wq, Wk = (torch.randn(G, 64, 32, generator=g, device=dev).bfloat16() for _ in range(2))
            ctx = linattn.LinAttn(G, 64, max_B=1, max_n=n)
            try:
                ctx.set_feature_map(Wq, Wk)
                fused = ctx.forward(q, k, v)
                fused_mixed = ctx.forward_mixed(q, k, v, v, 0.25)
                ctx.check()
                assert ctx.last_launch_count() == 1
                ctx.set_option(linattn.OPT_FUSE, 0)
                unfused = ctx.forward(q, k, v)
                unfused_mixed = ctx.forward_mixed(q, k, v, v, 0.25)
                ctx.check()
                assert torch.isfinite(fused.float()).all(), f"G={G} tiles per head={Tn}"
                assert torch.equal(fused, unfused), f"G={G} tiles per head={Tn}"
                assert torch.equal(fused_mixed, unfused_mixed), f"mixed attention, G={G} tiles per head={Tn}"
                checked += 1
            finally:
                ctx.destroy()
    assert checked > 60


@pytest.mark.parametrize("B,H,n", [(2, 3, 1000), (1, 5, 129), (2, 2, 300)])
def test_token_major_layout(B, H, n):
    x = _inputs(B, H, n, seed=n + H)
    ctx = _ctx(x)
    try:
        q, k, v = (x[t].cuda() for t in "qkv")
        ref = ctx.forward(q, k, v)
        soft = torch.randn_like(q)
        ref_mixed = ctx.forward_mixed(q, k, v, soft, 0.3)
        tm = lambda t: t.permute(0, 2, 1, 3).contiguous().view(B, H, n, 64)
        back = lambda t: t.view(B, n, H, 64).permute(0, 2, 1, 3)
        ctx.set_option(linattn.OPT_LAYOUT, linattn.LAYOUT_BNHD)
        got = ctx.forward(tm(q), tm(k), tm(v))
        got_mixed = ctx.forward_mixed(tm(q), tm(k), tm(v), tm(soft), 0.3)
        ctx.check()
        assert ctx.last_launch_count() == 1
        assert torch.equal(back(got), ref) and torch.equal(back(got_mixed), ref_mixed)
        assert_parity(back(got).cpu().double().numpy(), oracle.ref_linear(x["q"], x["k"], x["v"], x["Wq"], x["Wk"]), "[B][n][H][64]")
    finally:
        ctx.destroy()


def test_mixed_attention_and_relu():
    x = _inputs(1, 3, 1500, seed=9)
    ctx = _ctx(x)
    try:
        q, k, v = (x[t].cuda() for t in "qkv")
        soft = oracle.ref_softmax(x["q"], x["k"], x["v"], 1.0 / 8.0)
        soft_dev = torch.from_numpy(soft).bfloat16().cuda()
        lin = oracle.ref_linear(x["q"], x["k"], x["v"], x["Wq"], x["Wk"])
        for r in (0.0, 0.35, 1.0, 1.7):
            got = ctx.forward_mixed(q, k, v, soft_dev, r)
            ctx.check()
            assert_parity(got.cpu().double().numpy(), oracle.ref_mix(soft_dev.cpu().double().numpy(), lin, r), f"mixed r={r}")
        ctx.set_option(linattn.OPT_KERNEL_FUNCTION, linattn.PHI_RELU)
        got = ctx.forward(q, k, v)
        ctx.check()
        assert ctx.last_launch_count() == 1
        assert_parity(got.cpu().double().numpy(), oracle.ref_relu_linear(x["q"], x["k"], x["v"]), "ReLU, d = 64")
    finally:
        ctx.destroy()


def test_cogvideox_shaped_workload_full_size():
    """Config 6 at full size in the benchmark's launch configuration: S, z in full, 512 sampled rows against the
    right-hand form of Eq. 5 and 64 against the O(n^2) definition."""
    x = synth.make_inputs(6)
    B, H, n, d = x["q"].shape
    ctx = _ctx(x)
    try:
        q, k, v = (x[t].cuda() for t in "qkv")
        out = ctx.forward(q, k, v)
        again = ctx.forward(q, k, v)
        ctx.check()
        assert ctx.last_launch_count() == 1 and torch.equal(out, again)
        S, z = ctx.read_state(B)
    finally:
        ctx.destroy()
    rng = np.random.default_rng(6)
    rows = np.sort(np.unique(np.concatenate([[0, 127, n - 112, n - 1], rng.choice(n, 512, replace=False)])))
    want, S_ref, z_ref = oracle.ref_linear(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], rows=rows, return_state=True)
    assert_parity(out.cpu()[:, :, torch.from_numpy(rows)].double().numpy(), want, "config 6, sampled rows")
    assert errors(S.double().numpy(), S_ref)[0] <= 5e-3 and errors(z.double().numpy(), z_ref)[0] <= 5e-3
    rows_q = np.sort(np.unique(np.concatenate([[0, n - 1], rng.choice(n, 62, replace=False)])))
    want_q = oracle.ref_quadratic(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], rows=rows_q)
    assert_parity(out.cpu()[:, :, torch.from_numpy(rows_q)].double().numpy(), want_q, "config 6 vs the O(n^2) definition")
