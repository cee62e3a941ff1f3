"""GPU parity: the CUDA library, called through its C-ABI, against the fp64 CPU oracle.

Tolerances (on the whole output tensor, outputs widened to fp64):
    relative L2 <= 5e-3 and max-abs <= 2e-2.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2510_08318_b200 import linattn, synth
from util import assert_parity, errors, run_gpu

pytestmark = pytest.mark.gpu

# (path option, fuse option): automatic choice (one fused tensor-core kernel where it applies), the
# tensor-core kernels as three launches, and the CUDA-core kernels
MODES = [(linattn.PATH_AUTO, 1), (linattn.PATH_AUTO, 0), (linattn.PATH_SIMT, 0)]
MODE_IDS = ["auto", "unfused", "simt"]


def mode_param():
    return pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)


def run_mode(x, mode, **kw):
    return run_gpu(x, path=mode[0], fuse=mode[1], **kw)


def small_inputs(B, H, n, d, dtype, seed, wmode="random"):
    """Inputs with the value distributions of the bf16 workloads (N(0,1)/sqrt(d), unit-variance logits)."""
    g = torch.Generator().manual_seed(seed)
    sx = 1.0 / math.sqrt(d)
    q, k, v = (torch.randn(B, H, n, d, generator=g) * sx for _ in range(3))
    if wmode == "random":
        Wq, Wk = (torch.randn(H, d, d // 2, generator=g) / (math.sqrt(d) * sx) for _ in range(2))
    elif wmode == "zero":
        Wq = Wk = torch.zeros(H, d, d // 2)
    elif wmode == "identity":  # truncated identity [I ; 0], near-identity initialisation of the feature map
        Wq = Wk = torch.eye(d)[:, : d // 2].expand(H, d, d // 2).contiguous() * 8.0
    elif wmode == "shared":
        Wq, Wk = (torch.randn(d, d // 2, generator=g) / (math.sqrt(d) * sx) for _ in range(2))
    return {"q": q.to(dtype), "k": k.to(dtype), "v": v.to(dtype), "Wq": Wq.to(dtype), "Wk": Wk.to(dtype)}


def oracle_out(x, rows=None):
    return oracle.ref_linear(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], rows=rows)


# ---- config 1: the tiny fp32 case against the O(n^2) brute-force form --------------------------

@mode_param()
def test_config1_tiny_against_quadratic_form(mode):
    x = synth.make_inputs(1)
    got, S, z = run_mode(x, mode, return_state=True)
    want = oracle.ref_quadratic(x["q"], x["k"], x["v"], x["Wq"], x["Wk"])
    assert_parity(got, want, "config 1 vs quadratic form")
    _, S_ref, z_ref = oracle.ref_linear(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], return_state=True)
    assert errors(S, S_ref)[0] <= 5e-3 and errors(z, z_ref)[0] <= 5e-3


# ---- ragged sizes: several tiles plus a tail, the degenerate n = 1, 2 -----------------------------

@mode_param()
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("n", [1, 2, 127, 129, 1000, 4097])
def test_ragged_lengths(n, d, dtype, mode):
    x = small_inputs(2, 3, n, d, dtype, seed=1000 + n + d)
    got, S, z = run_mode(x, mode, return_state=True)
    assert_parity(got, oracle_out(x), f"n={n} d={d} {dtype}")
    _, S_ref, z_ref = oracle.ref_linear(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], return_state=True)
    assert errors(z, z_ref)[0] <= 5e-3, "z"
    assert abs(z.sum(-1) - 2.0 * n).max() <= 2e-3 * 2.0 * n, "sum(z) must be 2n: padded rows leaked into z"
    if n == 1:
        assert_parity(got, x["v"].double().numpy(), "n=1 returns v")


@mode_param()
@pytest.mark.parametrize("splits", [1, 2, 3, 7, 33])
def test_split_count_does_not_change_the_answer(splits, mode):
    x = small_inputs(1, 2, 2500, 128, torch.bfloat16, seed=77)
    got = run_mode(x, mode, splits=splits)
    assert_parity(got, oracle_out(x), f"splits={splits}")


# ---- special feature maps ---------------------------------------------------------------------------

@mode_param()
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_zero_weights_give_the_mean_of_v(dtype, mode):
    x = small_inputs(1, 2, 777, 128, dtype, seed=5, wmode="zero")
    got = run_mode(x, mode)
    mean_v = x["v"].double().numpy().mean(axis=2, keepdims=True)
    assert_parity(got, np.broadcast_to(mean_v, got.shape), "W=0 -> mean of V")


@mode_param()
@pytest.mark.parametrize("wmode", ["identity", "shared"])
def test_identity_and_shared_weights(wmode, mode):
    x = small_inputs(2, 2, 900, 128, torch.bfloat16, seed=6, wmode=wmode)
    assert_parity(run_mode(x, mode), oracle_out(x), wmode)


@mode_param()
def test_large_logits_do_not_overflow(mode):
    """Logits of magnitude ~50: exp without max subtraction would overflow fp32 sums / underflow to 0/0."""
    x = small_inputs(1, 2, 600, 128, torch.bfloat16, seed=8)
    x["Wq"] = (x["Wq"].float() * 40).to(torch.bfloat16)
    x["Wk"] = (x["Wk"].float() * 40).to(torch.bfloat16)
    assert_parity(run_mode(x, mode), oracle_out(x), "large logits")


# ---- reduced-size versions of the bf16 workloads (same distributions, fewer heads / tokens) ----------

@mode_param()
@pytest.mark.parametrize("config,H,n", [(2, 3, 4216), (3, 4, 4216), (4, 2, 9300), (5, 3, 4216)])
def test_reduced_workloads(config, H, n, mode):
    x = synth.make_inputs(config, H=H, n=n)
    assert_parity(run_mode(x, mode), oracle_out(x), f"config {config} reduced")


# ---- determinism and context reuse --------------------------------------------------------------------

@mode_param()
def test_bit_identical_across_runs_and_context_reuse(mode):
    x = small_inputs(2, 4, 3000, 128, torch.bfloat16, seed=9)
    ctx = linattn.LinAttn(4, 128, max_B=2, max_n=4000)
    try:
        ctx.set_option(linattn.OPT_PATH, mode[0])
        ctx.set_option(linattn.OPT_FUSE, mode[1])
        ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
        q, k, v = x["q"].cuda(), x["k"].cuda(), x["v"].cuda()
        first = ctx.forward(q, k, v).clone()
        for _ in range(20):
            again = ctx.forward(q, k, v)
            assert torch.equal(first, again)
        # a different, shorter problem on the same context, then the first one again
        y = small_inputs(1, 4, 333, 128, torch.bfloat16, seed=10)
        ctx.set_feature_map(y["Wq"].cuda(), y["Wk"].cuda())
        got = ctx.forward(y["q"].cuda(), y["k"].cuda(), y["v"].cuda()).cpu().double().numpy()
        assert_parity(got, oracle_out(y), "second problem on the same context")
        ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
        assert torch.equal(first, ctx.forward(q, k, v))
        ctx.check()
    finally:
        ctx.destroy()


def test_output_guard_bands_are_untouched():
    """The kernels must write exactly B*H*n*d elements: canaries on both sides of `out` survive."""
    x = small_inputs(1, 2, 1000, 128, torch.bfloat16, seed=11)
    B, H, n, d = x["q"].shape
    pad = 4096
    buf = torch.full((pad + B * H * n * d + pad,), 7.0, dtype=torch.bfloat16, device="cuda")
    out = buf[pad:pad + B * H * n * d].view(B, H, n, d)
    ctx = linattn.LinAttn(H, d, max_B=B, max_n=n)
    try:
        for mode in MODES:
            ctx.set_option(linattn.OPT_PATH, mode[0])
            ctx.set_option(linattn.OPT_FUSE, mode[1])
            ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
            ctx.forward(x["q"].cuda(), x["k"].cuda(), x["v"].cuda(), out=out)
            ctx.check()
            assert (buf[:pad] == 7.0).all() and (buf[-pad:] == 7.0).all()
            assert_parity(out.cpu().double().numpy(), oracle_out(x), "guarded output")
    finally:
        ctx.destroy()


@pytest.mark.parametrize("B,H,n,d,dtype", [(1, 2, 1500, 128, torch.bfloat16), (2, 3, 700, 128, torch.bfloat16),
                                           (2, 2, 300, 64, torch.float32)])
def test_host_buffer_entry_point(B, H, n, d, dtype):
    """Host buffers in, host buffer out; inside, the (b,h) pairs are pipelined one by one over three streams."""
    x = small_inputs(B, H, n, d, dtype, seed=12 + B)
    ctx = linattn.LinAttn(H, d, max_B=B, max_n=n)
    try:
        ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
        want, S_ref, z_ref = oracle.ref_linear(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], return_state=True)
        host_out = torch.empty_like(x["q"])
        ctx.forward_host(x["q"], x["k"], x["v"], host_out)          # pageable memory
        ctx.check()
        assert_parity(host_out.double().numpy(), want, "host entry point")
        S, z = ctx.read_state(B)
        assert errors(S.double().numpy(), S_ref)[0] <= 5e-3 and errors(z.double().numpy(), z_ref)[0] <= 5e-3
        pin = {k_: x[k_].pin_memory() for k_ in ("q", "k", "v")}
        host_out2 = torch.empty_like(x["q"]).pin_memory()
        for _ in range(3):                                              # pinned memory: the copies overlap
            host_out2.zero_()
            ctx.forward_host(pin["q"], pin["k"], pin["v"], host_out2)
            assert torch.equal(host_out, host_out2)
        # the device entry point on the same context afterwards is undisturbed
        dev = ctx.forward(x["q"].cuda(), x["k"].cuda(), x["v"].cuda()).cpu()
        ctx.check()
        assert_parity(dev.double().numpy(), want, "device entry point after the host one")
        rel, _ = errors(host_out.double().numpy(), dev.double().numpy())
        assert rel <= 5e-3
        # token-major layout: one piece
        ctx.set_option(linattn.OPT_LAYOUT, linattn.LAYOUT_BNHD)
        tm = lambda t: t.permute(0, 2, 1, 3).contiguous().view(B, H, n, d)
        host_out3 = torch.empty_like(x["q"])
        ctx.forward_host(tm(x["q"]), tm(x["k"]), tm(x["v"]), host_out3)
        assert torch.equal(host_out3.view(B, n, H, d).permute(0, 2, 1, 3), dev)
    finally:
        ctx.destroy()


def test_which_kernels_run():
    """bf16 activations -> the tensor-core kernels (one fused launch by default); fp32 activations -> CUDA cores."""
    x = small_inputs(1, 2, 700, 128, torch.bfloat16, seed=14)
    ctx = linattn.LinAttn(2, 128, max_B=1, max_n=700)
    try:
        ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
        q, k, v = x["q"].cuda(), x["k"].cuda(), x["v"].cuda()

        def names(path, fuse):
            ctx.set_option(linattn.OPT_PATH, path)
            ctx.set_option(linattn.OPT_FUSE, fuse)
            ctx.set_option(linattn.OPT_PROFILE, 1)
            ctx.forward(q, k, v)
            got = [kt["name"] for kt in ctx.kernel_times()]
            ctx.set_option(linattn.OPT_PROFILE, 0)
            return got, ctx.last_launch_count()

        assert names(linattn.PATH_AUTO, 1) == (["linattn_fused_tc"], 1)
        assert names(linattn.PATH_TENSOR, 0) == (["kside_tc", "combine_tc", "qside_tc"], 3)
        assert names(linattn.PATH_SIMT, 1) == (["kside_simt", "combine_state", "qside_simt"], 3)
        ctx.check()
        # fp32 weights with bf16 activations stay on the tensor cores (the weights enter as a bf16 hi + lo pair)
        ctx.set_feature_map(x["Wq"].float().cuda(), x["Wk"].float().cuda())
        assert names(linattn.PATH_AUTO, 1) == (["linattn_fused_tc"], 1)
        ctx.check()
    finally:
        ctx.destroy()
    # fp32 activations have no tensor-core kernels: asking for them is an error, not a silent detour
    xf = small_inputs(1, 2, 700, 128, torch.float32, seed=14)
    ctx = linattn.LinAttn(2, 128, max_B=1, max_n=700)
    try:
        ctx.set_feature_map(xf["Wq"].cuda(), xf["Wk"].cuda())
        qf, kf, vf = xf["q"].cuda(), xf["k"].cuda(), xf["v"].cuda()
        lib = linattn.load_library()
        ctx.set_option(linattn.OPT_PATH, linattn.PATH_TENSOR)
        assert lib.linattn_forward(ctx._h, qf.data_ptr(), kf.data_ptr(), vf.data_ptr(), torch.empty_like(qf).data_ptr(),
                                   1, 2, 700, 128, linattn.F32, None) == linattn.ERR_UNSUPPORTED
    finally:
        ctx.destroy()


@pytest.mark.parametrize("d", [128, 64])
@pytest.mark.parametrize("scale", [1.0, 40.0])
def test_fp32_feature_map_weights_on_the_tensor_cores(d, scale):
    """Weights given in fp32 that are NOT bf16 values: the oracle gets the fp32 weights, the kernels a bf16 hi + lo pair.
    With logits of magnitude ~50 (scale 40) weights rounded once to bf16 would be off by several per cent in phi."""
    g = torch.Generator().manual_seed(77 + d)
    B, H, n = 2, 3, 1500
    sx = 1.0 / math.sqrt(d)
    q, k, v = (torch.randn(B, H, n, d, generator=g).mul_(sx).bfloat16() for _ in range(3))
    Wq, Wk = (torch.randn(H, d, d // 2, generator=g).mul_(scale / (math.sqrt(d) * sx)) for _ in range(2))   # fp32, full mantissas
    assert not torch.equal(Wq.bfloat16().float(), Wq)
    want = oracle.ref_linear(q, k, v, Wq, Wk)
    ctx = linattn.LinAttn(H, d, max_B=B, max_n=n)
    try:
        ctx.set_feature_map(Wq.cuda(), Wk.cuda())
        for fuse in (1, 0):
            ctx.set_option(linattn.OPT_FUSE, fuse)
            out = ctx.forward(q.cuda(), k.cuda(), v.cuda())
            ctx.check()
            assert ctx.last_launch_count() == (1 if fuse else 3)
            assert_parity(out.cpu().double().numpy(), want, f"fp32 weights, d={d}, scale {scale}, fuse={fuse}")
        # the same weights after a switch to bf16 values and back
        ctx.set_feature_map(Wq.bfloat16().cuda(), Wk.bfloat16().cuda())
        out_b = ctx.forward(q.cuda(), k.cuda(), v.cuda())
        ctx.check()
        assert_parity(out_b.cpu().double().numpy(), oracle.ref_linear(q, k, v, Wq.bfloat16(), Wk.bfloat16()), "bf16 weights afterwards")
    finally:
        ctx.destroy()


# ---- argument checking on a live context (host-side; nothing invalid reaches a kernel) ------------------

def test_forward_argument_errors():
    lib = linattn.load_library()
    x = small_inputs(1, 2, 256, 128, torch.bfloat16, seed=13)
    q, k, v = x["q"].cuda(), x["k"].cuda(), x["v"].cuda()
    out = torch.empty_like(q)
    ctx = linattn.LinAttn(2, 128, max_B=1, max_n=256)
    try:
        def fwd(qp, kp, vp, op, B=1, H=2, n=256, d=128, dt=linattn.BF16):
            return lib.linattn_forward(ctx._h, qp, kp, vp, op, B, H, n, d, dt, None)
        P = (q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr())
        assert fwd(*P) == linattn.ERR_NO_FEATURE_MAP
        ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
        assert fwd(*P) == linattn.OK
        assert fwd(None, P[1], P[2], P[3]) == linattn.ERR_INVALID_ARG
        assert fwd(P[0] + 2, P[1], P[2], P[3]) == linattn.ERR_INVALID_ARG       # misaligned
        assert fwd(P[0], P[1], P[2], P[0]) == linattn.ERR_INVALID_ARG           # out aliases q
        assert fwd(*P, H=3) == linattn.ERR_INVALID_ARG
        assert fwd(*P, d=64) == linattn.ERR_INVALID_ARG
        assert fwd(*P, d=96) == linattn.ERR_UNSUPPORTED
        assert fwd(*P, dt=7) == linattn.ERR_UNSUPPORTED
        assert fwd(*P, n=0) == linattn.ERR_INVALID_ARG
        assert fwd(*P, n=257) == linattn.ERR_WORKSPACE
        assert fwd(*P, B=2) == linattn.ERR_WORKSPACE
        assert lib.linattn_set_option(ctx._h, 99, 0) == linattn.ERR_INVALID_ARG
        assert lib.linattn_set_option(ctx._h, linattn.OPT_SPLITS, -1) == linattn.ERR_INVALID_ARG
        ctx.check()
    finally:
        ctx.destroy()


def _fused_ctas(G, T, sms=148):
    """CTAs of the fused kernel (mirrors the library's rule: one per SM, or the same number per (b,h) pair when that
    uses at least 95 % of the SMs)."""
    if T <= sms:
        return T
    per_pair = sms // G
    return G * per_pair if per_pair >= 1 and G * per_pair * 100 >= 95 * sms else sms


@pytest.mark.parametrize("H,n", [(10, 2432), (10, 2688), (20, 1280), (20, 1536), (40, 768)])
def test_run_whose_first_piece_is_shorter_than_the_query_ring(H, n):
    """Shapes for which some CTA of the fused kernel starts one to four tiles before a head boundary and goes on into
    the next head: the first head's S, z must be fetched before the second head's are waited for."""
    Tn = (n + 127) // 128
    T = H * Tn
    P = _fused_ctas(H, T)
    assert T >= P
    short = [c for c in range(P) if (c * T // P) % Tn != 0 and Tn - (c * T // P) % Tn < 5 and (c + 1) * T // P > c * T // P + Tn - (c * T // P) % Tn]
    assert short, "the shape no longer exercises the case (148 SMs assumed)"
    x = small_inputs(1, H, n, 128, torch.bfloat16, seed=40 + H)
    ctx = linattn.LinAttn(H, 128, max_B=1, max_n=n)
    try:
        ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
        out = ctx.forward(x["q"].cuda(), x["k"].cuda(), x["v"].cuda())
        ctx.check()
        assert ctx.last_launch_count() == 1
        want = oracle.ref_linear(x["q"], x["k"], x["v"], x["Wq"], x["Wk"])
        assert_parity(out.cpu().double().numpy(), want, f"H={H} n={n}")
    finally:
        ctx.destroy()


def test_fused_kernel_equals_the_three_launch_form_over_many_tile_splits():
    """The fused kernel and the three-launch form split the tiles in the same way and sum the partials in the same
    order, so their outputs must agree bit for bit.  Swept over head counts and lengths that give every kind of run:
    one tile per CTA, runs inside a head, runs that cross one or several head boundaries at any offset, ragged tails."""
    dev = torch.device("cuda", 0)
    g = torch.Generator(device=dev).manual_seed(123)
    checked = 0
    for G in (1, 2, 3, 5, 7, 10, 13, 20, 37, 40, 41, 50, 75, 149):
        for Tn in (1, 2, 3, 4, 5, 6, 7, 9, 13, 21, 33):
            if G * Tn > 3000:
                continue
            n = Tn * 128 - (17 if Tn % 2 else 0)
            q, k, v = (torch.randn(1, G, n, 128, generator=g, device=dev).mul_(1 / math.sqrt(128)).bfloat16() for _ in range(3))
            Wq, Wk = (torch.randn(G, 128, 64, generator=g, device=dev).bfloat16() for _ in range(2))
            ctx = linattn.LinAttn(G, 128, max_B=1, max_n=n)
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
                assert ctx.last_launch_count() == 3
                assert torch.isfinite(fused.float()).all(), f"G={G} tiles per head={Tn}"
                assert torch.equal(fused, unfused), f"G={G} tiles per head={Tn}"
                assert torch.equal(fused_mixed, unfused_mixed), f"mixed attention, G={G} tiles per head={Tn}"
                checked += 1
            finally:
                ctx.destroy()
    assert checked > 100
