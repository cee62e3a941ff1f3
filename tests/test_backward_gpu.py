"""GPU parity of linattn_backward against the oracle's gradients (the chain rule through Eq. 5 and Eq. 6, which
is what the objective of Eq. 14 back-propagates through a linear-attention layer).

Both sides get the same stored (rounded) q, k, v, dO and weights.  Gradients have no natural scale (dv is of
order |dO| / n), so the absolute bound is taken relative to the largest reference entry: relative L2 <= 5e-3
over each gradient tensor and max-abs <= 2e-2 * max|reference|.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2510_08318_b200 import linattn
from util import errors

pytestmark = pytest.mark.gpu

NAMES = ("dq", "dk", "dv", "dWq", "dWk")


def _inputs(B, H, n, d, dtype, seed, shared=False):
    g = torch.Generator().manual_seed(seed)
    sx = 1.0 / math.sqrt(d)
    q, k, v = (torch.randn(B, H, n, d, generator=g) * sx for _ in range(3))
    wshape = (d, d // 2) if shared else (H, d, d // 2)
    Wq, Wk = (torch.randn(*wshape, generator=g) / (math.sqrt(d) * sx) for _ in range(2))
    dout = torch.randn(B, H, n, d, generator=g)
    return {"q": q.to(dtype), "k": k.to(dtype), "v": v.to(dtype), "Wq": Wq.to(dtype), "Wk": Wk.to(dtype),
            "dout": dout.to(dtype)}


def _assert_grads(got, want, what):
    for name, a, b in zip(NAMES, got, want):
        a = a.detach().cpu().double().numpy()
        assert np.isfinite(a).all(), f"{what}: {name} has non-finite entries"
        rel, mx = errors(a, b)
        scale = float(np.abs(b).max())
        assert rel <= 5e-3 and mx <= 2e-2 * scale, f"{what}: {name} rel-L2 {rel:.3e}, max-abs {mx:.3e} (largest reference entry {scale:.3e})"


PATHS = [linattn.PATH_AUTO, linattn.PATH_SIMT]
PATH_IDS = ["auto", "simt"]


def _tensor_core(x, path):
    return path != linattn.PATH_SIMT and x["q"].dtype == torch.bfloat16 and x["q"].shape[-1] == 128


def _run(x, per_head=True, layout=linattn.LAYOUT_BHND, path=linattn.PATH_AUTO):
    B, H, n, d = x["q"].shape
    ctx = linattn.LinAttn(H, d, max_B=B, max_n=n)
    try:
        ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
        ctx.set_option(linattn.OPT_LAYOUT, layout)
        ctx.set_option(linattn.OPT_PATH, path)
        args = [x[s].cuda() for s in ("q", "k", "v", "dout")]
        if layout == linattn.LAYOUT_BNHD:
            args = [t.permute(0, 2, 1, 3).contiguous().view(B, H, n, d) for t in args]
        got = ctx.backward(*args, per_head=per_head)
        again = ctx.backward(*args, per_head=per_head)
        ctx.check()
        assert ctx.last_launch_count() == (6 if _tensor_core(x, path) else 7)   # tensor-core kernels for bf16, d = 128
        for a, b in zip(got, again):
            assert torch.equal(a, b), "the gradients are not bit-reproducible"
        if layout == linattn.LAYOUT_BNHD:
            got = tuple(t.view(B, n, H, d).permute(0, 2, 1, 3) for t in got[:3]) + tuple(got[3:])
        return got, ctx.read_state(B)
    finally:
        ctx.destroy()


@pytest.mark.parametrize("B,H,n,d,dtype", [
    (2, 2, 300, 64, torch.float32),      # several chunks and a ragged tail
    (1, 3, 257, 128, torch.float32),
    (2, 2, 1000, 128, torch.bfloat16),
    (1, 2, 129, 64, torch.bfloat16),
    (1, 1, 1, 128, torch.float32),       # one token: o = v, so dq = dk = 0 and dv = dO
    (3, 1, 31, 64, torch.float32),       # less than one chunk
    (1, 12, 2048, 128, torch.bfloat16),  # the small workload's shape
    (1, 1, 1, 128, torch.bfloat16),
    (2, 5, 700, 128, torch.bfloat16),    # more heads than one CTA's run covers: segments of several heads per CTA
    (1, 2, 33000, 128, torch.bfloat16),  # runs of many tiles per CTA
    (2, 20, 1500, 128, torch.bfloat16),  # three to four tiles per CTA and twelve per head: most runs cross into another head
])
@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_gradients_match_the_oracle(B, H, n, d, dtype, path):
    x = _inputs(B, H, n, d, dtype, seed=200 + n)
    want = oracle.ref_backward(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], x["dout"])
    got, (S, z) = _run(x, path=path)
    if n == 1:
        # o = v whatever q and k are: every gradient but dv vanishes, so only absolute checks make sense
        for name, t in zip(NAMES, got):
            if name != "dv":
                # (bf16, tensor-core kernels: what is left of the cancellation dO S^T - (dO . o) z with S as a bf16 hi + lo pair)
                assert float(t.abs().max()) <= (1e-5 if dtype == torch.float32 else 2e-3), f"{name} must vanish for a single token"
        assert torch.allclose(got[2].cpu().float(), x["dout"].float(), rtol=1e-6 if dtype == torch.float32 else 1e-2, atol=0)
        assert np.abs(want[2] - x["dout"].double().numpy()).max() <= 1e-12
        return
    _assert_grads(got, want, f"B={B} H={H} n={n} d={d} {dtype}")
    # the call leaves the forward state of these k, v in the context
    _, S_ref, z_ref = oracle.ref_linear(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], rows=np.array([0]), return_state=True)
    assert errors(S.double().numpy(), S_ref)[0] <= 5e-3 and errors(z.double().numpy(), z_ref)[0] <= 5e-3


@pytest.mark.parametrize("d,dtype", [(64, torch.float32), (128, torch.bfloat16)])
def test_shared_feature_map_sums_the_weight_gradients_over_heads(d, dtype):
    x = _inputs(2, 3, 200, d, dtype, seed=31, shared=True)
    want = oracle.ref_backward(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], x["dout"])
    got, _ = _run(x, per_head=False)
    assert tuple(got[3].shape) == (d, d // 2)
    _assert_grads(got, want, "shared map")


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_token_major_layout(path):
    x = _inputs(2, 3, 333, 128, torch.bfloat16, seed=32)
    ref, _ = _run(x, path=path)
    got, _ = _run(x, layout=linattn.LAYOUT_BNHD, path=path)
    for name, a, b in zip(NAMES, got, ref):
        assert torch.equal(a, b), f"{name}: the [B][n][H][d] layout must give the same bits"


def test_heavy_tailed_keys():
    """Keys with a few large entries (the recipe of the heavy-tailed workload) make phi(k) nearly one-hot."""
    x = _inputs(1, 2, 600, 128, torch.bfloat16, seed=33)
    g = torch.Generator().manual_seed(34)
    k = x["k"].float()
    mask = torch.rand(k.shape, generator=g) < 0.01
    x["k"] = torch.where(mask, k * 12.0, k).to(torch.bfloat16)
    want = oracle.ref_backward(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], x["dout"])
    for path in PATHS:
        got, _ = _run(x, path=path)
        _assert_grads(got, want, f"heavy-tailed keys, path {path}")


def test_values_with_a_large_mean():
    """V with a mean of three standard deviations: dphi(q) = S dnum + dden z then is a small difference of large
    terms, which is why the tensor-core path carries S, dS and dnum as bf16 hi + lo pairs."""
    x = _inputs(1, 2, 1500, 128, torch.bfloat16, seed=37)
    x["v"] = (x["v"].float() + 3.0 / math.sqrt(128)).to(torch.bfloat16)
    want = oracle.ref_backward(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], x["dout"])
    for path in PATHS:
        got, _ = _run(x, path=path)
        _assert_grads(got, want, f"V with a large mean, path {path}")


def test_config2_full_size_two_heads_against_the_oracle():
    """Full size of the headline workload.  The heads are independent, so the oracle's gradients for two of the
    twelve heads (computed on those heads alone) pin the corresponding slices of the full-size result."""
    from paper_2510_08318_b200 import synth
    x = synth.make_inputs(2)
    B, H, n, d = x["q"].shape
    x["dout"] = torch.randn(B, H, n, d, generator=torch.Generator().manual_seed(36)).to(x["q"].dtype)
    got, _ = _run(x)
    for h in (0, 7):
        sl = {s: x[s][:, h:h + 1].contiguous() for s in ("q", "k", "v", "dout")}
        want = oracle.ref_backward(sl["q"], sl["k"], sl["v"], x["Wq"][h:h + 1].contiguous(), x["Wk"][h:h + 1].contiguous(), sl["dout"])
        mine = tuple(t[:, h:h + 1] for t in got[:3]) + tuple(t[h:h + 1] for t in got[3:])
        _assert_grads(mine, want, f"config 2, head {h}")


def test_state_left_by_the_forward_is_reused_only_when_it_belongs_to_the_same_problem():
    x = _inputs(1, 3, 900, 128, torch.bfloat16, seed=38)
    y = _inputs(1, 3, 900, 128, torch.bfloat16, seed=39)
    ctx = linattn.LinAttn(3, 128, max_B=1, max_n=900)
    try:
        ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
        dx = [x[s].cuda() for s in ("q", "k", "v", "dout")]
        dy = [y[s].cuda() for s in ("q", "k", "v", "dout")]
        ref_x = ctx.backward(*dx)
        ref_y = ctx.backward(*dy)
        assert ctx.last_launch_count() == 6
        ctx.set_option(linattn.OPT_REUSE_STATE, 1)
        ctx.forward(dx[0], dx[1], dx[2])
        got = ctx.backward(*dx)                       # same k, v as the forward: S, z are taken over
        assert ctx.last_launch_count() == 4
        for a, b in zip(got, ref_x):
            assert torch.equal(a, b)
        got = ctx.backward(*dy)                       # other k, v: recomputed
        assert ctx.last_launch_count() == 6
        for a, b in zip(got, ref_y):
            assert torch.equal(a, b)
        got = ctx.backward(*dy)                       # the backward's own state counts too
        assert ctx.last_launch_count() == 4
        for a, b in zip(got, ref_y):
            assert torch.equal(a, b)
        ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())   # new weights: nothing is taken over
        ctx.backward(*dy)
        assert ctx.last_launch_count() == 6
        ctx.forward(dx[0], dx[1], dx[2])
        ctx.set_option(linattn.OPT_REUSE_STATE, 0)
        ctx.backward(*dx)
        assert ctx.last_launch_count() == 6
        ctx.check()
    finally:
        ctx.destroy()
    # a forward that ran before the backward's workspace existed left no lo image of S: the first backward makes it
    fresh = linattn.LinAttn(3, 128, max_B=1, max_n=900)
    try:
        fresh.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
        fresh.set_option(linattn.OPT_REUSE_STATE, 1)
        fresh.forward(dx[0], dx[1], dx[2])
        got = fresh.backward(*dx)
        assert fresh.last_launch_count() == 5
        for a, b in zip(got, ref_x):
            assert torch.equal(a, b)
        fresh.forward(dx[0], dx[1], dx[2])
        got = fresh.backward(*dx)
        assert fresh.last_launch_count() == 4
        for a, b in zip(got, ref_x):
            assert torch.equal(a, b)
        fresh.check()
    finally:
        fresh.destroy()


@pytest.mark.parametrize("n", [1000, 2700])   # a ragged last tile; about one and about three tiles per CTA
def test_gradient_guard_bands_are_untouched(n):
    """dq, dk, dv are written by TMA stores that clip at the end of the sequence, the weight gradients by a kernel of
    their own: canaries on both sides of every output buffer must survive (called through the C-ABI, which takes the
    output pointers as they are)."""
    B, H, d = 2, 3, 128
    x = _inputs(B, H, n, d, torch.bfloat16, seed=300 + n)
    want = oracle.ref_backward(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], x["dout"])
    pad = 4096

    def guarded(numel, dtype):
        buf = torch.full((pad + numel + pad,), 7.0, dtype=dtype, device="cuda")
        return buf, buf[pad:pad + numel]

    bufs = [guarded(B * H * n * d, torch.bfloat16) for _ in range(3)] + [guarded(H * d * (d // 2), torch.float32) for _ in range(2)]
    ctx = linattn.LinAttn(H, d, max_B=B, max_n=n)
    try:
        ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
        q, k, v, dout = (x[s].cuda() for s in ("q", "k", "v", "dout"))
        st = ctx._lib.linattn_backward(ctx._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), dout.data_ptr(),
                                       *[inner.data_ptr() for _, inner in bufs], 1, B, H, n, d, linattn.BF16,
                                       torch.cuda.current_stream().cuda_stream)
        assert st == linattn.OK
        ctx.check()
        assert ctx.last_launch_count() == 6
        for buf, _ in bufs:
            assert (buf[:pad] == 7.0).all() and (buf[-pad:] == 7.0).all(), "a gradient kernel wrote outside its output"
        got = [bufs[i][1].view(B, H, n, d) for i in range(3)] + [bufs[i][1].view(H, d, d // 2) for i in (3, 4)]
        _assert_grads(got, want, f"guarded outputs, n={n}")
    finally:
        ctx.destroy()


def test_argument_errors():
    lib = linattn.load_library()
    x = _inputs(1, 2, 128, 64, torch.float32, seed=35)
    ctx = linattn.LinAttn(2, 64, max_B=1, max_n=128)
    try:
        ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
        q, k, v, g = (x[s].cuda() for s in ("q", "k", "v", "dout"))
        dq, dk, dv = (torch.empty_like(q) for _ in range(3))
        dWq, dWk = (torch.empty(2, 64, 32, device="cuda") for _ in range(2))

        def call(**kw):
            a = dict(q=q.data_ptr(), k=k.data_ptr(), v=v.data_ptr(), g=g.data_ptr(), dq=dq.data_ptr(), dk=dk.data_ptr(),
                     dv=dv.data_ptr(), dWq=dWq.data_ptr(), dWk=dWk.data_ptr(), n=128)
            a.update(kw)
            return lib.linattn_backward(ctx._h, a["q"], a["k"], a["v"], a["g"], a["dq"], a["dk"], a["dv"], a["dWq"],
                                        a["dWk"], 1, 1, 2, a["n"], 64, linattn.F32, None)
        assert call() == linattn.OK
        assert call(g=None) == linattn.ERR_INVALID_ARG
        assert call(dWk=None) == linattn.ERR_INVALID_ARG
        assert call(dk=dq.data_ptr()) == linattn.ERR_INVALID_ARG          # two outputs in one buffer
        assert call(dv=g.data_ptr()) == linattn.ERR_INVALID_ARG           # an output over an input
        assert call(dq=dq.data_ptr() + 4) == linattn.ERR_INVALID_ARG      # misaligned
        assert call(dWk=dWq.data_ptr()) == linattn.ERR_INVALID_ARG
        assert call(n=129) == linattn.ERR_WORKSPACE
        ctx.check()
    finally:
        ctx.destroy()
