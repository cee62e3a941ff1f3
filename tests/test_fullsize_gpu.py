"""GPU parity at the full sizes of the bf16 workloads, in the launch configuration the benchmark times
(automatic path: one fused tensor-core kernel per forward).

Config 2 is compared element by element over the whole output.  For the larger ones the oracle computes
S and z over all keys and the outputs of a sample of query rows (right-hand form of Eq. 5), and 64 sampled
rows per (batch, head) are also checked against the O(n^2) definition (left-hand form) at every one of the
four workloads; S and z themselves are compared in full.  Tolerances as everywhere (util.assert_parity):
relative L2 <= 5e-3, max-abs <= 2e-2 absolute and relative to max|reference|, every row within 8x the
relative-L2 tolerance of its own norm.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_08318_b200 import linattn, synth
from util import assert_parity, errors

pytestmark = pytest.mark.gpu


def _forward(x, ctx=None, repeat=1):
    B, H, n, d = x["q"].shape
    own = ctx is None
    if own:
        ctx = linattn.LinAttn(H, d, max_B=B, max_n=n)
    try:
        ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
        q, k, v = x["q"].cuda(), x["k"].cuda(), x["v"].cuda()
        out = ctx.forward(q, k, v)
        for _ in range(repeat - 1):
            again = ctx.forward(q, k, v)
            assert torch.equal(out, again), "the forward is not bit-reproducible"
        ctx.check()
        assert ctx.last_launch_count() == 1, "expected the fused tensor-core kernel"
        S, z = ctx.read_state(B)
        return out.cpu(), S.double().numpy(), z.double().numpy()
    finally:
        if own:
            ctx.destroy()


QUAD_ROWS = 64   # query rows per (batch, head) compared with the left-hand (O(n^2)) form of Eq. 5


def _sample_rows(n, count, seed):
    rng = np.random.default_rng(seed)
    rows = rng.choice(n, size=count, replace=False)
    rows[:4] = [0, 127, n - 128, n - 1]   # first tile, tile edge, start of the ragged tail tile, last token
    return np.sort(np.unique(rows))


def _check_sampled(x, out, S, z, rows_lin, rows_quad, what):
    want, S_ref, z_ref = oracle.ref_linear(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], rows=rows_lin, return_state=True)
    got = out[:, :, torch.from_numpy(rows_lin)].double().numpy()
    assert_parity(got, want, f"{what}: sampled rows vs right-hand form")
    rs, _ = errors(S, S_ref)
    rz, _ = errors(z, z_ref)
    assert rs <= 5e-3 and rz <= 5e-3, f"{what}: S rel-L2 {rs:.2e}, z rel-L2 {rz:.2e}"
    n = x["q"].shape[2]
    assert abs(z.sum(-1) - 2.0 * n).max() <= 2e-3 * 2.0 * n, "sum(z) must be 2n"
    want_q = oracle.ref_quadratic(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], rows=rows_quad)
    got_q = out[:, :, torch.from_numpy(rows_quad)].double().numpy()
    assert_parity(got_q, want_q, f"{what}: sampled rows vs the O(n^2) definition")


def test_config2_full_size_every_element():
    x = synth.make_inputs(2)
    out, S, z = _forward(x, repeat=3)
    want, S_ref, z_ref = oracle.ref_linear(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], return_state=True)
    assert_parity(out.double().numpy(), want, "config 2, whole output")
    assert errors(S, S_ref)[0] <= 5e-3 and errors(z, z_ref)[0] <= 5e-3
    rows = _sample_rows(x["q"].shape[2], QUAD_ROWS, seed=2)
    want_q = oracle.ref_quadratic(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], rows=rows)
    assert_parity(out[:, :, torch.from_numpy(rows)].double().numpy(), want_q, "config 2 vs the O(n^2) definition")


def test_config3_full_size_heavy_tailed_keys():
    x = synth.make_inputs(3)
    out, S, z = _forward(x)
    n = x["q"].shape[2]
    _check_sampled(x, out, S, z, _sample_rows(n, 512, seed=3), _sample_rows(n, QUAD_ROWS, seed=33), "config 3")


def test_config4_full_size_long_sequence():
    x = synth.make_inputs(4)
    out, S, z = _forward(x)
    n = x["q"].shape[2]
    _check_sampled(x, out, S, z, _sample_rows(n, 512, seed=4), _sample_rows(n, QUAD_ROWS, seed=44), "config 4")


def test_config5_full_size_two_layers_back_to_back():
    """Two of the thirty layers of the CFG-pair workload, each with its own context and feature map, enqueued
    back to back on one stream before anything is read back."""
    layers = [0, 29]
    xs = [synth.make_inputs(5, layer=l) for l in layers]
    B, H, n, d = xs[0]["q"].shape
    ctxs = [linattn.LinAttn(H, d, max_B=B, max_n=n) for _ in layers]
    try:
        dev = []
        for c, x in zip(ctxs, xs):
            c.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
            dev.append((x["q"].cuda(), x["k"].cuda(), x["v"].cuda()))
        outs = [c.forward(*t) for c, t in zip(ctxs, dev)]
        for c in ctxs:
            c.check()
        for l, x, o in zip(layers, xs, outs):
            want = oracle.ref_linear(x["q"], x["k"], x["v"], x["Wq"], x["Wk"])
            assert_parity(o.cpu().double().numpy(), want, f"config 5, layer {l}, whole output")
            rows = _sample_rows(n, QUAD_ROWS, seed=500 + l)
            want_q = oracle.ref_quadratic(x["q"], x["k"], x["v"], x["Wq"], x["Wk"], rows=rows)
            assert_parity(o.cpu()[:, :, torch.from_numpy(rows)].double().numpy(), want_q,
                          f"config 5, layer {l}, sampled rows vs the O(n^2) definition")
    finally:
        for c in ctxs:
            c.destroy()
