"""Helpers shared by the GPU parity tests: error metrics and running both sides on one input set."""
import numpy as np
import torch

REL_L2_TOL = 5e-3   # || o_gpu - o_ref ||_2 / || o_ref ||_2 over the whole tensor
MAX_ABS_TOL = 2e-2  # max | o_gpu - o_ref |


def errors(got, want):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    diff = got - want
    denom = np.sqrt((want ** 2).sum())
    rel = np.sqrt((diff ** 2).sum()) / (denom if denom > 0 else 1.0)
    return float(rel), float(np.abs(diff).max())


def assert_parity(got, want, what=""):
    assert np.isfinite(np.asarray(got, dtype=np.float64)).all(), f"{what}: non-finite output"
    rel, mx = errors(got, want)
    assert rel <= REL_L2_TOL and mx <= MAX_ABS_TOL, f"{what}: rel-L2 {rel:.3e} (tol {REL_L2_TOL}), max-abs {mx:.3e} (tol {MAX_ABS_TOL})"
    return rel, mx


def run_gpu(x, path=0, splits=0, ctx=None, return_state=False, fuse=1):
    """Run the CUDA library on the CPU tensors of `x` (q, k, v, Wq, Wk); returns a CPU float64 array."""
    from paper_2510_08318_b200 import linattn
    q = x["q"]
    B, H, n, d = q.shape
    own = ctx is None
    if own:
        ctx = linattn.LinAttn(H, d, max_B=B, max_n=n)
    try:
        ctx.set_option(linattn.OPT_PATH, path)
        ctx.set_option(linattn.OPT_SPLITS, splits)
        ctx.set_option(linattn.OPT_FUSE, fuse)
        ctx.set_feature_map(x["Wq"].cuda(), x["Wk"].cuda())
        out = ctx.forward(q.cuda(), x["k"].cuda(), x["v"].cuda())
        ctx.check()
        res = out.cpu().double().numpy()
        if return_state:
            S, z = ctx.read_state(B)
            return res, S.double().numpy(), z.double().numpy()
        return res
    finally:
        if own:
            ctx.destroy()
