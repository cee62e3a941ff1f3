"""Helpers shared by the GPU parity tests: error metrics and running both sides on one input set."""
import numpy as np
import torch

REL_L2_TOL = 5e-3   # || o_gpu - o_ref ||_2 / || o_ref ||_2 over the whole tensor
MAX_ABS_TOL = 2e-2  # max | o_gpu - o_ref |, absolute, and also relative to max | o_ref | (see assert_parity)
ROW_FACTOR = 8.0    # no single row (last axis) may be off by more than ROW_FACTOR * REL_L2_TOL of its own norm


def errors(got, want):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    diff = got - want
    denom = np.sqrt((want ** 2).sum())
    rel = np.sqrt((diff ** 2).sum()) / (denom if denom > 0 else 1.0)
    return float(rel), float(np.abs(diff).max())


def row_errors(got, want):
    """Relative L2 error of every row (last axis) against its own reference norm.  Rows whose reference norm is
    below a tenth of the root-mean-square row norm are measured against that floor instead (a nearly cancelled
    row has no scale of its own).  Returns (worst ratio, flat index of that row)."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    d = want.shape[-1]
    err = np.sqrt(((got - want) ** 2).reshape(-1, d).sum(-1))
    nrm = np.sqrt((want ** 2).reshape(-1, d).sum(-1))
    floor = 0.1 * np.sqrt((nrm ** 2).mean())
    ratio = err / np.maximum(np.maximum(nrm, floor), 1e-300)
    i = int(ratio.argmax())
    return float(ratio[i]), i


def assert_parity(got, want, what="", rows=True):
    """The stated tolerances (relative L2 over the tensor, absolute max-abs), made to bite at the workloads' scale:
    outputs of the long-sequence workloads are ~5e-4 in magnitude, so the absolute max-abs bound alone would accept an
    all-zero tensor, and one relative L2 over 4e5 rows would accept a handful of completely wrong rows.  Hence also
    max-abs <= MAX_ABS_TOL * max|reference| and a relative L2 bound on every single row."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, f"{what}: shape {got.shape} vs {want.shape}"
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    rel, mx = errors(got, want)
    scale = float(np.abs(want).max())
    assert rel <= REL_L2_TOL and mx <= MAX_ABS_TOL, f"{what}: rel-L2 {rel:.3e} (tol {REL_L2_TOL}), max-abs {mx:.3e} (tol {MAX_ABS_TOL})"
    assert mx <= MAX_ABS_TOL * scale, f"{what}: max-abs {mx:.3e} exceeds {MAX_ABS_TOL} * max|reference| = {MAX_ABS_TOL * scale:.3e}"
    if rows and want.ndim >= 2:
        worst, idx = row_errors(got, want)
        assert worst <= ROW_FACTOR * REL_L2_TOL, (f"{what}: row {idx} (flattened over the leading axes) has relative L2 error "
                                                  f"{worst:.3e} > {ROW_FACTOR * REL_L2_TOL:.1e}")
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
