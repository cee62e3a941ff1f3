"""linattn_forward_noalloc, the entry point for callers that cannot allocate device memory
(a plug-in inside someone else's memory pool, a serving thread that must not trigger
cudaMalloc's device-wide synchronisation).  Its scratch is a fixed device array shared by all
calls, so the test makes two different calls in a row and checks each against the ordinary
context-based entry point and against the fp64 CPU oracle (the context entry point runs the
same CUDA-core kernels, so agreement with it alone would not catch a fault they share).
Collected last on purpose (file name), so a failure here cannot hide any other test in a run
that stops at the first failure."""
import math

import pytest
import torch

import oracle
from paper_2510_08318_b200 import linattn
from util import assert_parity

pytestmark = pytest.mark.gpu


def _inputs(B, H, n, d, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    sx = 1.0 / math.sqrt(d)
    q, k, v = (torch.randn(B, H, n, d, generator=g).mul_(sx).to(dtype).cuda() for _ in range(3))
    # weights rounded to bf16 values so both entry points see identical numbers, held as fp32
    Wq, Wk = (torch.randn(H, d, d // 2, generator=g).div_(math.sqrt(d) * sx).bfloat16().float().cuda() for _ in range(2))
    return q, k, v, Wq, Wk


def _with_context(q, k, v, Wq, Wk):
    B, H, n, d = q.shape
    ctx = linattn.LinAttn(H, d, max_B=B, max_n=n)
    try:
        ctx.set_option(linattn.OPT_PATH, linattn.PATH_SIMT)
        ctx.set_feature_map(Wq, Wk)
        out = ctx.forward(q, k, v)
        ctx.check()
        return out
    finally:
        ctx.destroy()


def test_two_calls_in_a_row_match_the_context_entry_point():
    lib = linattn.load_library()
    # call 1: bf16, d = 128, ragged length; call 2: a different shape and type on the same scratch
    for (B, H, n, d, dtype, seed) in [(1, 4, 3001, 128, torch.bfloat16, 21), (2, 3, 777, 64, torch.float32, 22)]:
        q, k, v, Wq, Wk = _inputs(B, H, n, d, dtype, seed)
        out = torch.full_like(q, float("nan"))
        linattn.forward_noalloc(q, k, v, Wq, Wk, out)
        torch.cuda.synchronize()
        want = _with_context(q, k, v, Wq, Wk)
        assert_parity(out.double().cpu().numpy(), want.double().cpu().numpy(), f"noalloc B={B} H={H} n={n} d={d}")
        ref = oracle.ref_linear(q.cpu(), k.cpu(), v.cpu(), Wq.cpu(), Wk.cpu())
        assert_parity(out.double().cpu().numpy(), ref, f"noalloc vs the oracle, B={B} H={H} n={n} d={d}")
    # shared weights ([d, d/2]) on the same scratch again
    q, k, v, Wq, Wk = _inputs(1, 2, 500, 128, torch.bfloat16, 23)
    out = torch.empty_like(q)
    linattn.forward_noalloc(q, k, v, Wq[0].contiguous(), Wk[0].contiguous(), out)
    want = _with_context(q, k, v, Wq[0].contiguous(), Wk[0].contiguous())
    assert_parity(out.double().cpu().numpy(), want.double().cpu().numpy(), "noalloc shared weights")
    assert_parity(out.double().cpu().numpy(), oracle.ref_linear(q.cpu(), k.cpu(), v.cpu(), Wq[0].cpu(), Wk[0].cpu()),
                  "noalloc shared weights vs the oracle")
    # out may not overlap an input: refused before anything is launched
    st = lib.linattn_forward_noalloc(q.data_ptr(), k.data_ptr(), v.data_ptr(), q.data_ptr(), Wq.data_ptr(), Wk.data_ptr(),
                                     1, 1, 2, 500, 128, linattn.BF16, None)
    assert st == linattn.ERR_INVALID_ARG
    # beyond the fixed scratch: B*H = 17 > 16 is refused with the workspace error, nothing is launched
    q, k, v, Wq, Wk = _inputs(1, 17, 64, 64, torch.bfloat16, 24)
    st = lib.linattn_forward_noalloc(q.data_ptr(), k.data_ptr(), v.data_ptr(), torch.empty_like(q).data_ptr(),
                                     Wq.data_ptr(), Wk.data_ptr(), 1, 1, 17, 64, 64, linattn.BF16, None)
    assert st == linattn.ERR_WORKSPACE and "workspace" in linattn.status_string(st)
    torch.cuda.synchronize()
