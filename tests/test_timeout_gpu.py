"""The bounded device-side waits, exercised without faulting anything: a test option makes the single-kernel forward
wait, where the CTAs that share a head meet, for one arrival more than will ever come, with the wait limit cut to a
millisecond.  The wait runs out, the kernel records where, unwinds (copies in flight land, tensor memory is freed) and
returns; the host reads the status.  The context must then be usable again and give the same bits as before.

The tensor-core backward gets the same treatment: one warp of every CTA leaves out one arrival that the warp issuing
the tensor-core products waits for, in the query-side or in the key-side kernel; every role of the kernel (issuer, store
warp, element-wise warps) has to notice, unwind and meet at the kernel's last barrier.

Also here: the forward recorded in a CUDA graph and replayed (its synchronisation counters are cleared by the kernel
itself, so a replay starts from the same state as a fresh launch)."""
import math

import pytest
import torch

from paper_2510_08318_b200 import linattn

pytestmark = pytest.mark.gpu


def _inputs(B, H, n, d, seed):
    g = torch.Generator().manual_seed(seed)
    sx = 1.0 / math.sqrt(d)
    q, k, v = (torch.randn(B, H, n, d, generator=g).mul_(sx).bfloat16().cuda() for _ in range(3))
    Wq, Wk = (torch.randn(H, d, d // 2, generator=g).div_(math.sqrt(d) * sx).bfloat16().cuda() for _ in range(2))
    return q, k, v, Wq, Wk


@pytest.mark.parametrize("H,n", [(2, 1024), (10, 2048)])   # one tile per CTA; 148 CTAs whose runs cross head boundaries
def test_a_wait_that_runs_out_is_reported_and_the_context_recovers(H, n):
    q, k, v, Wq, Wk = _inputs(1, H, n, 128, seed=n)
    ctx = linattn.LinAttn(H, 128, max_B=1, max_n=n)
    fresh = linattn.LinAttn(H, 128, max_B=1, max_n=n)
    try:
        ctx.set_feature_map(Wq, Wk)
        fresh.set_feature_map(Wq, Wk)
        ref = ctx.forward(q, k, v)
        ctx.check()
        assert ctx.last_launch_count() == 1, "the test is about the single-kernel forward"

        ctx.set_option(linattn.OPT_WAIT_LIMIT_US, 1000)
        ctx.set_option(linattn.OPT_TEST_UNMET_ARRIVAL, 1)
        ctx.forward(q, k, v)
        with pytest.raises(linattn.LinAttnError) as info:
            ctx.check()
        assert info.value.status == linattn.ERR_TIMEOUT
        assert "timed out" in str(info.value) and "gave up" in str(info.value)
        ctx.check()   # the error word was cleared by the check that reported it

        ctx.set_option(linattn.OPT_TEST_UNMET_ARRIVAL, 0)
        ctx.set_option(linattn.OPT_WAIT_LIMIT_US, 2_000_000)
        again = ctx.forward(q, k, v)
        ctx.check()
        assert torch.equal(again, ref), "the context must give the same bits after a timed-out launch"
        other = fresh.forward(q, k, v)
        fresh.check()
        assert torch.equal(again, other)
    finally:
        ctx.destroy()
        fresh.destroy()


@pytest.mark.parametrize("side", [2, 3])                    # query-side kernel, key-side kernel
@pytest.mark.parametrize("H,n", [(2, 1024), (3, 32768)])     # at most one tile per CTA; five or six tiles per CTA (the pipelined path)
def test_a_backward_wait_that_runs_out_is_reported_and_the_context_recovers(side, H, n):
    q, k, v, Wq, Wk = _inputs(1, H, n, 128, seed=n + side)
    g = torch.Generator().manual_seed(99)
    dout = torch.randn(1, H, n, 128, generator=g).bfloat16().cuda()
    ctx = linattn.LinAttn(H, 128, max_B=1, max_n=n)
    try:
        ctx.set_feature_map(Wq, Wk)
        ref = ctx.backward(q, k, v, dout)
        ctx.check()
        assert ctx.last_launch_count() == 6, "the test is about the tensor-core backward"

        ctx.set_option(linattn.OPT_WAIT_LIMIT_US, 1000)
        ctx.set_option(linattn.OPT_TEST_UNMET_ARRIVAL, side)
        ctx.backward(q, k, v, dout)
        with pytest.raises(linattn.LinAttnError) as info:
            ctx.check()
        assert info.value.status == linattn.ERR_TIMEOUT
        assert "gave up" in str(info.value)
        ctx.check()   # the error word was cleared by the check that reported it

        ctx.set_option(linattn.OPT_TEST_UNMET_ARRIVAL, 0)
        ctx.set_option(linattn.OPT_WAIT_LIMIT_US, 2_000_000)
        again = ctx.backward(q, k, v, dout)
        ctx.check()
        for x, y in zip(again, ref):
            assert torch.equal(x, y), "the context must give the same bits after a timed-out launch"
    finally:
        ctx.destroy()


def test_wait_limit_option_range():
    lib = linattn.load_library()
    ctx = linattn.LinAttn(2, 128, max_B=1, max_n=128)
    try:
        assert lib.linattn_set_option(ctx._h, linattn.OPT_WAIT_LIMIT_US, 0) == linattn.ERR_INVALID_ARG
        assert lib.linattn_set_option(ctx._h, linattn.OPT_WAIT_LIMIT_US, 10**9) == linattn.ERR_INVALID_ARG
        assert lib.linattn_set_option(ctx._h, linattn.OPT_TEST_UNMET_ARRIVAL, 4) == linattn.ERR_INVALID_ARG
        assert lib.linattn_set_option(ctx._h, linattn.OPT_WAIT_LIMIT_US, 5000) == linattn.OK
    finally:
        ctx.destroy()


def test_forward_recorded_in_a_cuda_graph_and_replayed():
    B, H, n, d = 1, 4, 5000, 128
    q, k, v, Wq, Wk = _inputs(B, H, n, d, seed=5)
    ctx = linattn.LinAttn(H, d, max_B=B, max_n=n)
    try:
        ctx.set_feature_map(Wq, Wk)
        out = torch.empty_like(q)
        ctx.forward(q, k, v, out=out)   # first call: function attributes are set outside any capture
        ctx.check()
        ref = out.clone()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            ctx.forward(q, k, v, out=out)
        for _ in range(3):
            out.zero_()
            graph.replay()
            torch.cuda.synchronize()
            assert torch.equal(out, ref)
        # new contents in the same buffers: the replay computes on what is there now
        q2, k2, v2, _, _ = _inputs(B, H, n, d, seed=6)
        q.copy_(q2), k.copy_(k2), v.copy_(v2)
        graph.replay()
        torch.cuda.synchronize()
        replayed = out.clone()
        direct = ctx.forward(q, k, v)
        ctx.check()
        assert torch.equal(replayed, direct)
    finally:
        ctx.destroy()
