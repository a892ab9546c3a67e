"""CUDA-graph capture of the fused call: every replay must publish and wait for its own flags.

The captured launch carries the flag value of the capture; a replay that trusted flags left by
the previous replay would let consumers read a partial output that is still being written.
The workspace is poisoned before every captured launch, so such a read shows up as NaN.
"""
import numpy as np
import pytest
import torch

from oracle import entwine_oracle as O
from paper_2609_11562_b200 import inputs as I

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from paper_2609_11562_b200 import build as B
    B.build()

WL = I.Workload("graph_case", 4, 1024, 768, 192, "normal_fanin", "normal_fanin", 7, 0)


def _check(out, send, A, Bm, P, wl, rank):
    """out_shard and send_bufs against the oracle's definition on the buffers' current contents."""
    Ab, Bb, Pb = I.bits(A), I.bits(Bm), I.bits(P)
    C = O.partial_gemm(Ab, Bb)
    S = O.abs_gemm(Ab, Bb)
    ref_out, ref_send = O.reduce_scatter_ref(C, Pb, rank, wl.W)
    got = O.bf16_bits_to_f64(I.bits(out))
    assert np.isfinite(got).all()
    assert (np.abs(got - ref_out) <= O.tolerance(ref_out, O.out_magnitude_sum(S, Pb, rank, wl.W))).all()
    got_send = O.bf16_bits_to_f64(I.bits(send))
    R = wl.R
    for slot, d in enumerate(dd for dd in range(wl.W) if dd != rank):
        assert (np.abs(got_send[slot] - ref_send[slot]) <= O.tolerance(ref_send[slot], S[d * R:(d + 1) * R])).all()


@pytest.mark.parametrize("order,n_comm", [(1, 0), (0, 8)])
def test_captured_call_replays_with_fresh_flags(order, n_comm):
    from paper_2609_11562_b200 import entwine as E
    wl, rank = WL, 1
    A, Bm = I.make_operands(wl, device="cuda")
    P = I.make_peer_partials(wl, device="cuda")
    out = torch.empty(wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
    send = torch.empty(wl.W - 1, wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
    plan = E.Plan(wl.M, wl.N, wl.K, wl.W, order, n_comm, rank=rank, poison_partial=1)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        plan.gemm_rs(A, Bm, P, out, send)  # the eager launch that allocates
        plan.last_status()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            plan.gemm_rs(A, Bm, P, out, send)
        gen = torch.Generator(device="cuda").manual_seed(5)
        for it in range(4):
            # new operands in the captured buffers, result buffers dirtied
            A.copy_(torch.randn(A.shape, generator=gen, device="cuda").to(torch.bfloat16))
            P.copy_(torch.randn(P.shape, generator=gen, device="cuda").to(torch.bfloat16))
            out.fill_(float("nan"))
            send.fill_(float("nan"))
            g.replay()
            side.synchronize()
            st = plan.last_status()
            c = plan.counts()
            assert st["tiles_reduced"] == c["n_reduce"] and st["tiles_pushed"] == c["n_push"]
            assert st["flags_published"] == c["flags_published"]
            _check(out, send, A, Bm, P, wl, rank)
            partial = torch.empty(wl.M, wl.N, dtype=torch.bfloat16, device="cuda")
            plan.read_partial(partial)
            side.synchronize()
            # pushed tiles are copies of the stored partial, bit for bit
            R = wl.R
            for q, w in enumerate([w for w in range(wl.W) if w != rank]):
                assert torch.equal(send[q].view(torch.int16), partial[w * R:(w + 1) * R].view(torch.int16))
        # an eager call after the capture still works
        plan.gemm_rs(A, Bm, P, out, send)
        side.synchronize()
        plan.last_status()
        _check(out, send, A, Bm, P, wl, rank)
    plan.destroy()


@pytest.mark.filterwarnings("ignore:The CUDA Graph is empty")
def test_capture_before_the_first_launch_is_refused():
    from paper_2609_11562_b200 import entwine as E
    wl = WL
    A, Bm = I.make_operands(wl, device="cuda")
    P = I.make_peer_partials(wl, device="cuda")
    out = torch.empty(wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
    send = torch.empty(wl.W - 1, wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
    plan = E.Plan(wl.M, wl.N, wl.K, wl.W, 1, 0)
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            with pytest.raises(E.EntwineError) as ei:
                plan.gemm_rs(A, Bm, P, out, send)
    assert ei.value.code == E.ERR_INVALID
    plan.destroy()


def test_caller_workspace_first_launch_is_captured_and_allocates_nothing():
    """With entwine_plan_set_workspace the plan lives in the caller's block: its very first launch
    can be captured, no launch changes the amount of free device memory, and the results carry the
    same bits as those of a plan with memory of its own; the layer chain uses the same block."""
    from paper_2609_11562_b200 import entwine as E
    wl, rank = WL, 2
    A, Bm = I.make_operands(wl, device="cuda")
    P = I.make_peer_partials(wl, device="cuda")
    res, w = I.make_layer_inputs(wl, device="cuda")
    out = torch.empty(wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
    send = torch.empty(wl.W - 1, wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
    out0, send0 = torch.empty_like(out), torch.empty_like(send)
    hid, nrm, hid0, nrm0 = (torch.empty_like(out) for _ in range(4))
    own = E.Plan(wl.M, wl.N, wl.K, wl.W, 1, 0, rank=rank)
    own.gemm_rs(A, Bm, P, out0, send0)
    own.last_status()
    own.gemm_rs_norm(A, Bm, P, res, w, 1e-5, hid0, nrm0, send0)
    own.last_status()
    own.destroy()

    plan = E.Plan(wl.M, wl.N, wl.K, wl.W, 1, 0, rank=rank)
    n = plan.workspace_bytes()
    assert n >= wl.M * wl.N * 2
    ws = torch.empty(n + 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(E.EntwineError):
        plan.set_workspace(ws[1:], n)            # misaligned
    with pytest.raises(E.EntwineError):
        plan.set_workspace(ws, n - 256)          # too small
    plan.set_workspace(ws, n)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            # the plan's first launch, inside a capture: an allocation here would end the capture
            # with an error
            plan.gemm_rs(A, Bm, P, out, send)
        free0 = None
        for it in range(4):
            if it == 1:
                # (the first round also lets the driver load the kernels and the graph)
                torch.cuda.synchronize()
                free0 = torch.cuda.mem_get_info()[0]
            out.fill_(float("nan"))
            send.fill_(float("nan"))
            g.replay()
            side.synchronize()
            if it == 0:   # (the status query reports a replay only while the captured call is the plan's latest)
                st = plan.last_status()
                assert st["tiles_reduced"] == plan.counts()["n_reduce"]
            assert torch.equal(out, out0) and torch.equal(send, send0)
            plan.gemm_rs_norm(A, Bm, P, res, w, 1e-5, hid, nrm, send)
            side.synchronize()
            plan.last_status()
            assert torch.equal(hid, hid0) and torch.equal(nrm, nrm0)
            if free0 is not None:
                assert torch.cuda.mem_get_info()[0] == free0
    with pytest.raises(E.EntwineError):
        plan.set_workspace(ws, n)                # after a launch
    plan.destroy()
    del g
