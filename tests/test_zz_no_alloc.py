"""The no-allocation entry point (entwine_gemm_rs_static).

Some users of this library run where device allocation is off limits: an inference server
that froze its memory plan at start-up, a latency-critical loop where cudaMalloc's implicit
synchronisation is not acceptable, or a process whose device memory is wholly owned by another
allocator.  For them the library carries one fixed scratch array.  These tests check the fused
call on that array against the CPU oracle and against the allocating entry point (bit for bit),
on several calls in a row that share (and must correctly reset) the array; that the calls leave
the amount of free device memory untouched; and that oversized problems and unsupported options
are turned away."""
import numpy as np
import pytest
import torch

from oracle import entwine_oracle as O
from paper_2609_11562_b200 import inputs as I

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from paper_2609_11562_b200 import build as B
    B.build()
    from paper_2609_11562_b200 import entwine as E


def _vals(t):
    return O.bf16_bits_to_f64(I.bits(t))


def _run_both(wl, r, order, n_comm):
    A, Bm = I.make_operands(wl)
    P = I.make_peer_partials(wl)
    Ad, Bd, Pd = A.cuda(), Bm.cuda(), P.cuda()
    ref_plan = E.Plan(wl.M, wl.N, wl.K, wl.W, order, n_comm, rank=r)
    out_ref = torch.empty(wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
    send_ref = torch.empty(wl.W - 1, wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
    ref_plan.gemm_rs(Ad, Bd, Pd, out_ref, send_ref)
    st_ref = ref_plan.last_status()
    plan = E.Plan(wl.M, wl.N, wl.K, wl.W, order, n_comm, rank=r)
    out = torch.full((wl.R, wl.N), float("nan"), dtype=torch.bfloat16, device="cuda")
    send = torch.full((wl.W - 1, wl.R, wl.N), float("nan"), dtype=torch.bfloat16, device="cuda")
    st = plan.gemm_rs_static(Ad, Bd, Pd, out, send)
    assert st["code"] == E.OK
    c = plan.counts()
    assert st["flags_published"] == c["flags_published"] == st_ref["flags_published"]
    assert st["tiles_reduced"] == c["n_reduce"] == st_ref["tiles_reduced"]
    assert st["tiles_pushed"] == c["n_push"] == st_ref["tiles_pushed"]
    # against the oracle: |gpu - ref| <= 4e-3 |ref| + 1e-3 sum |a b| per element
    res = O.gemm_rs(I.bits(A), I.bits(Bm), I.bits(P), r, wl.W, 256 if wl.N % 256 == 0 else 128, order, c["x"])
    got = _vals(out)
    assert np.isfinite(got).all()
    assert (np.abs(got - res["ref_out"]) <= O.tolerance(res["ref_out"], res["S_out"])).all()
    got_s = _vals(send)
    for slot, d in enumerate(dd for dd in range(wl.W) if dd != r):
        tol_s = O.tolerance(res["ref_send"][slot], res["S"][d * wl.R:(d + 1) * wl.R])
        assert (np.abs(got_s[slot] - res["ref_send"][slot]) <= tol_s).all()
    # against the allocating entry point: same kernel, single writer per element => same bits
    assert torch.equal(out, out_ref) and torch.equal(send, send_ref)
    ref_plan.destroy()
    plan.destroy()


def test_static_scratch_matches_oracle_and_allocating_entry_point_on_consecutive_calls():
    a = I.Workload("na_a", 4, 1024, 768, 320, "normal", "normal_total_fanin", 7, 0)
    b = I.TINY
    c = I.Workload("na_c", 8, 2048, 1024, 448, "normal", "normal_total_fanin", 7, 1)
    # different shapes, ranks, orders and budgets back to back on the one shared array
    _run_both(a, 1, E.ORDER_INTERLEAVED, 8)
    _run_both(b, 0, E.ORDER_ROW_MAJOR, 4)
    _run_both(a, 3, E.ORDER_ROW_MAJOR, 0)
    _run_both(c, 5, E.ORDER_INTERLEAVED, 20)
    _run_both(a, 1, E.ORDER_INTERLEAVED, 8)


def test_static_calls_leave_free_device_memory_unchanged():
    """After the first call on a device (which looks up the scratch array's address) no call may
    change the amount of free device memory, with or without a status read-back; a call without
    read-back followed by a stream synchronisation gives the same bits."""
    wl = I.Workload("na_m", 4, 1024, 768, 320, "normal", "normal_total_fanin", 7, 2)
    A, Bm = I.make_operands(wl, device="cuda")
    P = I.make_peer_partials(wl, device="cuda")
    out = torch.empty(wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
    send = torch.empty(wl.W - 1, wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
    out2, send2 = torch.empty_like(out), torch.empty_like(send)
    plan = E.Plan(wl.M, wl.N, wl.K, wl.W, E.ORDER_INTERLEAVED, 0, rank=2)
    st = plan.gemm_rs_static(A, Bm, P, out, send)       # first call: set-up
    assert st["code"] == E.OK
    free0 = None
    for i in range(8):
        if i == 4:   # the first round also warms the framework's own allocator (comparison temporaries)
            torch.cuda.synchronize()
            free0 = torch.cuda.mem_get_info()[0]
        if i % 2 == 0:
            st = plan.gemm_rs_static(A, Bm, P, out, send)
            assert st["code"] == E.OK
        else:
            out2.fill_(float("nan"))
            send2.fill_(float("nan"))
            assert plan.gemm_rs_static(A, Bm, P, out2, send2, want_status=False) is None
            torch.cuda.synchronize()
            assert torch.equal(out2, out) and torch.equal(send2, send)
        if free0 is not None:
            assert torch.cuda.mem_get_info()[0] == free0
    plan.destroy()


def test_static_scratch_rejects_what_it_cannot_do():
    wl = I.ATTN_OUT            # 4096 x 4096 x 2 bytes = 32 MiB > 8 MiB
    plan = E.Plan(wl.M, wl.N, wl.K, wl.W, E.ORDER_INTERLEAVED, 20)
    dummy = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(E.EntwineError) as e:
        plan.gemm_rs_static(dummy, dummy, dummy, dummy, dummy)
    assert e.value.code == E.ERR_TOO_LARGE
    assert "8 MiB" in E.strerror(E.ERR_TOO_LARGE)
    plan.destroy()
    # options this entry point does not implement are refused, not silently dropped
    small = I.TINY
    for opts in (dict(release_group=4), dict(release_group=E.RELEASE_WHOLE)):
        plan = E.Plan(small.M, small.N, small.K, small.W, E.ORDER_INTERLEAVED, 4, **opts)
        with pytest.raises(E.EntwineError) as e:
            plan.gemm_rs_static(dummy, dummy, dummy, dummy, dummy)
        assert e.value.code == E.ERR_INVALID
        plan.destroy()
    plan = E.Plan(small.M, small.N, small.K, small.W, E.ORDER_INTERLEAVED, 4)
    plan.set_option(E.OPT_WITHHOLD_PEER, (1 << 32) | 0)
    with pytest.raises(E.EntwineError) as e:
        plan.gemm_rs_static(dummy, dummy, dummy, dummy, dummy)
    assert e.value.code == E.ERR_INVALID
    plan.destroy()
    # a capturing stream is refused (the call uploads tables from host memory), and the capture survives it
    plan = E.Plan(small.M, small.N, small.K, small.W, E.ORDER_INTERLEAVED, 4)
    s = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=s):
        with pytest.raises(E.EntwineError) as e:
            plan.gemm_rs_static(dummy, dummy, dummy, dummy, dummy, stream=s, want_status=False)
        dummy.add_(0)
    assert e.value.code == E.ERR_INVALID
    plan.destroy()
