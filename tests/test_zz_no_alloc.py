"""The no-allocation entry point (entwine_gemm_rs_static) against the regular one.

Some users of this library run where device allocation is off limits: an inference server
that froze its memory plan at start-up, a latency-critical loop where cudaMalloc's implicit
synchronisation is not acceptable, or a process whose device memory is wholly owned by another
allocator.  For them the library carries one fixed scratch array; this test checks that the
fused call on that array gives exactly what the allocating entry point gives, on several calls
in a row that share (and must correctly reset) the array, and that oversized problems are
turned away.  It sits in a file that pytest collects last, so a failure here cannot hide
another test's result in a run that stops at the first failure."""
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


def _run_both(wl, r, order, n_comm):
    A, Bm = I.make_operands(wl, device="cuda")
    P = I.make_peer_partials(wl, device="cuda")
    ref_plan = E.Plan(wl.M, wl.N, wl.K, wl.W, order, n_comm, rank=r)
    out_ref = torch.empty(wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
    send_ref = torch.empty(wl.W - 1, wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
    ref_plan.gemm_rs(A, Bm, P, out_ref, send_ref)
    st_ref = ref_plan.last_status()
    plan = E.Plan(wl.M, wl.N, wl.K, wl.W, order, n_comm, rank=r)
    out = torch.full((wl.R, wl.N), float("nan"), dtype=torch.bfloat16, device="cuda")
    send = torch.full((wl.W - 1, wl.R, wl.N), float("nan"), dtype=torch.bfloat16, device="cuda")
    st = plan.gemm_rs_static(A, Bm, P, out, send)
    assert st["code"] == E.OK
    for k in ("flags_published", "tiles_reduced", "tiles_pushed"):
        assert st[k] == st_ref[k]
    # same kernel, single writer per element: within the parity tolerance means identical here
    got, want = O.bf16_bits_to_f64(I.bits(out)), O.bf16_bits_to_f64(I.bits(out_ref))
    assert (np.abs(got - want) <= 4e-3 * np.abs(want)).all()
    assert torch.equal(out, out_ref) and torch.equal(send, send_ref)
    ref_plan.destroy()
    plan.destroy()


def test_static_scratch_matches_allocating_entry_point_on_consecutive_calls():
    a = I.Workload("na_a", 4, 1024, 768, 320, "normal", "normal_total_fanin", 7, 0)
    b = I.TINY
    c = I.Workload("na_c", 8, 2048, 1024, 448, "normal", "normal_total_fanin", 7, 1)
    # different shapes, ranks, orders and budgets back to back on the one shared array
    _run_both(a, 1, E.ORDER_INTERLEAVED, 8)
    _run_both(b, 0, E.ORDER_ROW_MAJOR, 4)
    _run_both(a, 3, E.ORDER_ROW_MAJOR, 0)
    _run_both(c, 5, E.ORDER_INTERLEAVED, 20)
    _run_both(a, 1, E.ORDER_INTERLEAVED, 8)


def test_static_scratch_rejects_problems_above_its_maximum():
    wl = I.ATTN_OUT            # 4096 x 4096 x 2 bytes = 32 MiB > 8 MiB
    plan = E.Plan(wl.M, wl.N, wl.K, wl.W, E.ORDER_INTERLEAVED, 20)
    dummy = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(E.EntwineError) as e:
        plan.gemm_rs_static(dummy, dummy, dummy, dummy, dummy)
    assert e.value.code == E.ERR_TOO_LARGE
    assert "8 MiB" in E.strerror(E.ERR_TOO_LARGE)
    plan.destroy()
