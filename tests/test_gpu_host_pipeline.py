"""The host-buffer call as a pipeline of depth two: same results, bit for bit, as the synchronous
host-buffer call, whatever the interleaving of begin and wait; one result also against the oracle."""
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


def _host_inputs(wl):
    A, Bm = I.make_operands(wl, device="cpu")
    P = I.make_peer_partials(wl, device="cpu")
    return A.pin_memory(), Bm.pin_memory(), P.pin_memory()


def test_pipelined_calls_match_the_synchronous_call():
    W, M, N, K, rank = 4, 1024, 768, 192, 2
    wls = [I.Workload("pipe", W, M, N, K, "normal", "normal_total_fanin", 13, i) for i in range(5)]
    ins = [_host_inputs(wl) for wl in wls]
    R = M // W
    sync_plan = E.Plan(M, N, K, W, 1, 0, rank=rank)
    want = []
    for A, Bm, P in ins:
        out = torch.empty(R, N, dtype=torch.bfloat16).pin_memory()
        send = torch.empty(W - 1, R, N, dtype=torch.bfloat16).pin_memory()
        sync_plan.gemm_rs_host(A, Bm, P, out, send)
        want.append((out.clone(), send.clone()))
    sync_plan.destroy()

    plan = E.Plan(M, N, K, W, 1, 0, rank=rank)
    outs = [(torch.full((R, N), float("nan"), dtype=torch.bfloat16).pin_memory(),
             torch.full((W - 1, R, N), float("nan"), dtype=torch.bfloat16).pin_memory()) for _ in ins]
    plan.gemm_rs_host_wait()  # nothing outstanding: returns at once
    for i, (A, Bm, P) in enumerate(ins):
        plan.gemm_rs_host_begin(A, Bm, P, outs[i][0], outs[i][1])
        if i >= 1:
            plan.gemm_rs_host_wait()  # call i-1 is complete, call i may still run
            assert torch.equal(outs[i - 1][0].view(torch.int16), want[i - 1][0].view(torch.int16))
            assert torch.equal(outs[i - 1][1].view(torch.int16), want[i - 1][1].view(torch.int16))
    plan.gemm_rs_host_wait()
    st = plan.last_status()
    assert st["tiles_reduced"] == plan.counts()["n_reduce"]
    assert torch.equal(outs[-1][0].view(torch.int16), want[-1][0].view(torch.int16))
    assert torch.equal(outs[-1][1].view(torch.int16), want[-1][1].view(torch.int16))

    # the last result against the oracle's definition
    A, Bm, P = ins[-1]
    Ab, Bb, Pb = I.bits(A), I.bits(Bm), I.bits(P)
    C, S = O.partial_gemm(Ab, Bb), O.abs_gemm(Ab, Bb)
    ref_out, ref_send = O.reduce_scatter_ref(C, Pb, rank, W)
    got = O.bf16_bits_to_f64(I.bits(outs[-1][0]))
    assert (np.abs(got - ref_out) <= O.tolerance(ref_out, O.out_magnitude_sum(S, Pb, rank, W))).all()

    # a third call without a wait is refused; the two outstanding ones still complete
    a = [(torch.empty(R, N, dtype=torch.bfloat16).pin_memory(),
          torch.empty(W - 1, R, N, dtype=torch.bfloat16).pin_memory()) for _ in range(3)]
    plan.gemm_rs_host_begin(*ins[0], *a[0])
    plan.gemm_rs_host_begin(*ins[1], *a[1])
    with pytest.raises(E.EntwineError) as ei:
        plan.gemm_rs_host_begin(*ins[2], *a[2])
    assert ei.value.code == E.ERR_INVALID
    plan.gemm_rs_host_wait()
    plan.gemm_rs_host_wait()
    assert torch.equal(a[0][0].view(torch.int16), want[0][0].view(torch.int16))
    assert torch.equal(a[1][1].view(torch.int16), want[1][1].view(torch.int16))
    plan.destroy()
