"""Full-size parity for the LLM-shaped configurations, in the launch configuration the
benchmark times.  The oracle computes sampled rows one by one (float64); properties that
hold at any size cover every element: pushed tiles are bit-identical to the stored partial,
the reduction is the order-exact fp32 sum of the stored contributions, counts are exact."""
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

# (workload, rank, orders, budgets): the budgets are the ones the configurations name
FULL = [
    (I.ATTN_OUT, 1, (1, 0), (0, 20)),
    (I.MLP_DOWN, 5, (1,), (0, 20)),
    (I.SHORT_K, 2, (1, 0), (0, 8, 16, 24)),
]


def _rows_to_f64(t, rows):
    return O.bf16_bits_to_f64(I.bits(t[rows]))


def _sampled_parity(wl, r, orders, budgets):
    """Sampled rows against the float64 oracle, every element against the properties that hold at
    any size, exact counts; for each tile order and communication budget."""
    A, Bm = I.make_operands(wl, device="cuda")
    P = I.make_peer_partials(wl, device="cuda")
    R, W = wl.R, wl.W
    rng = np.random.default_rng(wl.seed)
    # sampled rows of the M x N partial: a band in every partition incl. first / last rows
    rows = np.unique(np.concatenate(
        [np.array([d * R, d * R + R - 1]) for d in range(W)] +
        [rng.integers(0, wl.M, 48)] + [r * R + rng.integers(0, R, 48)]))
    Ab, Bb = I.bits(A[rows]), I.bits(Bm)
    C_rows = O.partial_gemm(Ab, Bb)           # float64, rows x N
    S_rows = O.abs_gemm(Ab, Bb)
    own = (rows >= r * R) & (rows < (r + 1) * R)
    own_rows = rows[own]
    peers_rows = np.stack([_rows_to_f64(P[q], own_rows) for q in range(W - 1)])
    ref_out = C_rows[own] + peers_rows.sum(0)
    S_out = S_rows[own] + np.abs(peers_rows).sum(0)
    for order in orders:
        for n_comm in budgets:
            p = E.Plan(wl.M, wl.N, wl.K, W, order, n_comm, rank=r)
            c = p.counts()
            out = torch.full((R, wl.N), float("nan"), dtype=torch.bfloat16, device="cuda")
            send = torch.full((W - 1, R, wl.N), float("nan"), dtype=torch.bfloat16, device="cuda")
            p.gemm_rs(A, Bm, P, out, send)
            st = p.last_status()
            assert st["flags_published"] == c["flags_published"] == W * c["Q"]
            assert st["tiles_reduced"] == c["n_reduce"] and st["tiles_pushed"] == c["n_push"]
            # sampled rows against the float64 oracle
            got_out = _rows_to_f64(out, own_rows - r * R)
            err = np.abs(got_out - ref_out)
            tol = O.tolerance(ref_out, S_out)
            assert (err <= tol).all(), f"out worst err/tol {np.max(err / tol):.3f}"
            for i, row in enumerate(rows):
                d = int(row // R)
                if d == r:
                    continue
                got = O.bf16_bits_to_f64(I.bits(send[O.peer_slot(d, r), row - d * R]))
                e = np.abs(got - C_rows[i])
                assert (e <= O.tolerance(C_rows[i], S_rows[i])).all()
            # every element: copies are exact, the reduction is the fp32 rank-order sum
            Cd = torch.empty((wl.M, wl.N), dtype=torch.bfloat16, device="cuda")
            p.read_partial(Cd)
            torch.cuda.synchronize()
            for slot, d in enumerate(dd for dd in range(W) if dd != r):
                assert torch.equal(send[slot], Cd[d * R:(d + 1) * R])
            acc = Cd[r * R:(r + 1) * R].float()
            for q in range(W - 1):
                acc = acc + P[q, r * R:(r + 1) * R].float()
            assert torch.equal(out, acc.to(torch.bfloat16))
            assert not torch.isnan(out.float()).any()
            del Cd, acc, out, send
            p.destroy()
    del A, Bm, P
    torch.cuda.empty_cache()


@pytest.mark.parametrize("wl,r,orders,budgets", FULL, ids=lambda v: getattr(v, "name", None))
def test_full_size_sampled_parity(wl, r, orders, budgets):
    _sampled_parity(wl, r, orders, budgets)


def _sweep_shape(M, K, W):
    return next(w for w in I.sweep_workloads() if (w.M, w.K, w.W) == (M, K, W))


# the four corners of the sweep grid (M x K_local, with the rank counts at the ends) and two
# interior points; budgets at both ends and the middle of the sweep's range, both tile orders
SWEEP_SAMPLE = [(2048, 512, 2), (32768, 4096, 8), (32768, 512, 2), (2048, 4096, 8), (8192, 1024, 4),
                (16384, 2048, 8)]


@pytest.mark.parametrize("M,K,W", SWEEP_SAMPLE)
def test_sweep_shapes_sampled_parity(M, K, W):
    """The sweep configuration against the oracle: sampled rows in float64, every element against
    the any-size properties, exact counts."""
    wl = _sweep_shape(M, K, W)
    assert wl.K >= 256  # the float64 bound is feasible for a bf16-stored partial (see test_gpu_parity)
    _sampled_parity(wl, W - 1 if M > 2048 else 0, (1, 0), (0, 16, 32))


def test_ring_handover_keeps_every_element_exact():
    """Co-located consumers move from the small ring beside the producer's buffers to the large
    ring that reuses those buffers when their CTA's producer work ends.  Steps still in flight
    in the small ring at that moment must not be overwritten: with the communication-heavy
    short-K shape (the consumers are busiest at the hand-over) and a poisoned workspace, every
    pushed tile equals the stored partial bit for bit and every reduced element is the
    rank-order fp32 sum, on repeated launches."""
    wl, r = I.SHORT_K, 2
    A, Bm = I.make_operands(wl, device="cuda")
    P = I.make_peer_partials(wl, device="cuda")
    R, W = wl.R, wl.W
    for order in (1, 0):
        p = E.Plan(wl.M, wl.N, wl.K, W, order, 0, rank=r, poison_partial=1)
        out = torch.empty((R, wl.N), dtype=torch.bfloat16, device="cuda")
        send = torch.empty((W - 1, R, wl.N), dtype=torch.bfloat16, device="cuda")
        Cd = torch.empty((wl.M, wl.N), dtype=torch.bfloat16, device="cuda")
        for _ in range(6):
            out.fill_(float("nan"))
            send.fill_(float("nan"))
            p.gemm_rs(A, Bm, P, out, send)
            p.read_partial(Cd)
            torch.cuda.synchronize()
            for slot, d in enumerate(dd for dd in range(W) if dd != r):
                assert torch.equal(send[slot].view(torch.int16), Cd[d * R:(d + 1) * R].view(torch.int16))
            acc = Cd[r * R:(r + 1) * R].float()
            for q in range(W - 1):
                acc = acc + P[q, r * R:(r + 1) * R].float()
            assert torch.equal(out, acc.to(torch.bfloat16))
        p.destroy()
