"""Layer chain (Sec. 5.2.3): GEMM + ReduceScatter, residual addition and RMSNorm in one launch,
against the oracle's definitions, through the C ABI."""
import itertools

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

EPS = 1e-5


def _vals(t):
    return O.bf16_bits_to_f64(I.bits(t))


def _run_and_check(wl, r, order, n_comm, A, Bm, P, res, w, oracle=None, **opts):
    p = E.Plan(wl.M, wl.N, wl.K, wl.W, order, n_comm, rank=r, **opts)
    R, W = wl.R, wl.W
    hidden = torch.full((R, wl.N), float("nan"), dtype=torch.bfloat16, device="cuda")
    normed = torch.full((R, wl.N), float("nan"), dtype=torch.bfloat16, device="cuda")
    send = torch.full((W - 1, R, wl.N), float("nan"), dtype=torch.bfloat16, device="cuda")
    p.gemm_rs_norm(A, Bm, P, res, w, EPS, hidden, normed, send)
    st = p.last_status()
    c = p.counts()
    assert st["flags_published"] == c["flags_published"]
    assert st["tiles_reduced"] == c["n_reduce"] and st["tiles_pushed"] == c["n_push"]
    Cd = torch.empty((wl.M, wl.N), dtype=torch.bfloat16, device="cuda")
    p.read_partial(Cd)
    torch.cuda.synchronize()
    # pushes are copies of the stored partial
    for slot, d in enumerate(dd for dd in range(W) if dd != r):
        assert torch.equal(send[slot], Cd[d * R:(d + 1) * R])
    # hidden = bf16 of the rank-order fp32 sum of the stored contributions plus the residual
    acc = Cd[r * R:(r + 1) * R].float()
    for q in range(W - 1):
        acc = acc + P[q, r * R:(r + 1) * R].float()
    acc = acc + res.float()
    assert torch.equal(hidden, acc.to(torch.bfloat16))
    # normed = the RMSNorm definition (float64) of the stored hidden values, one bf16 rounding
    ref_norm = O.rmsnorm_ref(_vals(hidden), _vals(w), EPS)
    got = _vals(normed)
    assert np.isfinite(got).all()
    err = np.abs(got - ref_norm)
    assert (err <= 4e-3 * np.abs(ref_norm) + 1e-6).all(), f"norm worst {np.max(err / (4e-3 * np.abs(ref_norm) + 1e-6)):.3f}"
    if oracle is not None:
        # the whole chain against the definition with no intermediate rounding
        ref_hidden, ref_full = oracle
        S = oracle_S[(wl.name, r)]
        tol = O.tolerance(ref_hidden, S)
        assert (np.abs(_vals(hidden) - ref_hidden) <= tol).all()
        # normalisation divides by the row RMS: the hidden tolerance scales with it
        inv = 1.0 / np.sqrt((ref_hidden ** 2).mean(-1, keepdims=True) + EPS)
        wv = np.abs(_vals(w))[None, :]
        # a row's RMS moves by at most the RMS of its elements' errors
        row_tol = np.sqrt((tol ** 2).mean(-1, keepdims=True))
        tol_n = 4e-3 * np.abs(ref_full) + tol * inv * wv + np.abs(ref_full) * row_tol * inv
        assert (np.abs(got - ref_full) <= tol_n).all()
    p.destroy()
    return hidden, normed, send


oracle_S = {}


@pytest.mark.parametrize("shape", [(4, 1024, 768, 320), (8, 2048, 1024, 448), (2, 512, 512, 272)],
                         ids=lambda s: "W%d_M%d_N%d_K%d" % s)
def test_layer_chain_matches_oracle(shape):
    W, M, N, K = shape
    wl = I.Workload("chain", W, M, N, K, "normal", "normal_total_fanin", 9, 20 + W)
    A, Bm = I.make_operands(wl)
    P = I.make_peer_partials(wl)
    res, w = I.make_layer_inputs(wl)
    Ab, Bb, Pb = I.bits(A), I.bits(Bm), I.bits(P)
    Ad, Bd, Pd, resd, wd = A.cuda(), Bm.cuda(), P.cuda(), res.cuda(), w.cuda()
    for r in (0, W - 1):
        C = O.partial_gemm(Ab, Bb)
        S = O.abs_gemm(Ab, Bb)
        ref_out, _ = O.reduce_scatter_ref(C, Pb, r, W)
        oracle_S[(wl.name, r)] = O.out_magnitude_sum(S, Pb, r, W) + np.abs(_vals(res))
        oracle = O.layer_chain_ref(ref_out, I.bits(res), I.bits(w), EPS)
        base = None
        # (reg: the co-located consumer on the shared-memory ring or on the register path)
        for order, n_comm, BN, reg in itertools.product((1, 0, 2), (0, 4, 20), (256, 128), (0, 1)):
            if N % BN:
                continue
            out = _run_and_check(wl, r, order, n_comm, Ad, Bd, Pd, resd, wd, oracle=oracle, block_n=BN,
                                 reg_consumer=reg)
            if base is None:
                base = out
            # scheduling never changes a bit of any result
            assert all(torch.equal(a, b) for a, b in zip(out, base))


def test_layer_chain_repeats_bitwise_and_rejects_bad_arguments():
    wl = I.Workload("chain_rep", 4, 1024, 1024, 256, "normal", "normal_total_fanin", 9, 31)
    A, Bm = I.make_operands(wl, device="cuda")
    P = I.make_peer_partials(wl, device="cuda")
    res, w = I.make_layer_inputs(wl, device="cuda")
    p = E.Plan(wl.M, wl.N, wl.K, wl.W, 1, 0, rank=2, poison_partial=1)
    outs = []
    for _ in range(3):
        hidden = torch.empty((wl.R, wl.N), dtype=torch.bfloat16, device="cuda")
        normed = torch.empty_like(hidden)
        send = torch.empty((wl.W - 1, wl.R, wl.N), dtype=torch.bfloat16, device="cuda")
        p.gemm_rs_norm(A, Bm, P, res, w, EPS, hidden, normed, send)
        p.last_status()
        outs.append((hidden, normed, send))
    for o in outs[1:]:
        assert all(torch.equal(a, b) for a, b in zip(o, outs[0]))
    # the plain call still works on the same plan afterwards, and the chain after it
    out = torch.empty((wl.R, wl.N), dtype=torch.bfloat16, device="cuda")
    send = torch.empty((wl.W - 1, wl.R, wl.N), dtype=torch.bfloat16, device="cuda")
    p.gemm_rs(A, Bm, P, out, send)
    p.last_status()
    assert torch.equal(send, outs[0][2])
    hidden, normed = torch.empty_like(out), torch.empty_like(out)
    with pytest.raises(E.EntwineError):
        p.gemm_rs_norm(A, Bm, P, None, w, EPS, hidden, normed, send)
    with pytest.raises(E.EntwineError):
        p.gemm_rs_norm(A, Bm, P, res, w, -1.0, hidden, normed, send)
    p.gemm_rs_norm(A, Bm, P, res, w, EPS, hidden, normed, send)
    p.last_status()
    assert torch.equal(hidden, outs[0][0]) and torch.equal(normed, outs[0][1])
    p.destroy()
    # more lists than consumer CTAs: a waiting CTA could starve a list, so the call is refused
    p = E.Plan(wl.M, wl.N, wl.K, wl.W, 1, 0, rank=2, lists=400)
    with pytest.raises(E.EntwineError):
        p.gemm_rs_norm(A, Bm, P, res, w, EPS, hidden, normed, send)
    p.destroy()


def test_layer_chain_full_size_attention_output():
    """The benchmark's attention out-projection with the chain, every element: bit-exact hidden
    against the stored contributions, RMSNorm of the stored hidden in float64 on the GPU."""
    wl, r = I.ATTN_OUT, 1
    A, Bm = I.make_operands(wl, device="cuda")
    P = I.make_peer_partials(wl, device="cuda")
    res, w = I.make_layer_inputs(wl, device="cuda")
    R, W = wl.R, wl.W
    for order, n_comm in ((1, 0), (0, 16)):
        p = E.Plan(wl.M, wl.N, wl.K, W, order, n_comm, rank=r)
        hidden = torch.empty((R, wl.N), dtype=torch.bfloat16, device="cuda")
        normed = torch.empty_like(hidden)
        send = torch.empty((W - 1, R, wl.N), dtype=torch.bfloat16, device="cuda")
        for _ in range(3):
            p.gemm_rs_norm(A, Bm, P, res, w, EPS, hidden, normed, send)
        p.last_status()
        Cd = torch.empty((wl.M, wl.N), dtype=torch.bfloat16, device="cuda")
        p.read_partial(Cd)
        acc = Cd[r * R:(r + 1) * R].float()
        for q in range(W - 1):
            acc = acc + P[q, r * R:(r + 1) * R].float()
        acc = acc + res.float()
        assert torch.equal(hidden, acc.to(torch.bfloat16))
        h64 = hidden.double()
        ref = h64 / torch.sqrt((h64 * h64).mean(-1, keepdim=True) + EPS) * w.double()
        err = (normed.double() - ref).abs()
        assert bool((err <= 4e-3 * ref.abs() + 1e-6).all())
        p.destroy()
