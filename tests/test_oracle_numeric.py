"""Pins for the floating-point part of the oracle: brute force on tiny shapes, textbook
special cases, the ReduceScatter invariant, and the bf16 helpers."""
import numpy as np
import pytest
import torch

from oracle import entwine_oracle as O
from paper_2609_11562_b200 import inputs as I


def _rand_bits(rng, shape, scale=1.0):
    v = O.bf16_round(rng.standard_normal(shape) * scale)
    return O.f64_to_bf16_bits(v)


def test_bf16_round_ties_and_known_values():
    # 8 significant bits: 1 + 2^-8 is a tie between 1 and 1 + 2^-7 -> even mantissa (1.0)
    assert O.bf16_round(np.array([1 + 2.0 ** -8]))[0] == 1.0
    # 1 + 3*2^-8 ties between 1+2^-7 and 1+2^-6 -> even mantissa 1+2^-6
    assert O.bf16_round(np.array([1 + 3 * 2.0 ** -8]))[0] == 1 + 2.0 ** -6
    assert O.bf16_round(np.array([1 + 2.0 ** -8 + 2.0 ** -20]))[0] == 1 + 2.0 ** -7
    assert O.bf16_round(np.array([-3.0, 0.0, 0.5, 255.0, 257.0]))[[0, 1, 2, 3]].tolist() == \
        [-3.0, 0.0, 0.5, 255.0]
    assert O.bf16_round(np.array([257.0]))[0] == 256.0     # tie -> even
    assert O.bf16_round(np.array([259.0]))[0] == 260.0     # tie -> even


def test_bf16_helpers_against_torch():
    g = torch.Generator().manual_seed(5)
    v = torch.randn(4096, generator=g, dtype=torch.float64) * torch.logspace(-6, 6, 4096,
                                                                            dtype=torch.float64)
    want = v.to(torch.float32).to(torch.bfloat16)
    # (float64 -> float32 -> bf16 double rounding can differ from direct rounding only on
    # measure-zero ties, which random doubles never hit)
    got = O.bf16_round(v.numpy())
    assert (got == want.to(torch.float64).numpy()).all()
    bits = O.f64_to_bf16_bits(got)
    assert (bits == I.bits(want)).all()
    assert (O.bf16_bits_to_f64(bits) == got).all()


def _brute_partial(A, B):
    M, K = A.shape
    N = B.shape[0]
    C = np.zeros((M, N))
    for i in range(M):
        for j in range(N):
            acc = 0.0
            for k in range(K):
                acc += A[i, k] * B[j, k]
            C[i, j] = acc
    return C


def test_partial_gemm_bruteforce():
    rng = np.random.default_rng(1)
    A_bits = _rand_bits(rng, (6, 20))
    B_bits = _rand_bits(rng, (5, 20))
    A, B = O.bf16_bits_to_f64(A_bits), O.bf16_bits_to_f64(B_bits)
    C = O.partial_gemm(A_bits, B_bits)
    assert C.shape == (6, 5)
    np.testing.assert_allclose(C, _brute_partial(A, B), rtol=1e-13, atol=1e-13)
    S = O.abs_gemm(A_bits, B_bits)
    np.testing.assert_allclose(S, _brute_partial(np.abs(A), np.abs(B)), rtol=1e-13)
    assert (S >= np.abs(C) - 1e-12).all()


def test_partial_gemm_special_cases():
    rng = np.random.default_rng(2)
    A_bits = _rand_bits(rng, (128, 64))
    A = O.bf16_bits_to_f64(A_bits)
    # B = identity (stored [N,K]) -> C = A
    eye = O.f64_to_bf16_bits(np.eye(64))
    assert (O.partial_gemm(A_bits, eye) == A).all()
    # a non-symmetric B catches a transposed operand: B[n,k] = 1 iff k == (n+1) % 64
    shift = np.zeros((64, 64))
    shift[np.arange(64), (np.arange(64) + 1) % 64] = 1
    assert (O.partial_gemm(A_bits, O.f64_to_bf16_bits(shift)) == np.roll(A, -1, axis=1)).all()
    # one-hot rows of A pick columns of B^T
    onehot = np.zeros((4, 64))
    onehot[np.arange(4), [3, 0, 63, 17]] = 1
    B_bits = _rand_bits(rng, (32, 64))
    B = O.bf16_bits_to_f64(B_bits)
    assert (O.partial_gemm(O.f64_to_bf16_bits(onehot), B_bits) == B[:, [3, 0, 63, 17]].T).all()


def _brute_reduce_scatter(C_r, peers, r, W):
    M, N = C_r.shape
    R = M // W
    out = np.zeros((R, N))
    for i in range(R):
        for j in range(N):
            acc = C_r[r * R + i, j]
            for q in range(W - 1):
                acc += peers[q, r * R + i, j]
            out[i, j] = acc
    return out


@pytest.mark.parametrize("W,r", [(2, 0), (2, 1), (3, 1), (4, 3)])
def test_reduce_scatter_bruteforce_and_special_cases(W, r):
    rng = np.random.default_rng(3 + W)
    M, N = 4 * W, 6
    C = rng.standard_normal((M, N))
    peers_bits = _rand_bits(rng, (W - 1, M, N))
    peers = O.bf16_bits_to_f64(peers_bits)
    out, send = O.reduce_scatter_ref(C, peers_bits, r, W)
    np.testing.assert_allclose(out, _brute_reduce_scatter(C, peers, r, W), rtol=1e-14)
    R = M // W
    others = [d for d in range(W) if d != r]
    for slot, d in enumerate(others):
        assert (send[slot] == C[d * R:(d + 1) * R]).all()
        assert O.peer_slot(d, r) == slot
    # zero peers -> the rank's own rows
    zero = np.zeros_like(peers_bits)
    out0, _ = O.reduce_scatter_ref(C, zero, r, W)
    assert (out0 == C[r * R:(r + 1) * R]).all()
    # zero own partial -> plain sum of the peers' rows
    outp, _ = O.reduce_scatter_ref(np.zeros_like(C), peers_bits, r, W)
    np.testing.assert_allclose(outp, peers[:, r * R:(r + 1) * R].sum(0), rtol=1e-14)
    # rows outside partition r of the peer buffers are never read
    poisoned = peers_bits.copy()
    mask = np.ones(M, bool)
    mask[r * R:(r + 1) * R] = False
    poisoned[:, mask] = 0x7FC0  # NaN
    outq, _ = O.reduce_scatter_ref(C, poisoned, r, W)
    assert (outq == out).all()


@pytest.mark.parametrize("W", [2, 4])
def test_concat_of_shards_is_unsplit_gemm(W):
    """Full mode: every rank computes its partial; peers' partials are taken unrounded, so
    concat_d O_d must equal [A_0 ... A_{W-1}] . [B_0 ... B_{W-1}]^T (Sec. 2.1)."""
    rng = np.random.default_rng(7)
    M, N, K = 128 * W, 128, 32
    A_bits = [_rand_bits(rng, (M, K)) for _ in range(W)]
    B_bits = [_rand_bits(rng, (N, K), 0.2) for _ in range(W)]
    C = [O.partial_gemm(A_bits[w], B_bits[w]) for w in range(W)]
    A_cat = np.concatenate([O.bf16_bits_to_f64(a) for a in A_bits], axis=1)
    B_cat = np.concatenate([O.bf16_bits_to_f64(b) for b in B_bits], axis=1)
    full = A_cat @ B_cat.T
    R = M // W
    shards = []
    for r in range(W):
        acc = C[r][r * R:(r + 1) * R].copy()
        for w in range(W):
            if w != r:
                # what rank w sends to r is its rows of partition r (ref_send of rank w)
                _, send_w = O.reduce_scatter_ref(C[w], np.zeros((W - 1, M, N), np.uint16), w, W)
                acc += send_w[O.peer_slot(r, w)]
        shards.append(acc)
    np.testing.assert_allclose(np.concatenate(shards), full, rtol=1e-12, atol=1e-12)


def test_staged_model_within_tolerance_on_tiny_config():
    wl = I.TINY
    A, B = I.make_operands(wl)
    P = I.make_peer_partials(wl)
    Ab, Bb, Pb = I.bits(A), I.bits(B), I.bits(P)
    for r in range(wl.W):
        res = O.gemm_rs(Ab, Bb, Pb, r, wl.W, 256, O.ORDER_INTERLEAVED, 4)
        out, send = O.staged_model(Ab, Bb, Pb, r, wl.W)
        tol = O.tolerance(res["ref_out"], res["S_out"])
        assert (np.abs(out - res["ref_out"]) <= tol).all()
        R = wl.R
        for slot, d in enumerate(dd for dd in range(wl.W) if dd != r):
            tol_s = O.tolerance(res["ref_send"][slot], res["S"][d * R:(d + 1) * R])
            assert (np.abs(send[slot] - res["ref_send"][slot]) <= tol_s).all()
        # the staged result differs from the definition by a few bf16 ulps at most
        assert np.abs(out - res["ref_out"]).max() <= 2.0 ** -7 * np.abs(res["ref_out"]).max()


def test_input_generators_are_seeded_and_shaped():
    wl = I.TINY
    A1, B1 = I.make_operands(wl)
    A2, B2 = I.make_operands(wl)
    assert torch.equal(A1, A2) and torch.equal(B1, B2)
    assert A1.shape == (wl.M, wl.K) and B1.shape == (wl.N, wl.K)
    assert A1.abs().max() <= 1.0
    P = I.make_peer_partials(wl)
    assert P.shape == (wl.W - 1, wl.M, wl.N) and P.dtype == torch.bfloat16
    assert 0.9 < P.float().std() < 1.1
    assert len(I.sweep_workloads()) == 60
    assert I.ATTN_OUT.comm_bytes == 4096 * 4096 * 2 * 11 // 4


def test_rmsnorm_closed_forms_and_library():
    """RMSNorm definition: constant rows normalise to sign * weight; a one-hot row of value v
    in N columns gives sqrt(N) * sign(v) * w at that column; scale invariance at eps = 0;
    float64 torch.nn.functional.rms_norm as the library routine."""
    rng = np.random.default_rng(5)
    N = 96
    w = rng.normal(size=N)
    const = np.full((3, N), -2.5)
    assert np.allclose(O.rmsnorm_ref(const, w, 0.0), -w[None, :].repeat(3, 0), rtol=1e-14)
    onehot = np.zeros((2, N))
    onehot[0, 7], onehot[1, 40] = 3.0, -0.25
    got = O.rmsnorm_ref(onehot, w, 0.0)
    assert np.isclose(got[0, 7], np.sqrt(N) * w[7]) and np.isclose(got[1, 40], -np.sqrt(N) * w[40])
    assert np.count_nonzero(got) == 2
    h = rng.normal(size=(5, N))
    assert np.allclose(O.rmsnorm_ref(h, w, 0.0), O.rmsnorm_ref(1e3 * h, w, 0.0), rtol=1e-12)
    # eps matters exactly as mean(h^2) + eps
    eps = 0.37
    manual = h / np.sqrt((h ** 2).sum(-1, keepdims=True) / N + eps) * w
    assert np.allclose(O.rmsnorm_ref(h, w, eps), manual, rtol=1e-14)
    lib = torch.nn.functional.rms_norm(torch.from_numpy(h), (N,), torch.from_numpy(w), eps).numpy()
    assert np.allclose(O.rmsnorm_ref(h, w, eps), lib, rtol=1e-12, atol=1e-14)


def test_layer_chain_is_residual_add_then_rmsnorm():
    rng = np.random.default_rng(6)
    R, N = 8, 64
    out = rng.normal(size=(R, N))
    res_bits = O.f64_to_bf16_bits(rng.normal(size=(R, N)))
    w_bits = O.f64_to_bf16_bits(1.0 + 0.1 * rng.normal(size=N))
    hidden, normed = O.layer_chain_ref(out, res_bits, w_bits, 1e-5)
    res, w = O.bf16_bits_to_f64(res_bits), O.bf16_bits_to_f64(w_bits)
    assert np.array_equal(hidden, out + res)
    for i in range(R):  # row by row, written out
        ms = sum(float(v) ** 2 for v in hidden[i]) / N
        assert np.allclose(normed[i], hidden[i] / np.sqrt(ms + 1e-5) * w, rtol=1e-13)
    # zero residual and unit weight: rows of unit RMS
    _, n1 = O.layer_chain_ref(out, np.zeros((R, N), np.uint16), O.f64_to_bf16_bits(np.ones(N)), 0.0)
    assert np.allclose((n1 ** 2).mean(-1), 1.0, rtol=1e-12)


def test_norm_task_order_hand_listed():
    """Two bands of three tile columns (R = 256 rows per rank, N = 384), listed by hand: band 0's
    tiles left to right, then band 1's.  A column-first walk, a band-last walk or a transposed
    (column, band) pair would each differ from this list."""
    order = O.norm_task_order(512, 384, 2)
    assert order.dtype == np.int32
    assert order.tolist() == [[0, 0], [0, 1], [0, 2], [1, 0], [1, 1], [1, 2]]
    # one band only: W = 4 leaves R = 128
    assert O.norm_task_order(512, 384, 4).tolist() == [[0, 0], [0, 1], [0, 2]]
