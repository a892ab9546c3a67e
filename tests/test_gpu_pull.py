"""Pull mode (the call of one rank of W ranks on GPUs of their own, Sec. 4.1 / 4.2) exercised on one
GPU, rank by rank, against the oracle.

All W segments of the symmetric heap live in one allocation.  No kernel ever waits for a
kernel that has not run: first every rank's producer runs alone (partials stored, flags sent
to their destinations), then every rank makes its full call, for which only its own flags
are cleared again, so that its consumers synchronise with its own producer while the peers'
contributions are already there.
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
    from paper_2609_11562_b200 import entwine as E


def _rank_workloads(W, M, N, K, call):
    return [I.Workload(f"pull_rank{q}", W, M, N, K, "normal", "normal_total_fanin", 11, 16 * call + q)
            for q in range(W)]


class Heap:
    def __init__(self, plan, W, M, N, pad=512):
        seg, self.flags_off = plan.heap_bytes()
        self.stride = seg + pad
        assert self.stride % 256 == 0
        self.W, self.M, self.N = W, M, N
        self.mem = torch.zeros(W * self.stride, dtype=torch.uint8, device="cuda")
        assert self.mem.data_ptr() % 256 == 0

    def partial(self, q, epoch):
        a = q * self.stride + (epoch & 1) * self.M * self.N * 2
        return self.mem[a:a + self.M * self.N * 2].view(torch.bfloat16).view(self.M, self.N)

    def flags(self, d, Q):
        a = d * self.stride + self.flags_off
        return self.mem[a:a + self.W * Q * 4].view(torch.int32).view(self.W, Q)


@pytest.mark.parametrize("consumer_tma", [1, 0], ids=["peer_tiles_by_tma", "peer_tiles_by_plain_loads"])
@pytest.mark.parametrize("W,M,N,K,order,n_comm", [
    (4, 1024, 768, 192, 1, 0),
    (2, 512, 512, 96, 0, 8),
    (8, 2048, 512, 64, 1, 16),
    (3, 768, 512, 80, 0, 0),
])
def test_every_rank_reduces_its_partition_from_the_heap(W, M, N, K, order, n_comm, consumer_tma):
    plans = [E.Plan(M, N, K, W, order, n_comm, rank=q, consumer_tma=consumer_tma) for q in range(W)]
    heap = Heap(plans[0], W, M, N)
    Q = plans[0].counts()["Q"]
    R = M // W
    for call in (1, 2, 3):  # both buffers, and a flag value that must grow
        epoch = call
        wls = _rank_workloads(W, M, N, K, call)
        ops = [I.make_operands(wl, device="cuda") for wl in wls]
        # phase 1: every producer alone
        for q in range(W):
            plans[q].gemm_rs_pull(ops[q][0], ops[q][1], heap.mem, heap.stride, epoch, None, produce_only=True)
            st = plans[q].last_status()
            assert st["flags_published"] == plans[q].counts()["flags_published"]
        torch.cuda.synchronize()
        C, S, stored = [], [], []
        for q in range(W):
            Ab, Bb = I.bits(ops[q][0]), I.bits(ops[q][1])
            C.append(O.partial_gemm(Ab, Bb))
            S.append(O.abs_gemm(Ab, Bb))
            stored.append(I.bits(heap.partial(q, epoch)).copy())
            got = O.bf16_bits_to_f64(stored[q])
            assert (np.abs(got - C[q]) <= O.tolerance(C[q], S[q])).all()
        # every flag of every destination carries the call's number
        for d in range(W):
            assert (heap.flags(d, Q) == epoch).all()
        # phase 2: full calls, one rank at a time
        outs = []
        for k in range(W):
            heap.flags(k, Q)[k].zero_()  # the rank's own flags: its consumers wait for its producer
            out = torch.full((R, N), float("nan"), dtype=torch.bfloat16, device="cuda")
            plans[k].gemm_rs_pull(ops[k][0], ops[k][1], heap.mem, heap.stride, epoch, out)
            st = plans[k].last_status()
            assert st["tiles_reduced"] == plans[k].counts()["n_reduce"] and st["tiles_pushed"] == 0
            torch.cuda.synchronize()
            assert (I.bits(heap.partial(k, epoch)) == stored[k]).all()  # the producer is deterministic
            assert (heap.flags(k, Q) == epoch).all()
            # ReduceTile on the W stored contributions (in the heap every contribution, the rank's
            # own too, is a bf16 tile; each was checked against the float64 product above)
            peers_bits = np.stack([stored[q] for q in range(W) if q != k])
            own = O.bf16_bits_to_f64(stored[k])
            ref_out, _ = O.reduce_scatter_ref(own, peers_bits, k, W)
            tol = O.tolerance(ref_out, O.out_magnitude_sum(np.abs(own), peers_bits, k, W))
            got = O.bf16_bits_to_f64(I.bits(out))
            assert np.isfinite(got).all()
            assert (np.abs(got - ref_out) <= tol).all(), f"rank {k}: worst {np.max(np.abs(got - ref_out) / tol):.3f}"
            outs.append(got)
        # the W shards together are the reduce-scatter of the whole product (K split over the ranks)
        A_full = np.concatenate([O.bf16_bits_to_f64(I.bits(a)) for a, _ in ops], axis=1)
        B_full = np.concatenate([O.bf16_bits_to_f64(I.bits(b)) for _, b in ops], axis=1)
        whole = A_full @ B_full.T
        # each stored contribution is within its own tolerance of the float64 partial; the
        # reduction adds one more rounding of the sum
        bound = 4e-3 * np.abs(whole) + sum(4.1e-3 * np.abs(c) + 1e-3 * s for c, s in zip(C, S))
        assert (np.abs(np.concatenate(outs, axis=0) - whole) <= bound).all()
    for p in plans:
        p.destroy()


def test_a_contribution_that_never_arrives_times_out_with_a_status():
    W, M, N, K = 2, 512, 256, 64
    plan = E.Plan(M, N, K, W, 1, 0, rank=0, wait_budget_ns=2_000_000)
    heap = Heap(plan, W, M, N, pad=0)
    A, Bm = I.make_operands(_rank_workloads(W, M, N, K, 1)[0], device="cuda")
    out = torch.empty(M // W, N, dtype=torch.bfloat16, device="cuda")
    plan.gemm_rs_pull(A, Bm, heap.mem, heap.stride, 1, out)  # rank 1 never produced
    with pytest.raises(E.EntwineError) as ei:
        plan.last_status()
    assert ei.value.code == E.ERR_TIMEOUT
    # the context is still usable, and the plan works once the contribution is there
    other = E.Plan(M, N, K, W, 1, 0, rank=1)
    A1, B1 = I.make_operands(_rank_workloads(W, M, N, K, 1)[1], device="cuda")
    other.gemm_rs_pull(A1, B1, heap.mem, heap.stride, 2, None, produce_only=True)
    other.last_status()
    plan.gemm_rs_pull(A, Bm, heap.mem, heap.stride, 2, out)
    st = plan.last_status()
    assert st["tiles_reduced"] == plan.counts()["n_reduce"]
    plan.destroy()
    other.destroy()


def test_bad_arguments_are_refused():
    W, M, N, K = 2, 512, 256, 64
    plan = E.Plan(M, N, K, W, 1, 0)
    heap = Heap(plan, W, M, N, pad=0)
    A, Bm = I.make_operands(_rank_workloads(W, M, N, K, 1)[0], device="cuda")
    out = torch.empty(M // W, N, dtype=torch.bfloat16, device="cuda")
    for args in ((heap.mem, heap.stride - 256, 1, out),       # stride below a segment
                 (heap.mem, heap.stride + 16, 1, out),        # stride not a multiple of 256
                 (heap.mem.data_ptr() + 16, heap.stride, 1, out),  # misaligned heap
                 (heap.mem, heap.stride, 0, out),             # epoch 0
                 (heap.mem, heap.stride, 1, None)):           # no output for a full call
        with pytest.raises(E.EntwineError) as ei:
            plan.gemm_rs_pull(A, Bm, *args)
        assert ei.value.code == E.ERR_INVALID
    coarse = E.Plan(M, N, K, W, 1, 0, release_group=4)
    with pytest.raises(E.EntwineError):
        coarse.gemm_rs_pull(A, Bm, heap.mem, heap.stride, 1, out)
    plan.destroy()
    coarse.destroy()


def test_full_size_attention_shape_rank_by_rank():
    """The benchmark's shape (W=4, 4096 x 4096 x 1024) in pull mode, all four ranks.  Sampled
    rows of every stored partial against the float64 oracle; for every element, each rank's
    shard is the order-exact fp32 sum of the stored contributions (own first, peers ascending)."""
    W, M, N, K = 4, 4096, 4096, 1024
    R = M // W
    plans = [E.Plan(M, N, K, W, 1, 0, rank=q) for q in range(W)]
    heap = Heap(plans[0], W, M, N, pad=0)
    Q = plans[0].counts()["Q"]
    rng = np.random.default_rng(5)
    rows = np.unique(np.concatenate([np.array([d * R, d * R + R - 1]) for d in range(W)] + [rng.integers(0, M, 40)]))
    for epoch in (1, 2):
        ops = [I.make_operands(I.Workload(f"pull_full{q}", W, M, N, K, "normal", "normal_fanin", 14, 4 * epoch + q),
                               device="cuda") for q in range(W)]
        for q in range(W):
            plans[q].gemm_rs_pull(ops[q][0], ops[q][1], heap.mem, heap.stride, epoch, None, produce_only=True)
            plans[q].last_status()
        torch.cuda.synchronize()
        stored = [heap.partial(q, epoch).clone() for q in range(W)]
        for q in range(W):
            Ab, Bb = I.bits(ops[q][0][rows]), I.bits(ops[q][1])
            C_rows, S_rows = O.partial_gemm(Ab, Bb), O.abs_gemm(Ab, Bb)
            got = O.bf16_bits_to_f64(I.bits(stored[q][rows]))
            assert (np.abs(got - C_rows) <= O.tolerance(C_rows, S_rows)).all()
        for k in range(W):
            assert bool((heap.flags(k, Q) == epoch).all())
            heap.flags(k, Q)[k].zero_()
            out = torch.full((R, N), float("nan"), dtype=torch.bfloat16, device="cuda")
            plans[k].gemm_rs_pull(ops[k][0], ops[k][1], heap.mem, heap.stride, epoch, out)
            st = plans[k].last_status()
            assert st["tiles_reduced"] == plans[k].counts()["n_reduce"] and st["tiles_pushed"] == 0
            assert torch.equal(heap.partial(k, epoch), stored[k])
            acc = stored[k][k * R:(k + 1) * R].float()
            for q in range(W):
                if q != k:
                    acc = acc + stored[q][k * R:(k + 1) * R].float()
            assert torch.equal(out, acc.to(torch.bfloat16))
    for p in plans:
        p.destroy()
