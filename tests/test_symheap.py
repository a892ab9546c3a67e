"""The symmetric heap of the pull-mode call, one process per rank.

CPU part (gloo, host-memory backend): descriptor exchange, uniform-stride mapping, zeroed
segments, visibility of a rank's writes in the other ranks' mappings, and the segment layout
the planner reports.  GPU part: two processes on one GPU map each other's device segments
through the CUDA virtual-memory API and run the pull-mode call phase by phase (every producer
first, a host barrier, then the full calls), so that no kernel waits for another process's
kernel; each rank checks its shard against the oracle.
"""
import ctypes
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _init(rank, world, port):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)


def _cpu_worker(rank, world, port, q):
    _init(rank, world, port)
    from paper_2609_11562_b200 import symheap as SH
    seg_bytes = 70_000  # not a multiple of the page size
    heap = SH.SymmetricHeap(seg_bytes, rank, world, dist, SH.MemfdBackend())
    ok = heap.stride % 256 == 0 and heap.stride >= seg_bytes
    # every segment starts zeroed
    for w in range(world):
        ok = ok and ctypes.string_at(heap.segment(w), heap.stride) == bytes(heap.stride)
    dist.barrier()
    # a rank's writes into its own segment, and a "flag" written into every peer's segment
    ctypes.memset(heap.segment(rank) + 128, rank + 1, 1000)
    for w in range(world):
        ctypes.memset(heap.segment(w) + 4096 + 16 * rank, 0x40 + rank, 16)
    dist.barrier()
    for w in range(world):
        ok = ok and ctypes.string_at(heap.segment(w) + 128, 1000) == bytes([w + 1]) * 1000
        for src in range(world):
            ok = ok and ctypes.string_at(heap.segment(w) + 4096 + 16 * src, 16) == bytes([0x40 + src]) * 16
    dist.barrier()
    heap.close()
    q.put((rank, bool(ok), heap.stride))
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_segments_of_all_ranks_are_mapped_at_a_uniform_stride(world):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + (os.getpid() + 7 * world) % 2000
    procs = [ctx.Process(target=_cpu_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[0] for g in got] == list(range(world))
    assert all(g[1] for g in got)
    assert len({g[2] for g in got}) == 1  # the same stride everywhere


def test_segment_layout_reported_by_the_planner():
    sys.path.insert(0, ROOT)
    from paper_2609_11562_b200 import build as B
    B.build()
    from paper_2609_11562_b200 import entwine as E
    M, N, K, W = 1024, 768, 192, 4
    plan = E.Plan(M, N, K, W, 1, 0, num_sms=148)
    seg, flags_off = plan.heap_bytes()
    Q = plan.counts()["Q"]
    assert flags_off == 2 * M * N * 2          # two partial-output buffers, then the flags
    assert seg >= flags_off + W * Q * 4 and seg % 256 == 0
    plan.destroy()


def _gpu_worker(rank, world, port, q, consumer_tma=1):
    try:
        _init(rank, world, port)
        torch.cuda.set_device(0)  # both ranks on the one GPU
        from oracle import entwine_oracle as O
        from paper_2609_11562_b200 import entwine as E, inputs as I, symheap as SH
        M, N, K = 1024, 512, 128
        plan = E.Plan(M, N, K, world, 1, 0, rank=rank, wait_budget_ns=50_000_000, consumer_tma=consumer_tma)
        seg, flags_off = plan.heap_bytes()
        heap = SH.SymmetricHeap(seg, rank, world, dist, SH.VmmBackend(0))
        Q, R = plan.counts()["Q"], M // world
        worst = 0.0
        for epoch in (1, 2, 3):
            wl = I.Workload(f"heap_rank{rank}", world, M, N, K, "normal", "normal_total_fanin", 12, 8 * epoch + rank)
            A, Bm = I.make_operands(wl, device="cuda")
            plan.gemm_rs_pull(A, Bm, heap.base, heap.stride, epoch, None, produce_only=True)
            plan.last_status()
            torch.cuda.synchronize()
            dist.barrier()  # every rank's contribution and flags are in place
            flags = heap.cuda_tensor(rank, flags_off, world * Q * 4).view(torch.int32).view(world, Q)
            assert bool((flags == epoch).all())
            flags[rank].zero_()  # live synchronisation with this rank's own producer
            out = torch.full((R, N), float("nan"), dtype=torch.bfloat16, device="cuda")
            plan.gemm_rs_pull(A, Bm, heap.base, heap.stride, epoch, out)
            st = plan.last_status()
            assert st["tiles_reduced"] == plan.counts()["n_reduce"] and st["tiles_pushed"] == 0
            torch.cuda.synchronize()
            off = (epoch & 1) * M * N * 2
            stored = [I.bits(heap.cuda_tensor(w, off, M * N * 2).view(torch.bfloat16).view(M, N)).copy()
                      for w in range(world)]
            C = O.partial_gemm(I.bits(A), I.bits(Bm))
            S = O.abs_gemm(I.bits(A), I.bits(Bm))
            own = O.bf16_bits_to_f64(stored[rank])
            assert (np.abs(own - C) <= O.tolerance(C, S)).all()
            peers_bits = np.stack([stored[w] for w in range(world) if w != rank])
            ref, _ = O.reduce_scatter_ref(own, peers_bits, rank, world)
            tol = O.tolerance(ref, O.out_magnitude_sum(np.abs(own), peers_bits, rank, world))
            got = O.bf16_bits_to_f64(I.bits(out))
            assert np.isfinite(got).all()
            worst = max(worst, float(np.max(np.abs(got - ref) / tol)))
            dist.barrier()  # nobody starts the next call's producer before all have read this one
        plan.destroy()
        heap.close()
        q.put((rank, worst))
        dist.destroy_process_group()
    except Exception as e:  # the parent reports it
        q.put((rank, repr(e)))
        raise


@pytest.mark.gpu
@pytest.mark.parametrize("consumer_tma", [1, 0], ids=["peer_tiles_by_tma", "peer_tiles_by_plain_loads"])
def test_two_processes_share_device_segments_and_reduce_each_others_partials(consumer_tma):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 33500 + os.getpid() % 2000 + 7 * consumer_tma
    world = 2
    procs = [ctx.Process(target=_gpu_worker, args=(r, world, port, q, consumer_tma)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=300) for _ in range(world))
    for p in procs:
        p.join(timeout=120)
    assert all(isinstance(g[1], float) for g in got), got
    assert all(g[1] <= 1.0 for g in got), got
    assert all(p.exitcode == 0 for p in procs)
