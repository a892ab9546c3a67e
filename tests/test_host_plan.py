"""CPU tests of the C-ABI library's host logic: every declared symbol is exported, shapes are
validated, and the exported integer tables equal the oracle's bit for bit (no GPU needed:
without a device a plan is host-only)."""
import ctypes
import itertools
import os
import re

import numpy as np
import pytest

from oracle import entwine_oracle as O
from paper_2609_11562_b200 import build as B

B.build()
from paper_2609_11562_b200 import entwine as E  # noqa: E402

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "entwine.h")).read()
    declared = set(re.findall(r"\b(entwine_[a-z_]+)\s*\(", header))
    declared.discard("entwine_plan_s")
    assert declared == set(E.SYMBOLS)
    lib = ctypes.CDLL(E.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert E.strerror(E.ERR_TIMEOUT).startswith("a device-side wait")
    assert "unknown" in E.strerror(-99)


@pytest.mark.parametrize("args", [
    (256, 256, 128, 1, 1, 4),       # W < 2
    (384, 256, 128, 2, 1, 4),       # M not a multiple of 128*W
    (256, 192, 128, 2, 1, 4),       # N not a multiple of 128
    (256, 256, 72, 2, 1, 4),        # K not a multiple of 16
    (256, 256, 128, 2, 7, 4),       # unknown tile order
    (256, 256, 128, 2, 1, -1),      # negative budget
    (256, 256, 128, 2, 1, 100000),  # more communication SMs than SMs
    (0, 256, 128, 2, 1, 4),
])
def test_plan_rejects_bad_arguments(args):
    with pytest.raises(E.EntwineError) as e:
        E.Plan(*args)
    assert e.value.code == E.ERR_INVALID


def test_options_validation_and_default_block_width():
    p = E.Plan(256, 384, 128, 2, E.ORDER_INTERLEAVED, 4, num_sms=148)
    assert p.counts()["cpb"] == 1          # N=384 only admits BN=128
    with pytest.raises(E.EntwineError):
        p.set_option(E.OPT_BLOCK_N, 256)
    with pytest.raises(E.EntwineError):
        p.set_option(E.OPT_RANK, 2)
    with pytest.raises(E.EntwineError):
        p.set_option(999, 0)
    with pytest.raises(E.EntwineError):
        p.set_option(E.OPT_WITHHOLD_PEER, (0 << 32) | 1)   # rank 0 is the emulated rank
    p.set_option(E.OPT_WITHHOLD_PEER, (1 << 32) | 1)
    p.set_option(E.OPT_WITHHOLD_PEER, -1)
    p.destroy()


CASES = [(256, 256, 128, 2), (512, 768, 64, 4), (384, 384, 64, 3), (2048, 1280, 64, 4),
         (4096, 4096, 1024, 4), (8192, 8192, 3584, 8), (16384, 5120, 512, 8)]


@pytest.mark.parametrize("M,N,K,W", CASES)
def test_exported_tables_equal_oracle(M, N, K, W):
    big = M * N > 2 ** 22
    orders = (E.ORDER_ROW_MAJOR, E.ORDER_INTERLEAVED, E.ORDER_M_MAJOR)
    bns = [bn for bn in (128, 256) if N % bn == 0]
    ranks = (W - 1,) if big else (0, W - 1)
    budgets = (20,) if big else (0, 1, 4, 24)
    for order, BN, r, n_comm in itertools.product(orders, bns, ranks, budgets):
        p = E.Plan(M, N, K, W, order, n_comm, num_sms=148, block_n=BN, rank=r)
        c = p.counts()
        x = c["x"]
        assert x == (148 if n_comm == 0 else n_comm)
        # CTA-pair tiles (two blocks sharing a block column) need an even number of producers
        rowsT = M // W // 128
        pair = BN == 256 and ((order == E.ORDER_INTERLEAVED and W % 2 == 0) or
                              (order == E.ORDER_ROW_MAJOR and rowsT % 2 == 0) or
                              (order == E.ORDER_M_MAJOR and (W * rowsT) % 2 == 0))
        want_g = (148 - n_comm) & ~1 if pair else 148 - n_comm
        assert c["n_gemm_ctas"] == want_g and c["n_comm_ctas"] == n_comm
        s = O.schedule(M, N, W, BN, order)
        g = s["geom"]
        want_order = np.stack([s["mb"], s["nb"], s["d"], s["l"]], axis=1).astype(np.int32)
        assert (p.export(E.EXPORT_ORDER).reshape(-1, 4) == want_order).all()
        assert (p.export(E.EXPORT_TILES).reshape(-1, g.cpb) == s["tiles"]).all()
        assert (p.export(E.EXPORT_FLAG_SEQ).reshape(-1, 3) == O.flag_sequence(s, r)).all()
        table, offs, peer_offs = O.index_maps(s, r, x)
        assert (p.export(E.EXPORT_LIST_OFFS) == offs).all()
        assert (p.export(E.EXPORT_TASKS).reshape(-1, 8) == table).all()
        assert (p.export(E.EXPORT_PEER_OFFS).reshape(-1, W - 1) == peer_offs).all()
        oc = O.traffic_counts(s, r, x)
        for k in ("P_blk", "Q", "cpb", "x", "n_tasks", "n_reduce", "n_push", "flags_published",
                  "peer_flags_prepublished", "min_flag_reads", "bytes_peer_read", "bytes_own_read",
                  "bytes_push_write", "bytes_out_write"):
            assert c[k] == oc[k], k
        p.destroy()


def test_list_count_option_follows_the_oracle():
    """x (the number of consumer lists) can be set apart from the number of consumer CTAs."""
    M, N, K, W, r = 2048, 1280, 64, 4, 3
    for order, x in itertools.product((0, 1), (1, 5, 40)):
        p = E.Plan(M, N, K, W, order, 8, num_sms=148, rank=r, lists=x)
        assert p.counts()["x"] == x
        s = O.schedule(M, N, W, 256, order)
        table, offs, peer_offs = O.index_maps(s, r, x)
        assert (p.export(E.EXPORT_LIST_OFFS) == offs).all()
        assert (p.export(E.EXPORT_TASKS).reshape(-1, 8) == table).all()
        p.destroy()


def test_fig3_example_through_the_library(golden):
    g = golden("fig3_example.txt")
    W, BN, M, N = (int(g[k][0][0]) for k in ("W", "BN", "M", "N"))
    x, r = int(g["x"][0][0]), int(g["rank"][0][0])
    p = E.Plan(M, N, 64, W, E.ORDER_INTERLEAVED, x, num_sms=148, block_n=BN, rank=r)
    order = p.export(E.EXPORT_ORDER).reshape(-1, 4)
    tiles = p.export(E.EXPORT_TILES).reshape(-1, 2)
    for pp, d, ta, tb in ([int(v) for v in row] for row in g["visit"]):
        assert order[pp, 2] == d and list(tiles[pp]) == [ta, tb]
    tasks = p.export(E.EXPORT_TASKS).reshape(-1, 8)
    for j, key in enumerate(("C0", "C1")):
        red = [int(t[2]) for t in tasks if t[0] == 0 and t[4] == j]
        assert red == [int(v) for v in g[key][0]]
    p.destroy()
    # the push lists of both traversals, as the library's planner builds them
    for name, order in (("push_interleaved", E.ORDER_INTERLEAVED), ("push_grouped", E.ORDER_ROW_MAJOR)):
        p = E.Plan(M, N, 64, W, order, x, num_sms=148, block_n=BN, rank=r)
        tasks = p.export(E.EXPORT_TASKS).reshape(-1, 8)
        for j in range(2):
            want = [tuple(int(v) for v in e.split(":")) for e in g[f"{name}_C{j}"][0]]
            assert [(int(t[1]), int(t[2])) for t in tasks if t[0] == 1 and t[4] == j] == want
        p.destroy()


def test_launch_without_device_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    p = E.Plan(256, 256, 128, 2, E.ORDER_INTERLEAVED, 4, num_sms=148)
    with pytest.raises(E.EntwineError) as e:
        p.gemm_rs(16, 16, 16, 16, 16, stream=0)
    assert e.value.code == E.ERR_CUDA
    p.destroy()


def test_release_group_option_validation():
    """ENTWINE_OPT_RELEASE_GROUP accepts a block count >= 1, the partition and whole-output
    values, and nothing else; it leaves the plan's tables untouched."""
    p = E.Plan(1024, 1024, 256, 4, 1, 4, num_sms=148)
    before = p.export(E.EXPORT_TASKS).copy()
    for ok in (1, 2, 7, 1000, E.RELEASE_PARTITION, E.RELEASE_WHOLE):
        p.set_option(E.OPT_RELEASE_GROUP, ok)
    for bad in (0, -3, 1 << 25):
        with pytest.raises(E.EntwineError):
            p.set_option(E.OPT_RELEASE_GROUP, bad)
    assert np.array_equal(before, p.export(E.EXPORT_TASKS))
    p.destroy()
