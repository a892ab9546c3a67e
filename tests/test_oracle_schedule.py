"""Pins for the integer part of the oracle: schedule, flag sequence, consumer lists, index
maps and byte counts, against what the paper prints and what the mathematics fixes."""
import itertools
import os

import numpy as np
import pytest

from oracle import entwine_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _kv(golden, name):
    g = golden(name)
    return g


def test_fig3_worked_example(golden):
    g = golden("fig3_example.txt")
    W, BN, M, N = (int(g[k][0][0]) for k in ("W", "BN", "M", "N"))
    x, r = int(g["x"][0][0]), int(g["rank"][0][0])
    s = O.schedule(M, N, W, BN, O.ORDER_INTERLEAVED)
    assert s["geom"].Q == 6 and s["geom"].cpb == 2
    for p, d, ta, tb in ([int(v) for v in row] for row in g["visit"]):
        assert s["d"][p] == d
        assert list(s["tiles"][p]) == [ta, tb]
    # no other block visits rank 1's partition
    visits = [p for p in range(s["geom"].P_blk) if s["d"][p] == r]
    assert visits == [int(row[0]) for row in g["visit"]]
    assert [int(v) for v in g["first4_dest"][0]] == list(s["d"][:4])
    lists = O.consumer_lists(s, r, x)
    for j, key in enumerate(("C0", "C1")):
        red = [t for (kind, d, t, k) in lists[j] if kind == O.KIND_REDUCE]
        assert red == [int(v) for v in g[key][0]]
    # the reduce lists do not depend on the producer's order of partitions
    s2 = O.schedule(M, N, W, BN, O.ORDER_ROW_MAJOR)
    lists2 = O.consumer_lists(s2, r, x)
    for j in range(2):
        assert [t for (kind, d, t, k) in lists2[j] if kind == O.KIND_REDUCE] == \
               [t for (kind, d, t, k) in lists[j] if kind == O.KIND_REDUCE]
    # the push lists do: non-owned tiles are dealt out in the order their flags are published
    # (hand-written vectors for both traversals; numbering by (d, t) instead would fail the
    # interleaved one, numbering by position alone would fail the split between C0 and C1)
    for name, ls in (("push_interleaved", lists), ("push_grouped", lists2)):
        for j in range(2):
            want = [tuple(int(v) for v in e.split(":")) for e in g[f"{name}_C{j}"][0]]
            assert [(d, t) for (kind, d, t, k) in ls[j] if kind == O.KIND_PUSH] == want


def _longest_local_run(dest, r):
    best = cur = 0
    for d in dest:
        cur = cur + 1 if d == r else 0
        best = max(best, cur)
    return best


def test_fig1_worked_example(golden):
    g = golden("fig1_example.txt")
    W, BN, M, N = (int(g[k][0][0]) for k in ("W", "BN", "M", "N"))
    row = O.schedule(M, N, W, BN, O.ORDER_ROW_MAJOR)
    inter = O.schedule(M, N, W, BN, O.ORDER_INTERLEAVED)
    assert row["geom"].P_blk == 9 and row["geom"].Q == 3
    assert list(row["d"]) == [int(v) for v in g["contiguous_dest"][0]]
    assert list(inter["d"]) == [int(v) for v in g["interleaved_dest"][0]]
    for r in range(W):
        assert _longest_local_run(row["d"], r) == int(g["contiguous_longest_local_run"][0][0])
        assert _longest_local_run(inter["d"], r) == int(g["interleaved_longest_local_run"][0][0])


def test_printed_wave_counts(golden):
    g = golden("wave_counts.txt")
    rows = [v for k in g for v in [[k] + r for r in g[k]]]
    assert len(rows) >= 3
    for M, N, BN, sms, printed in rows:
        M, N, BN, sms = int(M), int(N), int(BN), int(sms)
        waves = O.wave_count(M, N, BN, sms)
        digits = len(printed.split(".")[1]) if "." in printed else 0
        assert round(waves, digits) == float(printed)
        # the block count of the schedule is the one the wave count is made of
        s = O.schedule(M, N, 8, BN, O.ORDER_INTERLEAVED)
        assert s["geom"].P_blk == round(waves * sms)


SHAPES = [(256, 256, 2), (512, 768, 4), (384, 384, 3), (1024, 512, 8), (2048, 1280, 4),
          (3072, 256, 8), (1536, 1024, 6)]


@pytest.mark.parametrize("M,N,W", SHAPES)
@pytest.mark.parametrize("BN", [128, 256])
def test_eq1_closed_form_and_bijection(M, N, W, BN):
    if N % BN:
        pytest.skip("N not a multiple of BN")
    s = O.schedule(M, N, W, BN, O.ORDER_INTERLEAVED)
    g = s["geom"]
    p = np.arange(g.P_blk)
    assert (s["d"] == p % W).all()            # Eq. 1
    assert (s["l"] == p // W).all()           # Eq. 1
    for order in (O.ORDER_ROW_MAJOR, O.ORDER_INTERLEAVED):
        s = O.schedule(M, N, W, BN, order)
        assert O.check_every_tile_once(s)
        # a block's rows lie inside its destination's partition; its columns inside N
        assert (s["mb"] // g.rowsT == s["d"]).all()
        assert (s["nb"] < g.nBn).all()
        # tile index <-> geometric position, independent of BN
        for pp in range(g.P_blk):
            for c in range(g.cpb):
                t = s["tiles"][pp, c]
                assert t // g.nTn == s["mb"][pp] - s["d"][pp] * g.rowsT
                assert t % g.nTn == s["nb"][pp] * g.cpb + c
        # inside one partition, blocks are visited with l ascending
        for d in range(W):
            ls = [s["l"][pp] for pp in range(g.P_blk) if s["d"][pp] == d]
            assert ls == list(range(g.Lb))
    # the two orders visit the same set of blocks
    a = O.schedule(M, N, W, BN, O.ORDER_ROW_MAJOR)
    b = O.schedule(M, N, W, BN, O.ORDER_INTERLEAVED)
    assert sorted(zip(a["mb"], a["nb"])) == sorted(zip(b["mb"], b["nb"]))
    # run-length of local blocks: Lb when grouped, 1 when interleaved (Sec. 2.2)
    for r in range(W):
        assert _longest_local_run(a["d"], r) == g.Lb
        assert _longest_local_run(b["d"], r) == 1


@pytest.mark.parametrize("M,N,W", SHAPES)
@pytest.mark.parametrize("BN", [128, 256])
def test_m_major_order_is_column_major_walk_of_the_block_grid(M, N, W, BN):
    """The ablation's baseline order (Sec. 5.3.1) written out as a brute-force enumeration:
    for every block column, every block row of the whole output from top to bottom."""
    if N % BN:
        pytest.skip("N not a multiple of BN")
    s = O.schedule(M, N, W, BN, O.ORDER_M_MAJOR)
    g = s["geom"]
    walk = [(row, col) for col in range(N // BN) for row in range(M // 128)]
    assert list(zip(s["mb"].tolist(), s["nb"].tolist())) == walk
    assert O.check_every_tile_once(s)
    assert (s["mb"] // g.rowsT == s["d"]).all()
    assert (s["l"] == (s["mb"] - s["d"] * g.rowsT) * g.nBn + s["nb"]).all()
    for pp in range(g.P_blk):
        for c in range(g.cpb):
            t = s["tiles"][pp, c]
            assert t // g.nTn == s["mb"][pp] - s["d"][pp] * g.rowsT
            assert t % g.nTn == s["nb"][pp] * g.cpb + c
    # same set of blocks as Eq. 1; consecutive local blocks come in runs of one partition's
    # block rows (rowsT), not Lb and not 1
    b = O.schedule(M, N, W, BN, O.ORDER_INTERLEAVED)
    assert sorted(zip(s["mb"], s["nb"])) == sorted(zip(b["mb"], b["nb"]))
    for r in range(W):
        # rank W-1's run at the bottom of one column is not followed by its own blocks; the
        # others likewise: every run is exactly one partition's rows of one block column
        assert _longest_local_run(s["d"], r) == g.rowsT


def test_tile_numbering_same_for_both_block_widths():
    # the consumer uses the same 128x128 tiles with either producer (Sec. 4.2)
    for order in (0, 1):
        a = O.schedule(512, 1024, 2, 128, order)
        b = O.schedule(512, 1024, 2, 256, order)
        fa = {(d, t) for (_, d, t) in O.flag_sequence(a, 0)}
        fb = {(d, t) for (_, d, t) in O.flag_sequence(b, 0)}
        assert fa == fb
        # a wide block = the two narrow blocks that share its row and column pair
        for p in range(b["geom"].P_blk):
            t0, t1 = b["tiles"][p]
            assert t1 == t0 + 1 and t0 % 2 == 0


@pytest.mark.parametrize("M,N,W", SHAPES)
@pytest.mark.parametrize("x", [1, 2, 3, 5, 8, 20, 64])
def test_consumer_lists_rule(M, N, W, x):
    for order, BN, r in itertools.product((0, 1), (128, 256), (0, W - 1)):
        if N % BN:
            continue
        s = O.schedule(M, N, W, BN, order)
        g = s["geom"]
        lists = O.consumer_lists(s, r, x)
        x_r = min(x, g.Q)
        red_all, push_all = [], []
        for j, lst in enumerate(lists):
            red = [t for (kind, d, t, k) in lst if kind == O.KIND_REDUCE]
            # block j handles j, j+x, j+2x, ... below Q (grid capped by the tile count)
            assert red == (list(range(j, g.Q, x_r)) if j < x_r else [])
            ks = [k for (_, _, _, k) in lst]
            assert ks == sorted(ks)
            red_all += red
            push_all += [(d, t) for (kind, d, t, k) in lst if kind == O.KIND_PUSH]
        assert sorted(red_all) == list(range(g.Q))
        assert sorted(push_all) == [(d, t) for d in range(W) if d != r for t in range(g.Q)]
        # push load is balanced to within one task
        sizes = [sum(1 for task in lst if task[0] == O.KIND_PUSH) for lst in lists]
        x_p = min(x, (W - 1) * g.Q)
        assert max(sizes[:x_p]) - min(sizes[:x_p]) <= 1


@pytest.mark.parametrize("M,N,W", SHAPES)
def test_eq2_volume_and_counts(M, N, W):
    for order, BN, r, x in itertools.product((0, 1), (128, 256), (0, W - 1), (4, 16)):
        if N % BN:
            continue
        s = O.schedule(M, N, W, BN, order)
        c = O.traffic_counts(s, r, x)
        assert c["bytes_peer_read"] == O.v_comm(M, N, W, 2)        # Eq. 2
        assert c["bytes_push_write"] == O.v_comm(M, N, W, 2)       # same volume, source side
        assert c["bytes_own_read"] == M * N * 2
        assert c["bytes_out_write"] == M * N * 2 // W
        assert c["flags_published"] == W * s["geom"].Q
        assert c["n_tasks"] == W * s["geom"].Q
        seq = O.flag_sequence(s, r)
        assert len({(d, t) for (_, d, t) in seq}) == len(seq) == W * s["geom"].Q
        assert (seq[:, 0] == r).all()


def test_eq4_is_eq2_over_eq3():
    M, N, K, W, s, phi = 8192, 8192, 2048, 8, 2, 250e12
    t_g = 2 * M * N * K / phi                              # Eq. 3
    assert O.b_req(W, s, phi, K) == pytest.approx(O.v_comm(M, N, W, s) / t_g, rel=1e-12)


def test_index_maps_scatter_bruteforce():
    """Walk the task table on a matrix whose entries are their own flat index: the gathered
    source elements must be exactly the rows of the destination partition, and the target
    positions must tile out_shard / send_bufs exactly once."""
    M, N, W, BN = 768, 384, 3, 128
    for order, r, x in itertools.product((0, 1), range(W), (1, 4)):
        s = O.schedule(M, N, W, BN, order)
        g = s["geom"]
        table, offs, peer_offs = O.index_maps(s, r, x)
        C = np.arange(M * N, dtype=np.int64)
        out = -np.ones(g.R * N, np.int64)
        send = -np.ones((W - 1, g.R * N), np.int64)
        peers_flat = np.arange((W - 1) * M * N, dtype=np.int64)
        i_red = 0
        for row in table:
            kind, d, t, k, j, src, slot, dst = (int(v) for v in row)
            assert offs[j] <= np.where((table == row).all(1))[0][0] < offs[j + 1]
            for i in range(O.T):
                src_row = C[src + i * N: src + i * N + O.T]
                if kind == O.KIND_REDUCE:
                    assert (out[dst + i * N: dst + i * N + O.T] == -1).all()
                    out[dst + i * N: dst + i * N + O.T] = src_row
                else:
                    assert (send[slot, dst + i * N: dst + i * N + O.T] == -1).all()
                    send[slot, dst + i * N: dst + i * N + O.T] = src_row
            if kind == O.KIND_REDUCE:
                ws = [w for w in range(W) if w != r]
                for qi, w in enumerate(ws):
                    po = int(peer_offs[i_red, qi])
                    # same (row, col) of the M x N buffer, in the peer's slot
                    assert po == O.peer_slot(w, r) * M * N + src
                    assert peers_flat[po] // (M * N) == qi
                i_red += 1
        Cm = C.reshape(M, N)
        assert (out.reshape(g.R, N) == Cm[r * g.R:(r + 1) * g.R]).all()
        ds = [d for d in range(W) if d != r]
        for slot, d in enumerate(ds):
            assert (send[slot].reshape(g.R, N) == Cm[d * g.R:(d + 1) * g.R]).all()


def test_geometry_rejects_bad_shapes():
    for bad in [(256, 256, 1, 128), (384, 256, 2, 128), (256, 192, 2, 128),
                (256, 384, 2, 256), (256, 256, 2, 64)]:
        with pytest.raises(ValueError):
            O.Geometry(*bad)
