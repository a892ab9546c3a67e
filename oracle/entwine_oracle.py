"""CPU oracle for the fused GEMM-ReduceScatter path of Entwine (one-rank emulation).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain reference that the CUDA
library is checked against.  Only the tests, the smoke check and the CPU-baseline /
reference legs of the benchmark may import it; the product path never does.  It
shares no code with the CUDA library: every formula below is written out here from
the paper, and the library's host code restates them independently in C++.

Notation (paper Sec. 3.1, Sec. 4.2):
  W      ranks; r = the emulated rank; d = destination rank of a block / tile
  R      = M / W rows per output partition
  T      = 128, edge of the square reduction tile (Sec. 4.2)
  BN     producer block width, 128 or 256 (Sec. 4.2); cpb = BN / 128 tiles per block
  nTn    = N / 128 tile columns; nBn = N / BN block columns
  rowsT  = R / 128 tile rows per partition
  Lb     = rowsT * nBn blocks per partition; P_blk = W * Lb producer blocks
  Q      = rowsT * nTn tiles per partition (Sec. 3.1, "Matching task order")
  p      logical producer-block position; l ("ell") = within-partition block index
  x      number of consumer (communication) blocks (Sec. 3.2)

Operand layout used throughout: A is [M, K] (K contiguous); B is the weight shard of a
row-parallel linear layer stored as [N, K] (K contiguous); the rank's partial output is
C = A . B^T of shape [M, N].

Parity status of each function (what pins it is in tests/test_oracle_*.py):
  schedule, flag_sequence          pinned: Eq. 1 closed form, the worked examples of Fig. 1
                                   and Fig. 3, the printed wave counts, bijection
  consumer_lists (reduce part)     pinned: Fig. 3 (C0 -> t0,t2,t4; C1 -> t1,t3,t5)
  consumer_lists (push part)       the paper has no push; the rule is this build's reading of
                                   Sec. 3.1's assignment applied to the non-owned tiles (see
                                   its docstring).  Pinned: hand-written lists for the Fig. 3
                                   shape in both traversals, coverage, balance
  index_maps, traffic_counts       pinned: Eq. 2 volume, brute-force scatter on tiny shapes
  partial_gemm, reduce_scatter_ref pinned: brute-force triple loop, identity / one-hot /
                                   zero special cases, concat(shards) == unsplit GEMM
  bf16_round                       pinned: hand-computed ties, torch's conversion
  staged_model                     diagnostic; pinned against reduce_scatter_ref within
                                   the rounding bound derived in its docstring
  rmsnorm_ref, layer_chain_ref     pinned: closed forms (constant rows, one-hot rows, scale
                                   invariance at eps = 0), torch's rms_norm in float64
  norm_task_order                  the paper evaluates the operator chain of Sec. 5.2.3 but does
                                   not fuse it; the band rule is this build's design (see its
                                   docstring).  Pinned: a hand-listed 2-band x 3-column case
"""
from __future__ import annotations

import numpy as np

T = 128  # reduction-tile edge (Sec. 4.2)

ORDER_ROW_MAJOR = 0    # partition-grouped traversal (Fig. 1, top)
ORDER_INTERLEAVED = 1  # Eq. 1 (Fig. 1, bottom)
ORDER_M_MAJOR = 2      # the producer kernel's default traversal in the order ablation (Sec. 5.3.1)

KIND_REDUCE = 0
KIND_PUSH = 1


# --------------------------------------------------------------------------------------
# geometry
# --------------------------------------------------------------------------------------
class Geometry:
    """Derived sizes for an M x N output split over W ranks with 128 x BN producer blocks.

    Constraints are the ones stated in Sec. 4.1: equal partitions whose row count is a
    multiple of 128, and an output width that is a multiple of 128 (and of BN).
    """

    def __init__(self, M: int, N: int, W: int, BN: int = 256):
        if W < 2:
            raise ValueError("W must be >= 2")
        if BN not in (128, 256):
            raise ValueError("BN must be 128 or 256")
        if M <= 0 or N <= 0 or M % (T * W) != 0:
            raise ValueError("M must be a positive multiple of 128*W")
        if N % T != 0 or N % BN != 0:
            raise ValueError("N must be a multiple of 128 and of BN")
        self.M, self.N, self.W, self.BN = M, N, W, BN
        self.R = M // W
        self.cpb = BN // T
        self.nTn = N // T
        self.nBn = N // BN
        self.rowsT = self.R // T
        self.Lb = self.rowsT * self.nBn
        self.P_blk = W * self.Lb
        self.Q = self.rowsT * self.nTn


def wave_count(M: int, N: int, BN: int, n_sms: int) -> float:
    """GEMM wave count = producer thread-block count / number of SMs (Sec. 5.4.1)."""
    return (M // T) * (N // BN) / n_sms


# --------------------------------------------------------------------------------------
# a1. tile schedule (Sec. 3.1, Eq. 1; Fig. 1; Fig. 3)
# --------------------------------------------------------------------------------------
def schedule(M: int, N: int, W: int, BN: int, order: int):
    """Logical producer order.

    Returns a dict of int32 arrays indexed by the logical position p:
      d[p], l[p]   destination rank and within-partition block index
      mb[p], nb[p] block row (units of 128 rows of the M x N output) and block column
                   (units of BN columns)
      tiles[p, c]  within-partition index t of the c-th 128 x 128 tile the block covers

    Interleaved order is Eq. 1: d = p mod W, l = floor(p / W).
    Row-major order is the partition-grouped traversal of Fig. 1 (top): all blocks of
    partition 0, then partition 1, ...
    M-major order is the baseline of the computation-order ablation (Sec. 5.3.1): the block
    grid of the whole output is walked down the rows first, one block column after another,
    ignoring partitions and the consumer's order.
    Inside a partition l walks the block grid with the column index fastest (the
    "N-major" consumer order of Sec. 5.3.1), and tiles are numbered row-major over the
    partition's 128 x 128 grid, so a 128 x 256 block covers two consecutive tile indices
    (Fig. 3: block p=1 on four ranks supplies t0 and t1).
    """
    g = Geometry(M, N, W, BN)
    d = np.zeros(g.P_blk, np.int32)
    l = np.zeros(g.P_blk, np.int32)
    mb = np.zeros(g.P_blk, np.int32)
    nb = np.zeros(g.P_blk, np.int32)
    tiles = np.zeros((g.P_blk, g.cpb), np.int32)
    for p in range(g.P_blk):
        if order == ORDER_INTERLEAVED:
            dp = p % W
            lp = p // W
        elif order == ORDER_ROW_MAJOR:
            dp = p // g.Lb
            lp = p % g.Lb
        elif order == ORDER_M_MAJOR:
            # the block grid of the whole M x N output walked with the row index fastest
            rows_all = W * g.rowsT           # block rows of the output
            row_all = p % rows_all
            col_all = p // rows_all
            dp = row_all // g.rowsT
            lp = (row_all % g.rowsT) * g.nBn + col_all
        else:
            raise ValueError("unknown tile order")
        row_in_part = lp // g.nBn   # tile row inside the partition
        col_blk = lp % g.nBn        # block column
        d[p], l[p] = dp, lp
        mb[p] = dp * g.rowsT + row_in_part
        nb[p] = col_blk
        for c in range(g.cpb):
            tiles[p, c] = row_in_part * g.nTn + col_blk * g.cpb + c
    return {"d": d, "l": l, "mb": mb, "nb": nb, "tiles": tiles, "geom": g}


def flag_sequence(sched, r: int):
    """Logical publication sequence of rank r (Sec. 3.1 "completion signal F[r,d,t]",
    Sec. 4.2: a wide block publishes both of its tile flags after all of its stores).

    Entry k = p*cpb + c is the triple (src=r, d, t).  Physical completion order is up to
    the GPU scheduler; only this logical sequence, its set and its length are fixed.
    """
    g = sched["geom"]
    seq = np.zeros((g.P_blk * g.cpb, 3), np.int32)
    for p in range(g.P_blk):
        for c in range(g.cpb):
            seq[p * g.cpb + c] = (r, sched["d"][p], sched["tiles"][p, c])
    return seq


def check_every_tile_once(sched) -> bool:
    """Every (destination, tile) pair is produced by exactly one (block, slot)."""
    g = sched["geom"]
    seen = np.zeros((g.W, g.Q), np.int64)
    for p in range(g.P_blk):
        for c in range(g.cpb):
            seen[sched["d"][p], sched["tiles"][p, c]] += 1
    return bool((seen == 1).all())


# --------------------------------------------------------------------------------------
# a2. consumer task lists (Sec. 3.1 "Matching task order", Sec. 3.2 "Communication budget")
# --------------------------------------------------------------------------------------
def consumer_lists(sched, r: int, x: int):
    """Per-consumer-block task lists of the emulated rank r.

    Reduce tasks (the paper's rule): the Q tiles of the rank's own partition are numbered
    in producer traversal order; with the grid capped by the tile count, x_r = min(x, Q),
    consumer block j handles tiles j, j + x_r, j + 2 x_r, ... in increasing order.

    Push tasks (this build's emulation of peers pulling this rank's tiles; the paper has
    no push, so this rule is a reading): the non-owned tiles are numbered u = 0, 1, ... in
    the rank's logical publication order; with x_p = min(x, (W-1) Q), consumer block
    u mod x_p copies the u-th one.

    Each block walks the merge of its two lists by publication index k = p*cpb + c, so it
    checks tiles in the order their producer blocks are issued.

    Returns a list (length x) of lists of tuples (kind, d, t, k).
    """
    g = sched["geom"]
    if x < 1:
        raise ValueError("x must be >= 1")
    x_r = min(x, g.Q)
    x_p = min(x, (g.W - 1) * g.Q)
    lists = [[] for _ in range(x)]
    u = 0
    for p in range(g.P_blk):
        dp = int(sched["d"][p])
        for c in range(g.cpb):
            t = int(sched["tiles"][p, c])
            k = p * g.cpb + c
            if dp == r:
                lists[t % x_r].append((KIND_REDUCE, dp, t, k))
            else:
                lists[u % x_p].append((KIND_PUSH, dp, t, k))
                u += 1
    for j in range(x):
        lists[j].sort(key=lambda task: task[3])
    return lists


def peer_slot(w: int, r: int) -> int:
    """Slot of rank w != r in the (W-1)-entry peer / send buffers: ranks in ascending
    order with r left out."""
    if w == r:
        raise ValueError("rank r has no slot in its own peer buffers")
    return w if w < r else w - 1


def index_maps(sched, r: int, x: int):
    """Flattened task table with element offsets (Sec. 4.1: contributions sit at matching
    offsets in every rank's buffer).

    One row per task, in list order (list 0 first): int64 columns
      0 kind, 1 d, 2 t, 3 k, 4 list j,
      5 src_off   element offset of the tile's first element in the rank's partial C[M,N]
      6 dst_slot  -1 for a reduce task; peer_slot(d, r) for a push task
      7 dst_off   element offset of the tile's first element in out_shard[R,N] (reduce)
                  or in send_bufs[dst_slot][R,N] (push)
    plus list_offsets (int32[x+1]) delimiting each block's rows, and peer_offs
    (int64[n_reduce, W-1]): for every reduce task, in table order, the element offset of
    the tile in peer_partials[W-1][M][N] for each peer in ascending rank order.
    """
    g = sched["geom"]
    lists = consumer_lists(sched, r, x)
    rows = []
    peer_rows = []
    list_offsets = np.zeros(x + 1, np.int32)
    for j, lst in enumerate(lists):
        for (kind, dp, t, k) in lst:
            trow, tcol = t // g.nTn, t % g.nTn
            src_off = (dp * g.R + trow * T) * g.N + tcol * T
            in_part_off = (trow * T) * g.N + tcol * T
            if kind == KIND_REDUCE:
                rows.append((kind, dp, t, k, j, src_off, -1, in_part_off))
                peer_rows.append([peer_slot(w, r) * g.M * g.N + src_off
                                  for w in range(g.W) if w != r])
            else:
                rows.append((kind, dp, t, k, j, src_off, peer_slot(dp, r), in_part_off))
        list_offsets[j + 1] = len(rows)
    table = np.array(rows, np.int64).reshape(-1, 8)
    peer_offs = np.array(peer_rows, np.int64).reshape(-1, g.W - 1)
    return table, list_offsets, peer_offs


def traffic_counts(sched, r: int, x: int, elem_bytes: int = 2):
    """Counts that the schedule fixes, derived by walking the task table.

    Returns a dict.  bytes_peer_read must equal Eq. 2's V_comm = (W-1)/W * M*N*s.
    """
    g = sched["geom"]
    table, list_offsets, peer_offs = index_maps(sched, r, x)
    tile_bytes = T * T * elem_bytes
    n_reduce = int((table[:, 0] == KIND_REDUCE).sum())
    n_push = int((table[:, 0] == KIND_PUSH).sum())
    return {
        "P_blk": g.P_blk,
        "Q": g.Q,
        "cpb": g.cpb,
        "x": x,
        "n_tasks": n_reduce + n_push,
        "n_reduce": n_reduce,
        "n_push": n_push,
        "flags_published": g.P_blk * g.cpb,          # one per (d, t), by rank r
        "peer_flags_prepublished": (g.W - 1) * g.Q,  # emulated peers
        "min_flag_reads": g.W * n_reduce + n_push,   # W per reduce task, 1 per push
        "bytes_peer_read": n_reduce * (g.W - 1) * tile_bytes,
        "bytes_own_read": (n_reduce + n_push) * tile_bytes,
        "bytes_push_write": n_push * tile_bytes,
        "bytes_out_write": n_reduce * tile_bytes,
    }


def v_comm(M: int, N: int, W: int, s: int) -> float:
    """Eq. 2: remote-read volume to finalise one 1/W output partition."""
    return (W - 1) / W * M * N * s


def b_req(W: int, s: int, phi: float, K: int) -> float:
    """Eq. 4: average bandwidth needed to move V_comm inside the GEMM window of Eq. 3."""
    return (W - 1) / W * s * phi / (2 * K)


# --------------------------------------------------------------------------------------
# bf16 helpers (own implementation; round-to-nearest-even)
# --------------------------------------------------------------------------------------
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """uint16 bfloat16 bit patterns -> float64 values (exact)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def bf16_round(v: np.ndarray) -> np.ndarray:
    """Round float64 values to the nearest bfloat16 (8 significant bits, ties to even) and
    return them as float64.  Valid for finite values in bf16's normal range, which is all
    this path produces."""
    v = np.asarray(v, np.float64)
    m, e = np.frexp(v)                 # v = m * 2**e, 0.5 <= |m| < 1
    q = np.rint(m * 256.0) / 256.0     # 8 significant bits; rint rounds ties to even
    return np.ldexp(q, e)


def f64_to_bf16_bits(v: np.ndarray) -> np.ndarray:
    """float64 values that are exactly representable in bf16 -> uint16 bit patterns."""
    f = np.asarray(v, np.float64).astype(np.float32)
    return (f.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


# --------------------------------------------------------------------------------------
# a4-a8. numeric reference (Sec. 2.1: row-parallel GEMM followed by ReduceScatter)
# --------------------------------------------------------------------------------------
def partial_gemm(A_bits: np.ndarray, B_bits: np.ndarray) -> np.ndarray:
    """One rank's partial contribution C = A . B^T in float64 (Sec. 2.1, Sec. 3.3).
    A_bits [M,K], B_bits [N,K]: bf16 bit patterns."""
    return bf16_bits_to_f64(A_bits) @ bf16_bits_to_f64(B_bits).T


def abs_gemm(A_bits: np.ndarray, B_bits: np.ndarray) -> np.ndarray:
    """S[i,j] = sum_k |a_ik * b_jk|, the magnitude sum in the tolerance."""
    return np.abs(bf16_bits_to_f64(A_bits)) @ np.abs(bf16_bits_to_f64(B_bits)).T


def reduce_scatter_ref(C_r: np.ndarray, peers_bits: np.ndarray, r: int, W: int):
    """Definition of the emulated rank's two results, in float64.

    C_r [M,N]: rank r's partial (float64).  peers_bits [W-1, M, N]: incoming partials of
    the other ranks in ascending rank order (bf16 bits); only rows of partition r are read.

    ref_out [R,N]      = C_r[partition r] + sum over peers of their rows of partition r
                         (ReduceScatter: sum over ranks, row partition r to rank r).
    ref_send [W-1,R,N] = C_r[partition d] for d != r ascending: what rank r contributes to
                         every other destination.
    """
    M, N = C_r.shape
    R = M // W
    ref_out = C_r[r * R:(r + 1) * R].copy()
    for q in range(W - 1):
        ref_out += bf16_bits_to_f64(peers_bits[q, r * R:(r + 1) * R])
    ref_send = np.stack([C_r[d * R:(d + 1) * R] for d in range(W) if d != r])
    return ref_out, ref_send


def tolerance(ref: np.ndarray, S: np.ndarray) -> np.ndarray:
    """Per-element bound |gpu - ref| <= 4e-3 |ref| + 1e-3 * S, where S is the sum of the
    magnitudes of everything that was added into the element."""
    return 4e-3 * np.abs(ref) + 1e-3 * S


def out_magnitude_sum(S_r: np.ndarray, peers_bits: np.ndarray, r: int, W: int) -> np.ndarray:
    """Magnitude sum for out_shard: the rank's own |a*b| products plus |P_w| for each
    pre-generated partial (the value of a sum whose magnitude sum is at least that)."""
    M = S_r.shape[0]
    R = M // W
    S = S_r[r * R:(r + 1) * R].copy()
    for q in range(W - 1):
        S += np.abs(bf16_bits_to_f64(peers_bits[q, r * R:(r + 1) * R]))
    return S


def staged_model(A_bits, B_bits, peers_bits, r: int, W: int):
    """Diagnostic model of the stored-contribution pipeline (Sec. 4.2, ReduceTile): the
    rank's partial is accumulated in fp32 and stored as bf16; the reducer starts from the
    local contribution, adds the peers in ascending rank order in fp32, and stores bf16.

    It differs from the float64 definition by three roundings: fp32 accumulation of K
    products, one bf16 rounding of C (relative 2^-9), one bf16 rounding of the sum
    (relative 2^-9), plus W-1 fp32 adds - all far inside `tolerance`.
    Returns (out [R,N], send [W-1,R,N]) as float64 values that are exact bf16 numbers.
    """
    A = bf16_bits_to_f64(A_bits).astype(np.float32)
    B = bf16_bits_to_f64(B_bits).astype(np.float32)
    C32 = A @ B.T
    Cb = bf16_round(C32.astype(np.float64))
    M = Cb.shape[0]
    R = M // W
    acc = Cb[r * R:(r + 1) * R].astype(np.float32)
    for q in range(W - 1):
        acc = acc + bf16_bits_to_f64(peers_bits[q, r * R:(r + 1) * R]).astype(np.float32)
    out = bf16_round(acc.astype(np.float64))
    send = np.stack([Cb[d * R:(d + 1) * R] for d in range(W) if d != r])
    return out, send


# --------------------------------------------------------------------------------------
# layer-level chain: ReduceScatter -> residual add -> RMSNorm (Sec. 5.2.3)
# --------------------------------------------------------------------------------------
def rmsnorm_ref(h: np.ndarray, weight: np.ndarray, eps: float) -> np.ndarray:
    """RMSNorm over the last axis, float64: h / sqrt(mean(h^2) + eps) * weight."""
    h = np.asarray(h, np.float64)
    ms = np.mean(h * h, axis=-1, keepdims=True)
    return h / np.sqrt(ms + eps) * np.asarray(weight, np.float64)


def layer_chain_ref(ref_out: np.ndarray, residual_bits: np.ndarray, weight_bits: np.ndarray,
                    eps: float):
    """The operator chain that follows the ReduceScatter in the attention-output layer
    (Sec. 5.2.3): hidden = reduce-scattered output + residual; normed = RMSNorm(hidden).

    ref_out [R,N] float64 (reduce_scatter_ref); residual [R,N] and weight [N] as bf16 bits.
    Returns (hidden, normed) in float64, the definition with no intermediate rounding.
    """
    hidden = ref_out + bf16_bits_to_f64(residual_bits)
    return hidden, rmsnorm_ref(hidden, bf16_bits_to_f64(weight_bits), eps)


def norm_task_order(M: int, N: int, W: int):
    """Normalisation tasks of the emulated rank in the order they are handed out: one per
    128 x 128 tile of the rank's partition, tile row (a band of 128 complete rows) by tile
    row, tile column fastest.  A band's tasks may run once all nTn tiles of the band are
    reduced.  Returns int32 [Q, 2] of (band, tile column)."""
    rowsT = M // W // T
    nTn = N // T
    return np.array([(b, tc) for b in range(rowsT) for tc in range(nTn)], np.int32).reshape(-1, 2)


# --------------------------------------------------------------------------------------
# whole path, as the emulated rank runs it
# --------------------------------------------------------------------------------------
def gemm_rs(A_bits, B_bits, peers_bits, r: int, W: int, BN: int, order: int, x: int,
            rows=None):
    """All of the path for rank r: schedule, flag sequence, task table, float64 results.

    `rows`, if given, restricts the numeric part to those rows of the M x N partial (an
    index array); the integer part is always complete.  Returns a dict.
    """
    M, K = A_bits.shape
    N = B_bits.shape[0]
    sched = schedule(M, N, W, BN, order)
    out = {
        "sched": sched,
        "flags": flag_sequence(sched, r),
        "maps": index_maps(sched, r, x),
        "counts": traffic_counts(sched, r, x),
    }
    if rows is None:
        C = partial_gemm(A_bits, B_bits)
        S = abs_gemm(A_bits, B_bits)
        ref_out, ref_send = reduce_scatter_ref(C, peers_bits, r, W)
        out.update(C=C, S=S, ref_out=ref_out, ref_send=ref_send,
                   S_out=out_magnitude_sum(S, peers_bits, r, W))
    else:
        out.update(C_rows=partial_gemm(A_bits[rows], B_bits),
                   S_rows=abs_gemm(A_bits[rows], B_bits))
    return out
