"""The tuner's table logic and budget-model arithmetic (no GPU), and one small tuning run (GPU)."""
import numpy as np
import pytest
import torch

from oracle import entwine_oracle as O
from paper_2609_11562_b200 import autotune as T
from paper_2609_11562_b200 import inputs as I


def test_model_bytes_match_the_oracle_counts():
    """Eq. 2's link volume and the emulation's consumer bytes against the oracle's walk of the
    task table; Eq. 4 against the oracle's closed form through T_G = 2MNK / phi (Eq. 3)."""
    for M, N, W in ((512, 512, 2), (2048, 1024, 8), (1536, 1024, 6)):
        s = O.schedule(M, N, W, 128 if N % 256 else 256, O.ORDER_INTERLEAVED)
        c = O.traffic_counts(s, W - 1, 7)
        assert T.link_bytes(M, N, W) == c["bytes_peer_read"] == O.v_comm(M, N, W, 2)
        total = c["bytes_peer_read"] + c["bytes_own_read"] + c["bytes_push_write"] + c["bytes_out_write"]
        assert T.comm_bytes(M, N, W) == total
        K, phi = 768, 1.2e15
        t_g = 2.0 * M * N * K / phi
        link_part = T.b_req(M, N, W, t_g) * T.link_bytes(M, N, W) / T.comm_bytes(M, N, W)
        assert np.isclose(link_part, O.b_req(W, 2, phi, K), rtol=1e-12)
    assert T.comm_bytes(I.ATTN_OUT.M, I.ATTN_OUT.N, I.ATTN_OUT.W) == I.ATTN_OUT.comm_bytes


def test_table_round_trip_and_fallback(tmp_path):
    table = {"format": 1, "device": "x", "shapes": {
        T.shape_key(4096, 4096, 1024, 4): {"best": {"tile_order": "row_major", "n_comm_sms": 16, "stages": 3,
                                                   "block_n": 128}}}}
    path = tmp_path / "sub" / "tuned.json"
    T.save_table(table, str(path))
    back = T.load_table(str(path))
    assert back == table
    assert T.launch_options(back, 4096, 4096, 1024, 4) == (0, 16, {"stages": 3, "block_n": 128})
    # unknown shape and no table: the default configuration
    assert T.launch_options(back, 2048, 4096, 1024, 4) == (1, 0, {})
    assert T.launch_options(None, 4096, 4096, 1024, 4) == (1, 0, {})
    bad = tmp_path / "bad.json"
    bad.write_text('{"format": 7}')
    with pytest.raises(ValueError):
        T.load_table(str(bad))


@pytest.mark.gpu
def test_tuner_picks_the_fastest_measured_point_and_it_is_correct():
    from paper_2609_11562_b200 import build as B
    B.build()
    from paper_2609_11562_b200 import entwine as E
    wl = I.Workload("tune_small", 4, 2048, 1024, 512, "normal", "normal_total_fanin", 9, 11)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    entry = T.tune_shape(wl, flush, iters=3, budgets=(0, 8), stages=(0, 4), ranks=(0, 3))
    pts = entry["points"]
    assert len(pts) >= 8 and all(p["fused_us"] > 0 for p in pts)
    assert entry["best_us"] == min(p["fused_us"] for p in pts)
    assert entry["gain_over_default"] >= 1.0
    m = entry["model"]
    assert m["comm_bytes"] == wl.comm_bytes and m["b_req_GBps_eq4"] > 0 and m["b_measured_GBps"] > 0
    # the chosen configuration computes the same result as the default one
    table = {"format": 1, "shapes": {T.shape_key(wl.M, wl.N, wl.K, wl.W): entry}}
    order, n_comm, opts = T.launch_options(table, wl.M, wl.N, wl.K, wl.W)
    A, Bm = I.make_operands(wl, device="cuda")
    P = I.make_peer_partials(wl, device="cuda")
    res = []
    for o, n, kw in ((order, n_comm, opts), (1, 0, {})):
        p = E.Plan(wl.M, wl.N, wl.K, wl.W, o, n, rank=1, **kw)
        out = torch.empty(wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
        send = torch.empty(wl.W - 1, wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
        p.gemm_rs(A, Bm, P, out, send)
        p.last_status()
        p.destroy()
        res.append((out, send))
    assert torch.equal(res[0][0], res[1][0]) and torch.equal(res[0][1], res[1][1])
