"""Seeded synthetic inputs for the GEMM-ReduceScatter path.

This module only draws random tensors; it holds none of the method's arithmetic and is
the one piece of code that both the CUDA path's callers and the CPU oracle's callers use,
so that the two sides see identical operands.

The paper's workloads are shapes taken from LLM configurations (Table 1: Llama 3 8B/70B,
Llama 3.1 405B, Qwen2.5-72B projections at tensor-parallel width 8); it uses no dataset and
no trained weights.  The tensors below stand in for them: activations with unit scale,
weights with std = fan_in^-1/2, incoming partials with unit scale.

Each named tensor has its own generator stream (seed + a fixed per-tensor offset), so one
tensor's shape never perturbs another's values.
"""
from __future__ import annotations

import dataclasses
import math

import torch

BASE_SEED = 20260911


@dataclasses.dataclass(frozen=True)
class Workload:
    """One GEMM-ReduceScatter problem of the emulated rank."""
    name: str
    W: int
    M: int
    N: int
    K: int            # K_local, the per-rank reduction dimension
    a_dist: str       # "uniform" | "normal" | "swiglu" | "normal_fanin"
    b_dist: str       # "uniform" | "normal_total_fanin" | "normal_fanin"
    config_id: int
    shape_index: int = 0

    @property
    def seed(self) -> int:
        return BASE_SEED + 1000 * self.config_id + self.shape_index

    @property
    def R(self) -> int:
        return self.M // self.W

    @property
    def flops(self) -> int:
        return 2 * self.M * self.N * self.K

    @property
    def comm_bytes(self) -> int:
        """Push (read + write of the W-1 non-owned partitions) plus reduce (W reads and one
        write of the owned partition), bf16: M*N*2*(3W-1)/W."""
        return self.M * self.N * 2 * (3 * self.W - 1) // self.W


# The four fixed configurations and the sweep grid.
TINY = Workload("tiny", 2, 256, 256, 128, "uniform", "uniform", 1)
ATTN_OUT = Workload("attn_out_proj", 4, 4096, 4096, 1024, "normal", "normal_total_fanin", 2)
MLP_DOWN = Workload("mlp_down_proj", 8, 8192, 8192, 3584, "swiglu", "normal_total_fanin", 3)
SHORT_K = Workload("short_k_comm_bound", 8, 16384, 5120, 512, "normal_fanin", "normal_fanin", 4)
CONFIGS = {w.name: w for w in (TINY, ATTN_OUT, MLP_DOWN, SHORT_K)}

SWEEP_M = (2048, 4096, 8192, 16384, 32768)
SWEEP_K = (512, 1024, 2048, 4096)
SWEEP_W = (2, 4, 8)
SWEEP_COMM_SMS = tuple(range(0, 33, 4))


def sweep_workloads():
    """The 60 shapes of the sweep configuration (N = 8192)."""
    out = []
    idx = 0
    for M in SWEEP_M:
        for K in SWEEP_K:
            for W in SWEEP_W:
                out.append(Workload(f"sweep_M{M}_K{K}_W{W}", W, M, 8192, K,
                                    "normal_fanin", "normal_fanin", 5, idx))
                idx += 1
    return out


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _draw(dist: str, rows: int, cols: int, wl: Workload, seed: int, device) -> torch.Tensor:
    g = _gen(seed, device)
    if dist == "uniform":
        t = torch.rand(rows, cols, generator=g, device=device, dtype=torch.float32) * 2 - 1
    elif dist == "normal":
        t = torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32)
    elif dist == "swiglu":
        gate = torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32)
        up = torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32)
        t = torch.nn.functional.silu(gate) * up
    elif dist == "normal_fanin":
        t = torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32)
        t = t * (1.0 / math.sqrt(wl.K))
    elif dist == "normal_total_fanin":
        t = torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32)
        t = t * (1.0 / math.sqrt(wl.K * wl.W))
    else:
        raise ValueError(dist)
    return t.to(torch.bfloat16)


def make_operands(wl: Workload, device="cpu", seed_offset: int = 0):
    """A [M,K] and B [N,K] (the rank's weight shard, K contiguous) in bf16."""
    s = wl.seed + seed_offset
    A = _draw(wl.a_dist, wl.M, wl.K, wl, s * 16 + 1, device)
    B = _draw(wl.b_dist, wl.N, wl.K, wl, s * 16 + 2, device)
    return A, B


def make_peer_partials(wl: Workload, device="cpu", seed_offset: int = 0) -> torch.Tensor:
    """The W-1 incoming partial outputs [W-1, M, N] in bf16, N(0,1), one stream per peer."""
    s = wl.seed + seed_offset
    out = torch.empty(wl.W - 1, wl.M, wl.N, dtype=torch.bfloat16, device=device)
    for q in range(wl.W - 1):
        g = _gen(s * 16 + 3 + q, device)
        # drawn in row chunks to bound the fp32 temporary
        step = max(1, (1 << 26) // wl.N)
        for r0 in range(0, wl.M, step):
            r1 = min(wl.M, r0 + step)
            out[q, r0:r1] = torch.randn(r1 - r0, wl.N, generator=g, device=device,
                                        dtype=torch.float32).to(torch.bfloat16)
    return out


def make_layer_inputs(wl: Workload, device="cpu"):
    """Inputs of the layer chain that follows the reduction: the residual stream [R, N] ~ N(0,1)
    and the RMSNorm weight [N] ~ 1 + 0.1 N(0,1), bf16, streams of their own."""
    s = wl.seed
    res = torch.randn(wl.R, wl.N, generator=_gen(s * 16 + 11, device), device=device,
                      dtype=torch.float32).to(torch.bfloat16)
    w = (1.0 + 0.1 * torch.randn(wl.N, generator=_gen(s * 16 + 12, device), device=device,
                                 dtype=torch.float32)).to(torch.bfloat16)
    return res, w


def bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 bit patterns on the host (what the oracle consumes)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view("uint16")
