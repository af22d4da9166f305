"""Seeded synthetic inputs and the workload table.  Serves the CUDA path's tests and benchmark and the
oracle's tests alike, and therefore holds none of the reshard's arithmetic: no shard rule, no packing,
no cast.  Whoever calls it brings the buffer sizes and the replica groups from its own side's layout
query.

Weights are drawn ~N(0, 0.02) from the stated seed, in fp32 and, for bf16 buffers, rounded by torch.  They
stand in for the paper's trained checkpoints (Llama-3.1-8B, Qwen3-32B), which a reshard's cost and
correctness do not depend on: it moves bits.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch


@dataclass(frozen=True)
class Shape:
    layers: int
    hidden: int
    heads: int
    kv_heads: int
    ffn: int
    vocab: int


TINY = Shape(2, 256, 4, 2, 688, 1024)              # head_dim 64
LLAMA_8B = Shape(32, 4096, 32, 8, 14336, 128256)   # Llama-3-8B-shaped
DENSE_32B = Shape(64, 5120, 40, 8, 27648, 152064)  # 32B-shaped decoder


QKV_GROUPED = 1            # layout flags of a plan: order of the rows inside a rank's fused blocks
GATE_UP_INTERLEAVED = 2
VOCAB_PADDED = 4


def layout_of(plan: tuple) -> int:
    return plan[3] if len(plan) > 3 else 0


@dataclass(frozen=True)
class Stage:
    """One model-stage's transition: (tp, pp, dtype[, layout]) -> (tp, pp, dtype[, layout]); dtype is "bf16" or
    "fp32", layout a mask of QKV_GROUPED | GATE_UP_INTERLEAVED (0 when absent)."""
    name: str
    shape: Shape
    seed: int
    src: tuple
    dst: tuple
    value_head: bool = False
    replicas: int = 1          # identical destination units (Extend, Split into replica units)
    n_opt: int = 0             # fp32 optimizer tensors per parameter that follow the same layout (Adam: 2)


@dataclass(frozen=True)
class Workload:
    name: str
    stages: tuple
    round_trip: bool = False   # run src->dst, then dst->src back, chained
    note: str = ""
    # plan change executed through the primitive-level transition DAG instead of one direct transition: per
    # stage (kind, [(tp, pp, first GPU), ...] current units, [...] target units); kind 0/1/2 = generation /
    # inference / training
    dag: tuple = ()


WORKLOADS = {
    # 1. tiny Merge, the case the oracle finishes at once
    "tiny_tp2pp1_to_tp1pp1": Workload("tiny_tp2pp1_to_tp1pp1", (
        Stage("tiny", TINY, 0, (2, 1, "bf16"), (1, 1, "bf16")),)),
    # 2. 8B Split: the configuration the metric is quoted on
    "8b_tp1pp1_to_tp4pp2": Workload("8b_tp1pp1_to_tp4pp2", (
        Stage("8b", LLAMA_8B, 1, (1, 1, "bf16"), (4, 2, "bf16")),)),
    # its reverse, the Merge direction of the headline
    "8b_tp4pp2_to_tp1pp1": Workload("8b_tp4pp2_to_tp1pp1", (
        Stage("8b", LLAMA_8B, 1, (4, 2, "bf16"), (1, 1, "bf16")),)),
    # 3. fp32 master weights -> bf16 generation layout (train -> rollout weight sync)
    "8b_fp32_tp2pp2_to_bf16_tp4pp1": Workload("8b_fp32_tp2pp2_to_bf16_tp4pp1", (
        Stage("8b_master", LLAMA_8B, 2, (2, 2, "fp32"), (4, 1, "bf16")),)),
    # 4. five PPO model-stages in one table; critic and reward carry a value head
    "ppo5_8b": Workload("ppo5_8b", (
        Stage("actor_generation", LLAMA_8B, 3, (4, 1, "bf16"), (2, 1, "bf16")),
        Stage("actor_training", LLAMA_8B, 4, (2, 1, "bf16"), (4, 2, "bf16")),
        Stage("critic", LLAMA_8B, 5, (2, 1, "bf16"), (4, 2, "bf16"), value_head=True),
        Stage("reference", LLAMA_8B, 6, (4, 1, "bf16"), (2, 1, "bf16")),
        Stage("reward", LLAMA_8B, 7, (4, 1, "bf16"), (2, 1, "bf16"), value_head=True),
    ), note="generation/inference stages Merge TP4->TP2; training stages Split TP2->TP4, PP1->PP2"),
    # 5. 32B round trip
    "32b_tp2pp4_to_tp8pp1_and_back": Workload("32b_tp2pp4_to_tp8pp1_and_back", (
        Stage("32b", DENSE_32B, 8, (2, 4, "bf16"), (8, 1, "bf16")),), round_trip=True),
}

# Profiling stand-ins, kept for the commands quoted under profiles/ (not BASELINE configurations, never a
# bench line): the 8B shape cut to 4 layers (3.85 GB each side: larger than L2, small enough for a multi-pass
# profiler capture; same tensor classes and piece sizes as the full Split), and a 244 MiB table of the size
# class that runs one warp per tile
LLAMA_8B_4L = Shape(4, 4096, 32, 8, 14336, 128256)
WORKLOADS["8b4l_tp1pp1_to_tp4pp2"] = Workload("8b4l_tp1pp1_to_tp4pp2", (
    Stage("8b4l", LLAMA_8B_4L, 1, (1, 1, "bf16"), (4, 2, "bf16")),))
WORKLOADS["8b4l_tp4pp2_to_tp1pp1"] = Workload("8b4l_tp4pp2_to_tp1pp1", (
    Stage("8b4l", LLAMA_8B_4L, 1, (4, 2, "bf16"), (1, 1, "bf16")),))
WORKLOADS["8b4l_fp32_tp2pp2_to_bf16_tp4pp1"] = Workload("8b4l_fp32_tp2pp2_to_bf16_tp4pp1", (
    Stage("8b4l_master", LLAMA_8B_4L, 2, (2, 2, "fp32"), (4, 1, "bf16")),))
# ... and the 8B layer shape with 2 layers and a 32K vocabulary (1.41 GB per side in bf16): what multi-pass
# captures run on, a few GB on the device in all; the per-layer tensor classes and piece sizes are the 8B model's
LLAMA_8B_2L_V32K = Shape(2, 4096, 32, 8, 14336, 32768)
WORKLOADS["8b2l_tp1pp1_to_tp4pp2"] = Workload("8b2l_tp1pp1_to_tp4pp2", (
    Stage("8b2l", LLAMA_8B_2L_V32K, 1, (1, 1, "bf16"), (4, 2, "bf16")),))
WORKLOADS["8b2l_fp32_tp2pp2_to_bf16_tp4pp1"] = Workload("8b2l_fp32_tp2pp2_to_bf16_tp4pp1", (
    Stage("8b2l_master", LLAMA_8B_2L_V32K, 2, (2, 2, "fp32"), (4, 1, "bf16")),))
MID_244MIB = Shape(2, 2048, 16, 8, 5632, 8192)
WORKLOADS["mid244_tp1pp1_to_tp4pp1"] = Workload("mid244_tp1pp1_to_tp4pp1", (
    Stage("mid244", MID_244MIB, 1, (1, 1, "bf16"), (4, 1, "bf16")),))

# the next rows: k destination units (Extend / replica units) and the EMU's optimizer state
WORKLOADS["8b_extend_tp4pp2_x2"] = Workload("8b_extend_tp4pp2_x2", (
    Stage("8b", LLAMA_8B, 11, (4, 2, "bf16"), (4, 2, "bf16"), replicas=2),),
    note="Extend: two new rank-aligned replicas of a TP4PP2 unit, every shard read once")
WORKLOADS["8b_fp32_tp2pp2_to_bf16_tp4pp1_x2"] = Workload("8b_fp32_tp2pp2_to_bf16_tp4pp1_x2", (
    Stage("8b_master", LLAMA_8B, 12, (2, 2, "fp32"), (4, 1, "bf16"), replicas=2),),
    note="weight sync of fp32 master weights to two bf16 generation units")
WORKLOADS["8b_state_adam_tp2pp2_to_tp4pp1"] = Workload("8b_state_adam_tp2pp2_to_tp4pp1", (
    Stage("8b_train", LLAMA_8B, 13, (2, 2, "bf16"), (4, 1, "bf16"), n_opt=2),),
    note="parameters (bf16) plus Adam's two fp32 moments, same layout, one table")

WORKLOADS["8b_grouped_fp32_tp2pp2_to_blocked_bf16_tp4pp1"] = Workload(
    "8b_grouped_fp32_tp2pp2_to_blocked_bf16_tp4pp1", (
        Stage("8b_master", LLAMA_8B, 14, (2, 2, "fp32", QKV_GROUPED | GATE_UP_INTERLEAVED), (4, 1, "bf16", 0)),),
    note="weight sync from a trainer's layout (grouped QKV, interleaved gate/up, fp32) to a generation layout")

WORKLOADS["8b_dag_tp4pp8_to_tp8pp2"] = Workload("8b_dag_tp4pp8_to_tp8pp2", (
    Stage("8b_reward", LLAMA_8B, 15, (4, 8, "bf16"), (8, 2, "bf16")),),
    dag=((1, ((4, 8, 0),), ((8, 2, 0),)),),
    note="the paper's layout example through its primitives: Split into four (TP4,PP2) replicas, two Destroys, "
         "Merge of the other two into (TP8,PP2); one launch, two dependency levels")

WORKLOADS["8b_tp4pp1_to_tp16pp1"] = Workload("8b_tp4pp1_to_tp16pp1", (
    Stage("8b_generation", LLAMA_8B, 16, (4, 1, "bf16"), (16, 1, "bf16")),),
    note="TP beyond the 8 kv heads: every kv head replicated on two ranks")

# scaled-down stand-ins with the same structure, for parity tests the oracle finishes in seconds
SMALL = Shape(4, 512, 8, 4, 1376, 2048)            # head_dim 64; several tiles and ragged tails
MICRO = Shape(8, 64, 8, 8, 128, 128)               # head_dim 8; brute-force sized, TP up to 8, PP up to 8


def element_size(dtype: str) -> int:
    return {"bf16": 2, "fp32": 4}[dtype]


def normal_bytes(nbytes: int, dtype: str, seed: int, device="cpu", std: float = 0.02,
                 chunk_elems: int = 1 << 27) -> torch.Tensor:
    """A uint8 buffer of ``nbytes`` whose contents are N(0, std) values of ``dtype`` from ``seed``."""
    es = element_size(dtype)
    assert nbytes % es == 0
    n = nbytes // es
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    out = torch.empty(n, dtype=tdt, device=device)
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    for lo in range(0, n, chunk_elems):
        hi = min(n, lo + chunk_elems)
        tmp = torch.empty(hi - lo, dtype=torch.float32, device=device)
        tmp.normal_(0.0, std, generator=g)
        out[lo:hi] = tmp.to(tdt)
        del tmp
    return out.view(torch.uint8)


def make_shards(sizes, dtype: str, seed: int, device="cpu") -> list:
    """One buffer per shard; shard i draws from a stream derived from (seed, i)."""
    return [normal_bytes(int(nb), dtype, seed * 1000003 + i, device) for i, nb in enumerate(sizes)]


def tie_replicas(bufs, groups) -> None:
    """Make replicated state identical: ``groups`` is a list of lists of (shard, byte offset, nbytes);
    the first member's bytes are copied over the others."""
    for grp in groups:
        s0, o0, n0 = grp[0]
        for s, o, n in grp[1:]:
            assert n == n0
            bufs[s][o:o + n] = bufs[s0][o0:o0 + n0]


def sentinel_shards(sizes, device="cpu", value: int = 0xA5) -> list:
    """Destination buffers pre-filled with a sentinel byte, so unwritten or over-written bytes show."""
    return [torch.full((int(nb),), value, dtype=torch.uint8, device=device) for nb in sizes]
