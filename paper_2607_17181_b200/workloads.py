"""Seeded synthetic inputs shared by the oracle tests, the GPU parity tests and
the benchmark.

This module holds NONE of the method's arithmetic (no hashing, no matching, no
block-table copies): it only draws token ids, KV fill bytes, block tables,
session-replay schedules and weight-set shapes.  All randomness comes from
numpy's counter-based Philox generator seeded per configuration, so the CPU
oracle and the CUDA path always see identical bytes.

The shapes follow the workload statistics printed in the paper's Sec. 2.1 /
App. A (prompt length median 25K / p95 105K tokens, depth median 11 / p95 49
calls, 96.8% of continuations reusing more than half of the prior prefix); the
recorded agent traces themselves are not used.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

VOCAB = 151936                       # token ids are uniform in [0, VOCAB)
BASE_SEED = 0x7A1A51A                # seed = BASE_SEED + config id
HASH_SEED = 0x54414C41524941         # "TALARIA": stands for the model-name key


def rng(config_id: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[BASE_SEED + config_id, stream]))


@dataclass(frozen=True)
class KvShape:
    num_layers: int
    num_kv_heads: int
    block_tokens: int
    head_dim: int
    elt_bytes: int = 2
    num_planes: int = 2

    @property
    def chunk_bytes(self) -> int:
        """One block of one layer's K or V."""
        return self.num_kv_heads * self.block_tokens * self.head_dim * self.elt_bytes

    @property
    def bytes_per_block(self) -> int:
        return self.num_layers * self.num_planes * self.chunk_bytes

    @property
    def bytes_per_token(self) -> int:
        return self.bytes_per_block // self.block_tokens

    def blocks_for(self, tokens: int) -> int:
        return -(-tokens // self.block_tokens)


TINY = KvShape(num_layers=4, num_kv_heads=2, block_tokens=16, head_dim=64)
QWEN235 = KvShape(num_layers=94, num_kv_heads=4, block_tokens=16, head_dim=128)
QWEN235_B32 = KvShape(num_layers=94, num_kv_heads=4, block_tokens=32, head_dim=128)


def dense_strides(shape: KvShape, n_blocks: int, order: str) -> Tuple[int, int, int]:
    """(stride_layer, stride_plane, stride_block) in bytes of a dense host image.
    'LF' = layer-first (layer, plane, block); 'PF' = page-first (block, layer, plane)."""
    c = shape.chunk_bytes
    if order == "LF":
        return shape.num_planes * n_blocks * c, n_blocks * c, c
    if order == "PF":
        return shape.num_planes * c, c, shape.num_layers * shape.num_planes * c
    raise ValueError(order)


# ------------------------------------------------------------------ tokens


def tokens(g: np.random.Generator, n: int) -> np.ndarray:
    return g.integers(0, VOCAB, size=n, dtype=np.int32)


def continuation(g: np.random.Generator, sess: np.ndarray, total: int, shared: int) -> np.ndarray:
    """A prompt of `total` tokens whose first `shared` tokens equal the stored
    stream's and whose token at index `shared` is forced to differ (when both
    streams have one), so the longest common prefix is exactly `shared`."""
    assert 0 <= shared <= min(total, sess.size)
    out = tokens(g, total)
    out[:shared] = sess[:shared]
    if shared < total and shared < sess.size and out[shared] == sess[shared]:
        out[shared] = (int(sess[shared]) + 1) % VOCAB
    return out


# ---------------------------------------------------------------- KV bytes


def bf16_normal_bytes(g: np.random.Generator, nbytes: int) -> np.ndarray:
    """bf16 N(0,1) samples as raw bytes (round-to-nearest-even from fp32).  The
    content only has to differ from chunk to chunk so a misplaced copy shows."""
    assert nbytes % 2 == 0
    f = g.standard_normal(nbytes // 2, dtype=np.float32).view(np.uint32)
    r = ((f >> 16) & 1) + np.uint32(0x7FFF)
    return ((f + r) >> 16).astype(np.uint16).view(np.uint8)


def kv_pool(g: np.random.Generator, shape: KvShape, num_blocks: int) -> List[np.ndarray]:
    """One uint8 array per (layer, plane), each [num_blocks, kv_heads, block_tokens, head_dim]."""
    return [bf16_normal_bytes(g, num_blocks * shape.chunk_bytes)
            for _ in range(shape.num_layers * shape.num_planes)]


# ------------------------------------------------------------ block tables


def disjoint_tables(g: np.random.Generator, num_blocks: int, sizes: Sequence[int],
                    exclude: Optional[np.ndarray] = None) -> List[np.ndarray]:
    """Disjoint slices of one seeded permutation of the free block ids."""
    free = np.arange(num_blocks, dtype=np.int32)
    if exclude is not None and len(exclude):
        mask = np.ones(num_blocks, dtype=bool)
        mask[np.asarray(exclude)] = False
        free = free[mask]
    assert sum(sizes) <= free.size
    perm = g.permutation(free).astype(np.int32)
    out, at = [], 0
    for s in sizes:
        out.append(np.ascontiguousarray(perm[at:at + s]))
        at += s
    return out


def isolated_table(g: np.random.Generator, num_blocks: int, n: int) -> np.ndarray:
    """A heavily fragmented free list: only odd block ids, shuffled, so no two
    restored blocks are neighbours in the pool."""
    odd = np.arange(1, num_blocks, 2, dtype=np.int32)
    assert n <= odd.size
    return np.ascontiguousarray(g.permutation(odd)[:n].astype(np.int32))


# ------------------------------------------------------ session-replay mix


@dataclass
class Call:
    session: int
    index: int                 # call index inside its session
    prompt_tokens: int
    shared_tokens: int         # common prefix with the session's previous stream (0 for call 0)


def lognormal_sigma(median: float, p95: float) -> float:
    return math.log(p95 / median) / 1.6448536269514722


def session_replay(config_id: int = 4, n_sessions: int = 30, depth_median: float = 11,
                   depth_p95: float = 49, depth_max: int = 187, len_median: float = 25_000,
                   len_p95: float = 105_000, len_min: int = 256, len_max: int = 131_072,
                   p_high_reuse: float = 0.97) -> List[Call]:
    """Interleaved call schedule for a population of agent sessions."""
    g = rng(config_id)
    sd, sl = lognormal_sigma(depth_median, depth_p95), lognormal_sigma(len_median, len_p95)
    depths = np.clip(np.rint(np.exp(math.log(depth_median) + sd * g.standard_normal(n_sessions))),
                     1, depth_max).astype(int)
    per_session: List[List[Call]] = []
    for s in range(n_sessions):
        calls, prev = [], 0
        for k in range(int(depths[s])):
            t = int(np.clip(round(math.exp(math.log(len_median) + sl * g.standard_normal())),
                            len_min, len_max))
            if k == 0:
                shared = 0
            else:
                f = g.uniform(0.5, 1.0) if g.uniform() < p_high_reuse else g.uniform(0.0, 0.5)
                shared = min(int(f * prev), t - 1)
            calls.append(Call(s, k, t, shared))
            prev = t
        per_session.append(calls)
    # closed-loop interleaving: repeatedly pick a live session at random
    cursor = [0] * n_sessions
    order: List[Call] = []
    live = [s for s in range(n_sessions)]
    while live:
        s = live[int(g.integers(0, len(live)))]
        order.append(per_session[s][cursor[s]])
        cursor[s] += 1
        if cursor[s] == len(per_session[s]):
            live.remove(s)
    return order


# ------------------------------------------------------------- weight set


@dataclass
class WeightSet:
    sizes: List[int]                    # bytes per tensor, in physical order
    names: List[str] = field(default_factory=list)

    @property
    def total_bytes(self) -> int:
        return sum(self.sizes)


def moe_weight_set(num_layers: int = 94, num_experts: int = 128, expert_rows: int = 4096,
                   expert_cols: int = 192, hidden: int = 4096, q_heads: int = 8, kv_heads: int = 1,
                   head_dim: int = 128, vocab_shard: int = VOCAB // 8, elt: int = 2) -> WeightSet:
    """Per-rank share of a 235B-parameter MoE at TP=8: per layer 128 experts of
    three [4096 x 192] matrices, attention projections, router and two norms,
    plus the embedding and output-head shards."""
    sizes, names = [], []
    for l in range(num_layers):
        for name, nbytes in (("q_proj", hidden * q_heads * head_dim * elt),
                             ("k_proj", hidden * kv_heads * head_dim * elt),
                             ("v_proj", hidden * kv_heads * head_dim * elt),
                             ("o_proj", q_heads * head_dim * hidden * elt),
                             ("q_norm", head_dim * elt), ("k_norm", head_dim * elt),
                             ("input_norm", hidden * elt), ("post_norm", hidden * elt),
                             ("router", hidden * num_experts * elt)):
            sizes.append(nbytes)
            names.append(f"l{l}.{name}")
        for e in range(num_experts):
            for m in ("gate", "up", "down"):
                sizes.append(expert_rows * expert_cols * elt)
                names.append(f"l{l}.e{e}.{m}")
    sizes += [vocab_shard * hidden * elt, vocab_shard * hidden * elt, hidden * elt]
    names += ["embed", "lm_head", "final_norm"]
    return WeightSet(sizes, names)


def stage_plan(ws_sizes: Sequence[int], chunk_bytes: int, align: int = 256):
    """Cut a weight set into fixed-size staging chunks.  Returns a list of
    (offset, nbytes, chunk_id): tensors are laid out back to back at `align`
    and each tensor is cut into chunks of at most chunk_bytes (the last chunk of
    a tensor may be short).  The same offsets are used in the staging region,
    in the host copy and in the stable slots."""
    plan, at, cid = [], 0, 0
    for nbytes in ws_sizes:
        off = 0
        while off < nbytes:
            n = min(chunk_bytes, nbytes - off)
            plan.append((at + off, n, cid))
            cid += 1
            off += n
        at += -(-nbytes // align) * align
    return plan, at
