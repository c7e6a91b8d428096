"""Block-partition planner of the oracle.  TEST INFRASTRUCTURE ONLY.

Written independently of the library's planner from Section 4.1 of the paper:
  (1) embedding and attention-output blocks: no momentum;
  (2) query, key and MLP blocks: low-rank momentum with correction;
  (3) value blocks: full momentum.
Section 5.1 adds: rank r = 5% (read as floor(5 min(m,n) / 100), at least 1) and a
learning rate multiplier 0.75 for blocks without momentum.  The Adam-mini
combination keeps one second-moment scalar per group: one per attention head
for query/key, one per output row for value / attention-output / MLP, one per
token row for embeddings and output heads, one per 1-D tensor.

Tensors the partition does not mention: 1-D tensors get full momentum and no
weight decay; position embeddings and an untied output head are treated as
embeddings; a fused [3d, d] QKV weight is split by rows into Q, K, V blocks.
Every tensor starts at a multiple of 8 elements in the flat buffer.
"""
from __future__ import annotations

from typing import List, Sequence

from .adapm_oracle import Block, MOM_NONE, MOM_FULL, MOM_LOWRANK, V_ELEMENT, V_BLOCKMEAN

# role numbers, restated here so that this file depends on nothing else
EMBED, Q, K, V, QKV_FUSED, ATTN_OUT, MLP, LM_HEAD, VECTOR, OTHER = range(10)
ALIGN = 8


def select_rank(rows: int, cols: int, rank_pct: int, rank_override: int = 0) -> int:
    lo = min(rows, cols)
    if rank_override > 0:
        return min(rank_override, lo)
    return max(1, (rank_pct * lo) // 100)


def plan(tensors: Sequence, weight_decay: float, rank_pct: int = 5, blockmean: bool = True,
         rank_override: int = 0) -> List[Block]:
    """tensors: objects with .role .rows .cols .heads, in storage order."""
    out: List[Block] = []
    cursor = 0
    for t in tensors:
        cursor = -(-cursor // ALIGN) * ALIGN
        pieces = []   # (role, row offset, rows)
        if t.role == QKV_FUSED:
            if t.rows % 3:
                raise ValueError("fused QKV rows must be a multiple of 3")
            d = t.rows // 3
            pieces = [(Q, 0, d), (K, d, d), (V, 2 * d, d)]
        else:
            pieces = [(t.role, 0, t.rows)]
        for role, r0, rows in pieces:
            b = Block(rows=rows, cols=t.cols, offset=cursor + r0 * t.cols)
            if b.offset % ALIGN:
                raise ValueError("block offset is not a multiple of 8 elements")
            if role in (EMBED, LM_HEAD, ATTN_OUT):
                b.mom_mode, b.lr_scale, b.weight_decay, group = MOM_NONE, 0.75, weight_decay, 1
            elif role in (Q, K):
                b.mom_mode, b.lr_scale, b.weight_decay = MOM_LOWRANK, 1.0, weight_decay
                group = rows // t.heads if (t.heads > 0 and rows % t.heads == 0) else 1
            elif role == MLP:
                b.mom_mode, b.lr_scale, b.weight_decay, group = MOM_LOWRANK, 1.0, weight_decay, 1
            elif role == V or role == OTHER:
                b.mom_mode, b.lr_scale, b.weight_decay, group = MOM_FULL, 1.0, weight_decay, 1
            elif role == VECTOR:
                b.mom_mode, b.lr_scale, b.weight_decay, group = MOM_FULL, 1.0, 0.0, 0
            else:
                raise ValueError(f"unknown role {role}")
            if b.mom_mode == MOM_LOWRANK:
                b.rank = select_rank(b.rows, b.cols, rank_pct, rank_override)
            if blockmean:
                b.v_mode, b.v_group_rows = V_BLOCKMEAN, group
            else:
                b.v_mode, b.v_group_rows = V_ELEMENT, 0
            out.append(b)
        cursor += t.rows * t.cols
    return out


def total_elems(tensors: Sequence) -> int:
    """Length of the flat parameter / gradient buffer, padding included."""
    cursor = 0
    for t in tensors:
        cursor = -(-cursor // ALIGN) * ALIGN + t.rows * t.cols
    return -(-cursor // ALIGN) * ALIGN
