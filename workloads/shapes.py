"""Tensor tables of the five synthetic parameter sets.

Each set lists the tensors of a decoder-only language model in storage order,
row-major ``[rows, cols] = [out_features, in_features]`` (Algorithm 1 speaks of
"an m x n layer W"; m = rows).  Only shapes, roles and head counts are given
here; the momentum mode, rank and second-moment grouping of every tensor are
decided by a planner (the library's, and independently the oracle's).

Shapes follow the model families the paper trains (Section 5.1: GPT-2 124M to
1.5B, Llama 60M to 350M); the data sets and weights of those runs are not
needed for an optimizer step and are replaced by seeded random values.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List

# Tensor roles understood by the planners (Section 4.1 names the first six
# classes; VECTOR/OTHER cover what the paper's partition does not mention).
ROLE_EMBED = 0
ROLE_Q = 1
ROLE_K = 2
ROLE_V = 3
ROLE_QKV_FUSED = 4
ROLE_ATTN_OUT = 5
ROLE_MLP = 6
ROLE_LM_HEAD = 7
ROLE_VECTOR = 8
ROLE_OTHER = 9


@dataclass(frozen=True)
class Tensor:
    name: str
    role: int
    rows: int
    cols: int
    heads: int = 0          # attention heads, for Q / K / fused QKV tensors
    init: str = "normal"    # "normal" N(0, 0.02^2), "ones", "zeros"

    @property
    def numel(self) -> int:
        return self.rows * self.cols


@dataclass
class Workload:
    name: str
    tensors: List[Tensor]
    grad_dtype: str               # "f32" | "bf16"
    grad_recipe: str              # see gen.grad_for_tensor
    steps: int
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.95
    eps: float = 1e-8
    weight_decay: float = 0.1
    rank_pct: int = 5
    rank_override: int = 0        # >0: every low-rank block uses this rank
    v_mode: str = "blockmean"     # headline second-moment mode of the set
    notes: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def numel(self) -> int:
        return sum(t.numel for t in self.tensors)


def _gpt2(n_layer: int, d: int, heads: int, ffn: int, vocab: int, ctx: int) -> List[Tensor]:
    t: List[Tensor] = [
        Tensor("wte", ROLE_EMBED, vocab, d),          # tied with the output head
        Tensor("wpe", ROLE_EMBED, ctx, d),
    ]
    for i in range(n_layer):
        p = f"h{i}."
        t += [
            Tensor(p + "ln_1.weight", ROLE_VECTOR, 1, d, init="ones"),
            Tensor(p + "ln_1.bias", ROLE_VECTOR, 1, d, init="zeros"),
            Tensor(p + "attn.c_attn.weight", ROLE_QKV_FUSED, 3 * d, d, heads=heads),
            Tensor(p + "attn.c_attn.bias", ROLE_VECTOR, 1, 3 * d, init="zeros"),
            Tensor(p + "attn.c_proj.weight", ROLE_ATTN_OUT, d, d),
            Tensor(p + "attn.c_proj.bias", ROLE_VECTOR, 1, d, init="zeros"),
            Tensor(p + "ln_2.weight", ROLE_VECTOR, 1, d, init="ones"),
            Tensor(p + "ln_2.bias", ROLE_VECTOR, 1, d, init="zeros"),
            Tensor(p + "mlp.c_fc.weight", ROLE_MLP, ffn, d),
            Tensor(p + "mlp.c_fc.bias", ROLE_VECTOR, 1, ffn, init="zeros"),
            Tensor(p + "mlp.c_proj.weight", ROLE_MLP, d, ffn),
            Tensor(p + "mlp.c_proj.bias", ROLE_VECTOR, 1, d, init="zeros"),
        ]
    t += [
        Tensor("ln_f.weight", ROLE_VECTOR, 1, d, init="ones"),
        Tensor("ln_f.bias", ROLE_VECTOR, 1, d, init="zeros"),
    ]
    return t


def _llama(n_layer: int, d: int, heads: int, ffn: int, vocab: int, kv_heads: int = 0) -> List[Tensor]:
    """kv_heads > 0: grouped-query attention, key and value projections have kv_heads * (d / heads) rows."""
    kv_rows = d if kv_heads <= 0 else kv_heads * (d // heads)
    t: List[Tensor] = [Tensor("embed_tokens", ROLE_EMBED, vocab, d)]
    for i in range(n_layer):
        p = f"layers.{i}."
        t += [
            Tensor(p + "input_layernorm.weight", ROLE_VECTOR, 1, d, init="ones"),
            Tensor(p + "self_attn.q_proj", ROLE_Q, d, d, heads=heads),
            Tensor(p + "self_attn.k_proj", ROLE_K, kv_rows, d, heads=heads if kv_heads <= 0 else kv_heads),
            Tensor(p + "self_attn.v_proj", ROLE_V, kv_rows, d),
            Tensor(p + "self_attn.o_proj", ROLE_ATTN_OUT, d, d),
            Tensor(p + "post_attention_layernorm.weight", ROLE_VECTOR, 1, d, init="ones"),
            Tensor(p + "mlp.gate_proj", ROLE_MLP, ffn, d),
            Tensor(p + "mlp.up_proj", ROLE_MLP, ffn, d),
            Tensor(p + "mlp.down_proj", ROLE_MLP, d, ffn),
        ]
    t += [
        Tensor("norm.weight", ROLE_VECTOR, 1, d, init="ones"),
        Tensor("lm_head", ROLE_LM_HEAD, vocab, d),
    ]
    return t


WORKLOAD_NAMES = ("tiny", "llama60m", "gpt2_124m", "llama350m", "gpt2_1p5b")
EXTRA_WORKLOAD_NAMES = ("llama3_8b",)      # Section 5.2's fine-tuning model, shapes only


def get_workload(name: str, rank_override: int = 0, rank_pct: int = 5) -> Workload:
    """Return one of the five parameter sets.

    tiny       2-layer GPT-2 style, d=256, 4 heads, FFN 1024, vocab 4096, ctx 2048; fp32 grads.
    llama60m   8 layers, d=512, 8 heads, SwiGLU 1376, vocab 32000; bf16 grads with per-row scales.
    gpt2_124m  12 layers, d=768, 12 heads, FFN 3072, vocab 50257, ctx 1024; bf16 Student-t grads.
    llama350m  24 layers, d=1024, 16 heads, SwiGLU 2736, vocab 32000; bf16 grads, 5% heavy rows.
    gpt2_1p5b  48 layers, d=1600, 25 heads, FFN 6400, vocab 50257, ctx 1024; bf16 Gaussian grads.
    llama3_8b  32 layers, d=4096, 32 heads (8 key/value heads), SwiGLU 14336, vocab 128256, untied head; bf16
               Gaussian grads.  The shapes of the model fine-tuned in Section 5.2; rank 5% of 4096 = 204.
    "gpt2_1p5b@L" / "llama3_8b@L": the same shapes with L layers.  rank_pct: percent of the full rank (Section
    5.1.2 sweeps 2, 5, 10 and 50).
    """
    layers = None
    if "@" in name:                  # "gpt2_1p5b@4": the same shapes with 4 layers (small profiling captures)
        name, _, n_l = name.partition("@")
        layers = int(n_l)
    if layers is not None:
        if name == "gpt2_1p5b":
            w = Workload(f"{name}@{layers}", _gpt2(layers, 1600, 25, 6400, 50257, 1024), "bf16", "normal", steps=20)
        elif name == "llama3_8b":
            w = Workload(f"{name}@{layers}", _llama(layers, 4096, 32, 14336, 128256, kv_heads=8), "bf16", "normal",
                         steps=20)
        else:
            raise KeyError("a layer count can only be given for gpt2_1p5b and llama3_8b")
        w.rank_override = int(rank_override)
        w.rank_pct = int(rank_pct)
        return w
    if name == "tiny":
        w = Workload(name, _gpt2(2, 256, 4, 1024, 4096, 2048), "f32", "normal", steps=10,
                     beta2=0.999)
    elif name == "llama60m":
        w = Workload(name, _llama(8, 512, 8, 1376, 32000), "bf16", "rowscale", steps=20)
    elif name == "gpt2_124m":
        w = Workload(name, _gpt2(12, 768, 12, 3072, 50257, 1024), "bf16", "student_t3", steps=20)
    elif name == "llama350m":
        w = Workload(name, _llama(24, 1024, 16, 2736, 32000), "bf16", "heavyrows", steps=20)
    elif name == "gpt2_1p5b":
        w = Workload(name, _gpt2(48, 1600, 25, 6400, 50257, 1024), "bf16", "normal", steps=20)
    elif name == "llama3_8b":
        w = Workload(name, _llama(32, 4096, 32, 14336, 128256, kv_heads=8), "bf16", "normal", steps=20)
    else:
        raise KeyError(f"unknown workload {name!r}; choose from {WORKLOAD_NAMES}")
    w.rank_override = int(rank_override)
    w.rank_pct = int(rank_pct)
    return w
