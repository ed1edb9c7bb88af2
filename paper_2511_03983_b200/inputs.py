"""Seeded synthetic inputs and workload presets for the TwIST training-round hot path.

This module holds NO arithmetic of the method: only the shapes of the five
workloads and seeded draws of weights, activations and targets.  It is the one
module that both the CPU oracle's tests and the CUDA path's tests/bench use, so
that both sides see identical bytes.

Value distributions (the synthetic stand-in for tokens of a language-model
corpus pushed through a pretrained transformer, which the paper's experiments
use): weights ~ N(0, 0.02^2) (std 0.02, the GPT-2 convention), activations and
regression targets ~ N(0, 1).  bf16 workloads round every draw to bf16
(round-to-nearest-even) at generation time, so the stored bytes are exact in
both bf16 and wider formats.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, Tuple

import numpy as np

FFN_RELU, FFN_GELU, FFN_SWIGLU = 0, 1, 2
DTYPE_FP32, DTYPE_BF16 = 0, 1
MODE_COVER, MODE_IID = 0, 1
KIND_FFN, KIND_HEAD = 0, 1


@dataclass(frozen=True)
class Workload:
    """Shape of one workload (names follow the paper: S subnets, N_sub kept blocks)."""
    name: str
    n_layers: int
    d_model: int
    n_heads: int          # H (0: the workload has no attention projections)
    n_kv_heads: int       # H_kv (== n_heads for plain multi-head attention)
    d_head: int
    d_ff: int             # F = d_inner
    ffn_kind: int
    n_subnets: int        # S
    ffn_keep: int         # N_sub for the FFN kind, in blocks
    head_keep: int        # N_sub for the head kind
    ffn_block: int        # neurons per FFN block (d_ff / R)
    tokens: int           # T: tokens per (subnet, local step)
    local_steps: int      # K: local steps per round (the repartition interval)
    rounds: int
    dtype: int
    sample_mode: int
    lr: float = 1e-2
    seed_w: int = 1000
    seed_x: int = 2000
    seed_mask: int = 3000
    common_ffn: Tuple[int, ...] = field(default_factory=tuple)
    common_heads: Tuple[int, ...] = field(default_factory=tuple)
    optimizer: str = "sgd"   # "sgd" (the workloads) or "adam" (the optimiser of the paper's experiments)
    beta1: float = 0.9
    beta2: float = 0.999
    adam_eps: float = 1e-8
    n_seqs: int = 1       # sequences per batch (tokens = n_seqs * sequence length); matters to the attention core only
    shared_layers: Tuple[int, ...] = field(default_factory=tuple)   # layers every worker holds whole (N_sub = N_full)
    layer_norm: bool = False   # chained composition only: the two layer normalisations of the pre-LN layer
    ln_eps: float = 1e-5

    @property
    def n_ffn_blocks(self) -> int:
        return self.d_ff // self.ffn_block

    @property
    def f_sub(self) -> int:           # f' kept neurons per subnet
        return self.ffn_keep * self.ffn_block

    @property
    def a_sub(self) -> int:           # a' = H' * d_head
        return self.head_keep * self.d_head

    @property
    def nmat(self) -> int:
        return 3 if self.ffn_kind == FFN_SWIGLU else 2

    @property
    def tokens_per_round(self) -> int:
        return self.n_subnets * self.local_steps * self.tokens


def _w(name, **kw) -> Workload:
    return Workload(name=name, **kw)


# The five workloads (1-based numbering; index 0 is unused so PRESETS[i] is "config i").
PRESETS: Dict[int, Workload] = {
    1: _w("cfg1-tiny-relu-ffn-fp32", n_layers=1, d_model=64, n_heads=0, n_kv_heads=0, d_head=0, d_ff=256,
          ffn_kind=FFN_RELU, n_subnets=2, ffn_keep=128, head_keep=0, ffn_block=1, tokens=128, local_steps=1,
          rounds=1, dtype=DTYPE_FP32, sample_mode=MODE_COVER, seed_w=1001, seed_x=2001, seed_mask=3001),
    2: _w("cfg2-gpt2-small-gelu-bf16", n_layers=12, d_model=768, n_heads=12, n_kv_heads=12, d_head=64, d_ff=3072,
          ffn_kind=FFN_GELU, n_subnets=4, ffn_keep=1536, head_keep=6, ffn_block=1, tokens=8 * 1024, local_steps=4,
          n_seqs=8, rounds=10, dtype=DTYPE_BF16, sample_mode=MODE_COVER, seed_w=1002, seed_x=2002, seed_mask=3002),
    3: _w("cfg3-tinyllama-swiglu-gqa-bf16", n_layers=22, d_model=2048, n_heads=32, n_kv_heads=4, d_head=64,
          d_ff=5632, ffn_kind=FFN_SWIGLU, n_subnets=4, ffn_keep=2816, head_keep=16, ffn_block=1,
          tokens=16 * 2048, local_steps=8, n_seqs=16, rounds=5, dtype=DTYPE_BF16, sample_mode=MODE_COVER,
          seed_w=1003, seed_x=2003, seed_mask=3003),
    4: _w("cfg4-llama7b-swiglu-bf16", n_layers=32, d_model=4096, n_heads=32, n_kv_heads=32, d_head=128,
          d_ff=11008, ffn_kind=FFN_SWIGLU, n_subnets=8, ffn_keep=2752, head_keep=8, ffn_block=1,
          tokens=8 * 4096, local_steps=4, n_seqs=8, rounds=3, dtype=DTYPE_BF16, sample_mode=MODE_COVER,
          seed_w=1004, seed_x=2004, seed_mask=3004),
    # config 5 is a sweep over (S, keep); this entry is its S=8, keep=0.25 cell, see sweep_cfg5().
    5: _w("cfg5-7b-ffn-gather-aggregate-sweep", n_layers=32, d_model=4096, n_heads=0, n_kv_heads=0, d_head=0,
          d_ff=11008, ffn_kind=FFN_SWIGLU, n_subnets=8, ffn_keep=2752, head_keep=0, ffn_block=1, tokens=1024,
          local_steps=1, rounds=1, dtype=DTYPE_BF16, sample_mode=MODE_IID, seed_w=1005, seed_x=2005,
          seed_mask=3005),
}


def sweep_cfg5():
    """All 12 cells of the gather/aggregate sweep: S in {2,4,8,16} x keep in {.25,.5,.75}."""
    base = PRESETS[5]
    cells = []
    for S in (2, 4, 8, 16):
        for keep in (0.25, 0.5, 0.75):
            n_sub = int(np.floor(keep * base.n_ffn_blocks))
            cells.append(replace(base, name=f"cfg5-S{S}-keep{keep}", n_subnets=S, ffn_keep=n_sub))
    return cells


def scaled_twin(w: Workload, *, d_model, d_ff, d_head, tokens, n_layers=1, local_steps=None, rounds=1) -> Workload:
    """A scaled-down twin of a workload: same structure (kind, S, keep ratios, head
    counts, GQA grouping), smaller dimensions, ragged dimensions kept ragged."""
    keep_ratio = w.ffn_keep / w.n_ffn_blocks
    return replace(w, name=w.name + "-twin", d_model=d_model, d_ff=d_ff, d_head=d_head, tokens=tokens,
                   n_layers=n_layers, ffn_keep=int(np.floor(keep_ratio * (d_ff // w.ffn_block))),
                   local_steps=w.local_steps if local_steps is None else local_steps, rounds=rounds)


# --------------------------------------------------------------------------------------
# bf16 storage helpers (pure format conversion, no method arithmetic)
# --------------------------------------------------------------------------------------

def bf16_bits_from_f32(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest-even); returns the 16-bit patterns (uint16)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def f32_from_bf16_bits(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal(seed: int, tag: int, shape, std: float, dtype: int) -> np.ndarray:
    """Seeded N(0, std^2) draw as float32 values; for bf16 workloads the values are
    already bf16-representable.  (seed, tag) selects an independent stream."""
    rng = np.random.Generator(np.random.Philox(key=[np.uint64(seed), np.uint64(tag)]))
    x = rng.standard_normal(size=shape, dtype=np.float32) * np.float32(std)
    if dtype == DTYPE_BF16:
        x = f32_from_bf16_bits(bf16_bits_from_f32(x))
    return x


# Stream tags.  Weights: (layer, matrix).  Activations: (batch kind, round, subnet, step).
MAT_GATE, MAT_UP, MAT_DOWN, MAT_QKV, MAT_O = 0, 1, 2, 3, 4
BATCH_X, BATCH_TGT_D, BATCH_TGT_QKV, BATCH_A = 0, 1, 2, 3


def weight(w: Workload, layer: int, mat: int) -> np.ndarray:
    """Full-model matrix `mat` of `layer`, stored row = one neuron / one head-dim,
    d_model contiguous: gate, up, down [F, d]; qkv [(H + 2 H_kv) d_head, d]; o [H d_head, d]."""
    rows = {MAT_GATE: w.d_ff, MAT_UP: w.d_ff, MAT_DOWN: w.d_ff,
            MAT_QKV: (w.n_heads + 2 * w.n_kv_heads) * w.d_head, MAT_O: w.n_heads * w.d_head}[mat]
    return normal(w.seed_w, layer * 8 + mat, (rows, w.d_model), 0.02, w.dtype)


LN_PARAMS = ("ln_a_g", "ln_a_b", "ln_f_g", "ln_f_b")     # gain / bias of the attention and the FFN normalisation


def ln_param(w: Workload, layer: int, name: str, spread: float = 0.1) -> np.ndarray:
    """Layer-normalisation parameter [d_model] (float32).  The customary initial values are gain 1 and bias 0;
    `spread` adds a seeded N(0, spread^2) perturbation so that tests can tell the parameters apart (0: exact
    initial values)."""
    base = np.float32(1.0 if name.endswith("_g") else 0.0)
    if spread == 0:
        return np.full(w.d_model, base, dtype=np.float32)
    return base + normal(w.seed_w, layer * 8 + 5 + 65536 * (1 + LN_PARAMS.index(name)), (w.d_model,), spread, DTYPE_FP32)


def batch(w: Workload, kind: int, rnd: int, subnet: int, step: int, width: int, tokens: int | None = None):
    """One [T, width] batch of N(0,1) activations or targets for (round, subnet, local step)."""
    T = w.tokens if tokens is None else tokens
    tag = ((kind * 1024 + rnd) * 64 + subnet) * 1024 + step
    return normal(w.seed_x, tag, (T, width), 1.0, w.dtype)
