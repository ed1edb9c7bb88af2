"""Sequencing of one TwIST round on one GPU.

This module only allocates device buffers (torch) and calls the C ABI in order:
sample masks -> per layer { gather -> K local steps (forward, MSE, backward with fused
SGD) for the FFN block, the QKV projection and the output projection -> aggregate }.
Every arithmetic step runs in the CUDA library; nothing here computes on tensors.

Layers are streamed (BLOCKWISE, RoundEngine): slices, masters and activations exist for one
layer at a time, which is what lets the 7B-shaped workloads fit (per layer ~2.4 GB of slices
+ masters at S=8, keep 25%, instead of 78 GB for all 32 layers).  StackEngine chains the
layers (attention core, skip connections, optionally the two layer normalisations).

A layer is either partitioned (N_sub = the workload's keep counts) or shared (N_sub = N_full
in both kinds: every worker holds the whole layer and the aggregate is the plain mean); the two
kinds have different slice sizes, so the engine keeps one set of buffers per kind ("geometry")
and binds the set of the layer it is working on.
"""
from __future__ import annotations

import math
from contextlib import contextmanager
from functools import partial
from typing import Dict, List, Optional, Tuple

import torch

from . import binding as B
from .inputs import DTYPE_BF16, FFN_SWIGLU, LN_PARAMS, Workload


def _tdtype(w: Workload):
    return torch.bfloat16 if w.dtype == DTYPE_BF16 else torch.float32


class Geometry:
    """Slice sizes and output scales of a layer whose subnets keep `ffn_keep` FFN blocks and `head_keep` heads."""

    def __init__(self, w: Workload, ffn_keep: int, head_keep: int):
        self.ffn_keep, self.head_keep = ffn_keep, head_keep
        self.f_sub = ffn_keep * w.ffn_block
        self.g = 2 if w.ffn_kind == FFN_SWIGLU else 1
        self.gf = self.g * self.f_sub
        self.alpha_f = math.sqrt(w.n_ffn_blocks / ffn_keep)            # activation-shift scale, Sec. 3.4
        self.kv_max = self.a_sub = self.nq = 0
        self.alpha_a = 1.0
        if w.n_heads > 0:
            self.kv_max = min(w.n_kv_heads, head_keep)
            self.a_sub = head_keep * w.d_head
            self.nq = self.a_sub + 2 * self.kv_max * w.d_head
            self.alpha_a = math.sqrt(w.n_heads / head_keep)


_SLICES = ("w_gu", "w_down", "w_qkv", "w_o")


class RoundEngine:
    BLOCKS = ("ffn", "qkv", "o")

    def __init__(self, w: Workload, device: str = "cuda", keep_f32_full: bool = False, compute_dx: bool = True,
                 dump_grads: bool = False, fuse_loss: bool = True, store_outputs: bool = True,
                 lazy_master: bool = True):
        """fuse_loss: evaluate the loss inside the forward call's output kernel (otherwise with the
        stand-alone twist_mse_fwd_bwd).  store_outputs=False (fused loss, bf16 only) skips storing the
        block outputs, which nothing reads once the loss gradient exists.  lazy_master (bf16): the gather
        writes only the bf16 slices; the fp32 masters come into being in the first weight update of the round,
        which reads the bf16 slice (exactly the master's value) instead."""
        self.w, self.dev = w, torch.device(device)
        self.compute_dx, self.dump_grads = compute_dx, dump_grads or w.dtype != DTYPE_BF16
        self.fuse_loss = fuse_loss
        self.store_outputs = store_outputs or not fuse_loss or w.dtype != DTYPE_BF16
        td, dev = _tdtype(w), self.dev
        S, T, d = w.n_subnets, w.tokens, w.d_model
        self.g = 2 if w.ffn_kind == FFN_SWIGLU else 1
        L, F = w.n_layers, w.d_ff
        self.has_attn = w.n_heads > 0
        bf16 = w.dtype == DTYPE_BF16
        # full model (the central model of the paper's server)
        # gate rows then up rows of a layer lie back to back ([L][g F][d]), so that a full-width layer is itself a
        # valid w_gu operand (Masked / Hybrid TwIST, evaluation of the full model); the dictionary holds views
        self.full_gu = torch.empty(L, self.g * F, d, dtype=td, device=dev)
        self.full: Dict[str, torch.Tensor] = {"up": self.full_gu[:, (self.g - 1) * F:],
                                              "down": torch.empty(L, F, d, dtype=td, device=dev)}
        if self.g == 2:
            self.full["gate"] = self.full_gu[:, :F]
        if self.has_attn:
            H, Hkv, dh = w.n_heads, w.n_kv_heads, w.d_head
            self.full["qkv"] = torch.empty(L, (H + 2 * Hkv) * dh, d, dtype=td, device=dev)
            self.full["o"] = torch.empty(L, H * dh, d, dtype=td, device=dev)
        self.full_f32, self.full_gu_f32 = None, None
        if keep_f32_full and bf16:
            self.full_gu_f32 = torch.empty(L, self.g * F, d, dtype=torch.float32, device=dev)
            self.full_f32 = {m: (self.full_gu_f32[:, (self.g - 1) * F:] if m == "up" else
                                 self.full_gu_f32[:, :F] if m == "gate" else
                                 torch.empty(v.shape, dtype=torch.float32, device=dev)) for m, v in self.full.items()}
        # aggregator index data (the same shape for every layer), all layers
        nb = w.n_ffn_blocks
        i32 = dict(dtype=torch.int32, device=dev)
        self.cover_ffn = torch.empty(L, nb, **i32)
        self.pos_ffn = torch.empty(L, S, nb, **i32)
        if self.has_attn:
            self.cover_head = torch.empty(L, w.n_heads, **i32)
            self.pos_head = torch.empty(L, S, w.n_heads, **i32)
            self.kv_idx = torch.empty(L, S, w.n_kv_heads, **i32)
            self.kv_count = torch.empty(L, S, **i32)
            self.kv_cols = torch.empty(L, S, **i32)
            self.kv_cover = torch.empty(L, w.n_kv_heads, **i32)
            self.kv_pos = torch.empty(L, S, w.n_kv_heads, **i32)
        self.adam = w.optimizer == "adam"
        assert not self.adam or bf16, "the fused Adam update exists for the bf16 dtype"
        self.lazy_master = lazy_master and bf16 and w.local_steps > 0
        # geometries: partitioned layers, and shared layers (N_sub = N_full) if the workload has any
        self.shared_layers = frozenset(w.shared_layers)
        assert all(0 <= l < L for l in self.shared_layers)
        self.geo: Dict[str, Geometry] = {"part": Geometry(w, w.ffn_keep, w.head_keep)}
        if self.shared_layers:
            self.geo["shared"] = Geometry(w, w.n_ffn_blocks, w.n_heads)
        self.bufs: Dict[str, Dict[str, object]] = {}
        self.batches: Dict[str, Dict[str, List[torch.Tensor]]] = {k: {"Tq": [], "A": []} for k in self.geo}
        # activations of one (layer, step) whose size does not depend on the geometry
        act = lambda width: torch.empty(S, T, width, dtype=td, device=dev)
        self.y, self.dy = act(d), act(d)
        self.dx = act(d) if compute_dx else None
        self.loss = torch.zeros(L, 3, max(1, w.local_steps), S, dtype=torch.float32, device=dev)
        # the plan: shapes of the workload and the cache of encoded tensor maps; every GEMM / attention call carries it
        self.plan = B.Plan(w)
        self._ffn_args = partial(B.ffn_args, plan=self.plan)
        self._proj_args = partial(B.proj_args, plan=self.plan)
        self._attn_core_args = partial(B.attn_core_args, plan=self.plan)
        self.ws = torch.empty(self.plan.workspace_bytes(), dtype=torch.uint8, device=dev)     # scratch of the loss calls
        # batches: lists over the local step k of [S][T][width] tensors (Tq and A: per geometry, see the properties)
        self.X: List[torch.Tensor] = []
        self.Td: List[torch.Tensor] = []
        self.launches = 0
        # what the gather reads as blueprint, what the aggregate reads as ranks, and the activation mask of the FFN
        # calls: the sampler's outputs and none, unless a subclass (Masked TwIST) substitutes its own
        self._gather_idx_override, self._agg_pos_override, self.h_mask = None, None, None
        # optional per-phase CUDA-event timing (events on the launching stream)
        self.timing = False
        self.events: Dict[str, List[Tuple[torch.cuda.Event, torch.cuda.Event]]] = {}
        self._cur = None
        self._use_kind("part")

    # ------------------------------------------------------------------ geometries
    def _alloc(self, kind: str) -> Dict[str, object]:
        """Buffers of one geometry: blueprints, slices (+ fp32 masters and Adam moments in bf16 mode), the
        activations and gradient dumps whose width depends on the kept sizes."""
        w, gm, dev, td = self.w, self.geo[kind], self.dev, _tdtype(self.w)
        S, T, d, L = w.n_subnets, w.tokens, w.d_model, w.n_layers
        bf16 = w.dtype == DTYPE_BF16
        i32 = dict(dtype=torch.int32, device=dev)
        b: Dict[str, object] = {"idx_ffn": torch.empty(L, S, gm.ffn_keep, **i32)}
        if self.has_attn:
            b["idx_head"] = torch.empty(L, S, gm.head_keep, **i32)
        rows = {"w_gu": gm.gf, "w_down": gm.f_sub, "w_qkv": gm.nq, "w_o": gm.a_sub}
        names = _SLICES if self.has_attn else _SLICES[:2]
        moments = []
        for n in names:
            b[n] = torch.empty(S, rows[n], d, dtype=td, device=dev)
            b[n + "_m"] = torch.empty(S, rows[n], d, dtype=torch.float32, device=dev) if bf16 else None
            if self.adam:      # Adam moments live with the worker's copy of the slice: zeroed at every gather
                for tag in ("_m1", "_m2"):
                    b[n + tag] = torch.zeros_like(b[n + "_m"])
                    moments.append(n + tag)
            b["d" + n] = torch.empty(S, rows[n], d, dtype=torch.float32, device=dev) if self.dump_grads else None
        b["moment_names"] = moments
        act = lambda width: torch.empty(S, T, width, dtype=td, device=dev)
        b["pre"], b["dpre"], b["hh"] = act(gm.gf), act(gm.gf), act(gm.f_sub)
        if self.has_attn:
            b["qkv_out"], b["dqkv"] = act(gm.nq), act(gm.nq)
            b["da"] = act(gm.a_sub) if self.compute_dx else None
        return b

    def _use_kind(self, kind: str):
        if kind == self._cur:
            return
        if kind not in self.bufs:
            self.bufs[kind] = self._alloc(kind)
        gm = self.geo[kind]
        for n in ("f_sub", "gf", "a_sub", "nq", "kv_max", "alpha_f", "alpha_a", "ffn_keep", "head_keep"):
            setattr(self, n, getattr(gm, n))
        for n, t in self.bufs[kind].items():
            setattr(self, n, t)
        self._cur = kind

    def kind_of(self, l: int) -> str:
        return "shared" if l in self.shared_layers else "part"

    def _use(self, l: int):
        """Binds the sizes and buffers of layer l's geometry onto the engine."""
        self._use_kind(self.kind_of(l))

    @property
    def Tq(self) -> List[torch.Tensor]:      # targets of the QKV block (width nq) of the bound geometry
        return self.batches[self._cur]["Tq"]

    @Tq.setter
    def Tq(self, v):
        self.batches[self._cur]["Tq"] = v

    @property
    def A(self) -> List[torch.Tensor]:       # inputs of the output projection (width a') of the bound geometry
        return self.batches[self._cur]["A"]

    @A.setter
    def A(self, v):
        self.batches[self._cur]["A"] = v

    @property
    def gather_idx_ffn(self):
        return self.idx_ffn if self._gather_idx_override is None else self._gather_idx_override

    @property
    def agg_pos_ffn(self):
        return self.pos_ffn if self._agg_pos_override is None else self._agg_pos_override

    @contextmanager
    def _timed(self, name: str):
        if not self.timing:
            yield
            return
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        yield
        b.record()
        self.events.setdefault(name, []).append((a, b))

    def phase_ms(self) -> Dict[str, Tuple[float, int]]:
        """Total milliseconds and number of timed calls per phase (call after a synchronize)."""
        return {k: (sum(a.elapsed_time(b) for a, b in v), len(v)) for k, v in self.events.items()}

    # ------------------------------------------------------------------ steps of the round
    def _layer_runs(self):
        """Maximal runs of consecutive layers of the same kind: (first layer, count, kind)."""
        runs, l, L = [], 0, self.w.n_layers
        while l < L:
            k, n = self.kind_of(l), 1
            while l + n < L and self.kind_of(l + n) == k:
                n += 1
            runs.append((l, n, k))
            l += n
        return runs

    def sample_masks(self, rnd: int):
        w = self.w
        with self._timed("sample_masks"):
            for l0, n, kind in self._layer_runs():
                self._use_kind(kind)
                sl = slice(l0, l0 + n)
                B.twist_sample_masks(w.seed_mask, rnd, l0, n, B.KIND_FFN, w.n_ffn_blocks, w.n_subnets, self.ffn_keep,
                                     list(w.common_ffn), w.sample_mode, self.idx_ffn[sl], self.cover_ffn[sl],
                                     self.pos_ffn[sl])
                self.launches += 2
                if self.has_attn:
                    B.twist_sample_masks(w.seed_mask, rnd, l0, n, B.KIND_HEAD, w.n_heads, w.n_subnets, self.head_keep,
                                         list(w.common_heads), w.sample_mode, self.idx_head[sl], self.cover_head[sl],
                                         self.pos_head[sl])
                    B.twist_kv_groups(self.idx_head[sl], n, w.n_subnets, self.head_keep, w.n_heads, w.n_kv_heads,
                                      w.d_head, self.kv_idx[sl], self.kv_count[sl], self.kv_cols[sl], self.kv_cover[sl],
                                      self.kv_pos[sl])
                    self.launches += 4

    def _gather_master(self, master):
        """Destination of the gather's fp32 copy: none when the first weight update creates the masters."""
        return None if self.lazy_master else master

    def _first(self, k: int) -> dict:
        """Argument of a backward call: the first update after a gather reads the bf16 slice in place of the master."""
        return dict(master_from_slice=True) if (self.lazy_master and k == 0) else {}

    def gather_layer(self, l: int, which=("ffn", "attn")):
        self._use(l)
        w, d = self.w, self.w.d_model
        f, gf, keep = self.f_sub, self.gf, self.ffn_keep
        nb = w.n_ffn_blocks
        gm = self._gather_master
        segs = []
        if "ffn" in which:
            if self.g == 2:
                segs.append(B.gather_segment(self.full["gate"][l], self.w_gu, gm(self.w_gu_m), self.gather_idx_ffn[l], None,
                                             keep, keep, w.ffn_block, 0, gf * d, 0, nb))
            segs.append(B.gather_segment(self.full["up"][l], self.w_gu, gm(self.w_gu_m), self.gather_idx_ffn[l], None,
                                         keep, keep, w.ffn_block, 0, gf * d, f if self.g == 2 else 0, nb))
            segs.append(B.gather_segment(self.full["down"][l], self.w_down, gm(self.w_down_m), self.gather_idx_ffn[l], None,
                                         keep, keep, w.ffn_block, 0, f * d, 0, nb))
        if self.has_attn and "attn" in which:
            H, Hkv, dh, hk = w.n_heads, w.n_kv_heads, w.d_head, self.head_keep
            qkv = self.full["qkv"][l]
            segs.append(B.gather_segment(qkv, self.w_qkv, gm(self.w_qkv_m), self.idx_head[l], None, hk, hk, dh, 0,
                                         self.nq * d, 0, H))
            segs.append(B.gather_segment(qkv, self.w_qkv, gm(self.w_qkv_m), self.kv_idx[l], self.kv_count[l], Hkv,
                                         self.kv_max, dh, H * dh, self.nq * d, self.a_sub, Hkv))
            segs.append(B.gather_segment(qkv, self.w_qkv, gm(self.w_qkv_m), self.kv_idx[l], self.kv_count[l], Hkv,
                                         self.kv_max, dh, (H + Hkv) * dh, self.nq * d, self.a_sub + self.kv_max * dh,
                                         Hkv))
            segs.append(B.gather_segment(self.full["o"][l], self.w_o, gm(self.w_o_m), self.idx_head[l], None, hk, hk, dh, 0,
                                         self.a_sub * d, 0, H))
        with self._timed("gather"):
            B.twist_gather_subnets(segs, w.n_subnets, d, w.dtype)
            for n in self.moment_names:        # a fresh worker state: first and second moments start at zero
                getattr(self, n).zero_()
        self.launches += 1

    def _aggregate_segments(self, l: int, which, dst, f32, central=lambda m: None):
        """The aggregate's row ranges of layer l.  dst(m) / f32(m): destination of matrix m in the workload's dtype and
        its fp32 companion (or None); central(m): a source in full-matrix geometry (or None)."""
        w, d = self.w, self.w.d_model
        f, gf, keep = self.f_sub, self.gf, self.ffn_keep
        bf16 = w.dtype == DTYPE_BF16
        sub = lambda lo, master: master if bf16 else lo
        nb = w.n_ffn_blocks
        segs = []
        if "ffn" in which:
            if self.g == 2:
                segs.append(B.aggregate_segment(dst("gate"), f32("gate"), sub(self.w_gu, self.w_gu_m),
                                                self.cover_ffn[l], self.agg_pos_ffn[l], nb, w.ffn_block, 0, gf * d, 0,
                                                keep, central=central("gate")))
            segs.append(B.aggregate_segment(dst("up"), f32("up"), sub(self.w_gu, self.w_gu_m),
                                            self.cover_ffn[l], self.agg_pos_ffn[l], nb, w.ffn_block, 0, gf * d,
                                            f if self.g == 2 else 0, keep, central=central("up")))
            segs.append(B.aggregate_segment(dst("down"), f32("down"), sub(self.w_down, self.w_down_m),
                                            self.cover_ffn[l], self.agg_pos_ffn[l], nb, w.ffn_block, 0, f * d, 0,
                                            keep, central=central("down")))
        if self.has_attn and "attn" in which:
            H, Hkv, dh = w.n_heads, w.n_kv_heads, w.d_head
            q_sub = sub(self.w_qkv, self.w_qkv_m)
            cq = central("qkv")
            segs.append(B.aggregate_segment(dst("qkv"), f32("qkv"), q_sub, self.cover_head[l],
                                            self.pos_head[l], H, dh, 0, self.nq * d, 0, self.head_keep, central=cq))
            segs.append(B.aggregate_segment(dst("qkv"), f32("qkv"), q_sub, self.kv_cover[l], self.kv_pos[l],
                                            Hkv, dh, H * dh, self.nq * d, self.a_sub, self.kv_max, central=cq))
            segs.append(B.aggregate_segment(dst("qkv"), f32("qkv"), q_sub, self.kv_cover[l], self.kv_pos[l],
                                            Hkv, dh, (H + Hkv) * dh, self.nq * d, self.a_sub + self.kv_max * dh,
                                            self.kv_max, central=cq))
            segs.append(B.aggregate_segment(dst("o"), f32("o"), sub(self.w_o, self.w_o_m), self.cover_head[l],
                                            self.pos_head[l], H, dh, 0, self.a_sub * d, 0, self.head_keep,
                                            central=central("o")))
        return segs

    def aggregate_layer(self, l: int, live: int = 0xFFFFFFFF, which=("ffn", "attn")):
        self._use(l)
        w = self.w
        f32 = (lambda m: self.full_f32[m][l]) if self.full_f32 is not None else (lambda m: None)
        segs = self._aggregate_segments(l, which, lambda m: self.full[m][l], f32)
        with self._timed("aggregate"):
            B.twist_aggregate(segs, w.n_subnets, w.d_model, w.dtype, live)
        self.launches += 1

    def _opt(self, k: int, *names):
        """Optimiser arguments of local step k (0-based) for the slices `names`: (opt, moments...) keyword args."""
        if not self.adam:
            return {}
        w = self.w
        kw = {"opt": B.adam(k + 1, w.beta1, w.beta2, w.adam_eps)}
        for arg, n in names:
            kw["m" + arg] = getattr(self, n + "_m1")
            kw["v" + arg] = getattr(self, n + "_m2")
        return kw

    def _mse(self, y, tgt, dy, loss, width, valid_cols=None, seg_begin=0, seg_width=0):
        w = self.w
        with self._timed("mse"):
            B.twist_mse_fwd_bwd(y, tgt, dy, loss, w.n_subnets, w.tokens, width, valid_cols, seg_begin, seg_width,
                                w.dtype, self.ws)
        self.launches += 2

    def ffn_step(self, l: int, k: int, lr: Optional[float] = None):
        self._use(l)
        w = self.w
        lr = w.lr if lr is None else lr
        fused = dict(tgt=self.Td[k], loss=self.loss[l, 0, k], loss_ws=self.ws) if self.fuse_loss else {}
        a = self._ffn_args(w.ffn_kind, w.dtype, w.n_subnets, w.tokens, w.d_model, self.f_sub, self.alpha_f, lr,
                       x=self.X[k], w_gu=self.w_gu, w_down=self.w_down, w_gu_master=self.w_gu_m,
                       w_down_master=self.w_down_m, pre=self.pre, hh=self.hh,
                       y=self.y if self.store_outputs else None, dy=self.dy, dpre=self.dpre,
                       dx=self.dx, dw_gu=self.dw_gu, dw_down=self.dw_down, hidden_mask=self.h_mask, **fused,
                       **self._first(k), **self._opt(k, ("_gu", "w_gu"), ("_down", "w_down")))
        with self._timed("ffn_fwd"):
            B.twist_subnet_ffn_fwd(a)
        if self.fuse_loss:
            self.launches += 0 if w.dtype == DTYPE_BF16 else 2      # bf16: the loss is finished inside the output GEMM
        else:
            self._mse(self.y, self.Td[k], self.dy, self.loss[l, 0, k], w.d_model)
        with self._timed("ffn_bwd"):
            B.twist_subnet_ffn_bwd(a)
        bf16 = w.dtype == DTYPE_BF16
        self.launches += (2 + 3 + (1 if self.compute_dx else 0)) if bf16 else (3 + 4 + (1 if self.compute_dx else 0) + 2)

    def _qkv_loss_mask(self, l: int) -> dict:
        """Which columns of the QKV block's output count in its loss: all, or (grouped-query attention) the K / V
        groups each subnet holds."""
        w = self.w
        if w.n_kv_heads == w.n_heads:
            return {}
        return dict(valid_cols=self.kv_cols[l], seg_begin=self.a_sub, seg_width=self.kv_max * w.d_head)

    def _o_mask(self, l: int) -> dict:
        return {}

    def qkv_step(self, l: int, k: int, lr: Optional[float] = None):
        self._use(l)
        w = self.w
        lr = w.lr if lr is None else lr
        mask = self._qkv_loss_mask(l)
        ragged = bool(mask)
        fused = dict(tgt=self.Tq[k], loss=self.loss[l, 1, k], loss_ws=self.ws, **mask) if self.fuse_loss else {}
        a = self._proj_args(B.PROJ_QKV, w.dtype, w.n_subnets, w.tokens, w.d_model, self.nq, 1.0, lr, in_=self.X[k],
                        w=self.w_qkv, w_master=self.w_qkv_m, out=self.qkv_out if self.store_outputs else None,
                        d_out=self.dqkv, d_in=self.dx, dw=self.dw_qkv, **fused, **self._first(k),
                        **self._opt(k, ("", "w_qkv")))
        with self._timed("qkv_fwd"):
            B.twist_subnet_attn_proj_fwd(a)
        if self.fuse_loss:
            self.launches += 0 if w.dtype == DTYPE_BF16 else 2      # bf16: the loss is finished inside the output GEMM
        else:
            self._mse(self.qkv_out, self.Tq[k], self.dqkv, self.loss[l, 1, k], self.nq,
                      self.kv_cols[l] if ragged else None, self.a_sub, self.kv_max * w.d_head)
        with self._timed("qkv_bwd"):
            B.twist_subnet_attn_proj_bwd(a)
        self.launches += 1 + 1 + (1 if self.compute_dx else 0) + (0 if w.dtype == DTYPE_BF16 else 1)

    def o_step(self, l: int, k: int, lr: Optional[float] = None):
        self._use(l)
        w = self.w
        lr = w.lr if lr is None else lr
        fused = dict(tgt=self.Td[k], loss=self.loss[l, 2, k], loss_ws=self.ws) if self.fuse_loss else {}
        a = self._proj_args(B.PROJ_O, w.dtype, w.n_subnets, w.tokens, w.d_model, self.a_sub, self.alpha_a, lr,
                        in_=self.A[k], w=self.w_o, w_master=self.w_o_m, out=self.y if self.store_outputs else None,
                        d_out=self.dy, d_in=self.da, dw=self.dw_o, **fused, **self._o_mask(l), **self._first(k),
                        **self._opt(k, ("", "w_o")))
        with self._timed("o_fwd"):
            B.twist_subnet_attn_proj_fwd(a)
        if self.fuse_loss:
            self.launches += 0 if w.dtype == DTYPE_BF16 else 2      # bf16: the loss is finished inside the output GEMM
        else:
            self._mse(self.y, self.Td[k], self.dy, self.loss[l, 2, k], w.d_model)
        with self._timed("o_bwd"):
            B.twist_subnet_attn_proj_bwd(a)
        self.launches += 1 + 1 + (1 if self.compute_dx else 0) + (0 if w.dtype == DTYPE_BF16 else 1)

    # ------------------------------------------------------------------ deployment / evaluation (Sec. 4.2)
    def export_subnet(self, s: int) -> Dict[str, torch.Tensor]:
        """The dense smaller model of subnet s for the layer gathered last (Sec. 4.2, Deployment: the pruned model
        mirrors the subnet generation of training): copies of its slices, w_gu = gate rows then up rows."""
        out = {"w_gu": self.w_gu[s].clone(), "w_down": self.w_down[s].clone()}
        if self.has_attn:
            out.update(w_qkv=self.w_qkv[s].clone(), w_o=self.w_o[s].clone())
        return out

    def evaluate_subnets(self, l: int, k: int) -> torch.Tensor:
        """Evaluation mode for subnets (Sec. 4.2): forward only, on the slices gathered for layer l, with the
        subnet's own scale (an engine built with other keep counts than the training run evaluates a mismatched
        subnet ratio).  Returns the losses [blocks][S] (device); the caller averages over the workers."""
        self._use(l)
        w = self.w
        assert self.fuse_loss, "evaluation uses the loss fused into the forward kernels"
        a = self._ffn_args(w.ffn_kind, w.dtype, w.n_subnets, w.tokens, w.d_model, self.f_sub, self.alpha_f, 0.0, x=self.X[k],
                       w_gu=self.w_gu, w_down=self.w_down, pre=self.pre, hh=self.hh,
                       y=self.y if self.store_outputs else None, dy=self.dy, tgt=self.Td[k], loss=self.loss[l, 0, k],
                       loss_ws=self.ws)
        B.twist_subnet_ffn_fwd(a)
        self.launches += 2
        if self.has_attn:
            ragged = w.n_kv_heads != w.n_heads
            mask = dict(valid_cols=self.kv_cols[l], seg_begin=self.a_sub, seg_width=self.kv_max * w.d_head) if ragged else {}
            q = self._proj_args(B.PROJ_QKV, w.dtype, w.n_subnets, w.tokens, w.d_model, self.nq, 1.0, 0.0, in_=self.X[k],
                            w=self.w_qkv, out=self.qkv_out if self.store_outputs else None, d_out=self.dqkv,
                            tgt=self.Tq[k], loss=self.loss[l, 1, k], loss_ws=self.ws, **mask)
            B.twist_subnet_attn_proj_fwd(q)
            o = self._proj_args(B.PROJ_O, w.dtype, w.n_subnets, w.tokens, w.d_model, self.a_sub, self.alpha_a, 0.0,
                            in_=self.A[k], w=self.w_o, out=self.y if self.store_outputs else None, d_out=self.dy,
                            tgt=self.Td[k], loss=self.loss[l, 2, k], loss_ws=self.ws)
            B.twist_subnet_attn_proj_fwd(o)
            self.launches += 2
        return self.loss[l, : 3 if self.has_attn else 1, k]

    def evaluate_full_ffn(self, l: int, k: int) -> torch.Tensor:
        """Evaluation mode for the full model (Sec. 4.2: assessed directly, no scaling, no masking), FFN block of
        layer l on every worker's batch k.  Returns the losses [S] (device)."""
        w = self.w
        assert w.dtype == DTYPE_BF16, "the full-width evaluation runs the bf16 kernels"
        T, d, F = w.tokens, w.d_model, w.d_ff
        if not hasattr(self, "e_pre"):
            bf = torch.bfloat16
            self.e_pre = torch.empty(1, T, self.g * F, dtype=bf, device=self.dev)
            self.e_hh = torch.empty(1, T, F, dtype=bf, device=self.dev)
            self.e_loss = torch.zeros(w.n_subnets, dtype=torch.float32, device=self.dev)
        for s in range(w.n_subnets):
            a = self._ffn_args(w.ffn_kind, w.dtype, 1, T, d, F, 1.0, 0.0, x=self.X[k][s:s + 1], w_gu=self.full_gu[l],
                           w_down=self.full["down"][l], pre=self.e_pre, hh=self.e_hh, y=None, dy=self.dy[s:s + 1],
                           tgt=self.Td[k][s:s + 1], loss=self.e_loss[s:s + 1], loss_ws=self.ws)
            B.twist_subnet_ffn_fwd(a)
            self.launches += 2
        return self.e_loss

    def run_layer(self, l: int):
        self.gather_layer(l)
        for k in range(self.w.local_steps):
            self.ffn_step(l, k)
            if self.has_attn:
                self.qkv_step(l, k)
                self.o_step(l, k)
        self.aggregate_layer(l)

    def run_round(self, rnd: int):
        """One full round: resample every layer's blueprints, then stream the layers."""
        self.sample_masks(rnd)
        for l in range(self.w.n_layers):
            self.run_layer(l)


class MaskedRoundEngine(RoundEngine):
    """Masked TwIST (Sec. 4.1): every worker holds a full-width copy of the layer and is turned into its subnet by
    masks; nothing is physically smaller.  FFN blocks: an activation mask (y = M * f(x)).  Attention blocks: a head
    mask -- the columns of the dropped heads stay out of the QKV block's loss, the dropped heads' outputs are zero
    at the output projection's input and no gradient flows into them.  The "gather" is a copy of the whole layer to
    every worker (the identity blueprint), the masks come from the sampled blueprints' cover bits, and the
    aggregator averages every block over the workers whose blueprint holds it.  In exact arithmetic the round
    equals RoundEngine's, at N_full / N_sub times its flops and S full copies of a layer: a simulation mode and an
    on-device check of "masked = gathered", not a fast path.
    Batches of the attention blocks are full-width: Tq [S][T][(H + 2 H_kv) d_head] (only the held columns are
    read) and A [S][T][H d_head] (the head mask is applied to it before the output projection)."""

    def __init__(self, w: Workload, device: str = "cuda", **kw):
        from dataclasses import replace as _replace
        assert w.dtype == DTYPE_BF16 and not w.shared_layers, "bf16 workloads without shared layers"
        nb, H, Hkv = w.n_ffn_blocks, w.n_heads, w.n_kv_heads
        super().__init__(_replace(w, ffn_keep=nb, head_keep=H), device=device, **kw)      # storage: full-width slices
        assert self.fuse_loss or not self.has_attn, "the head mask of the QKV block acts in the fused loss"
        self.true_w = w
        L, S = w.n_layers, w.n_subnets
        i32 = dict(dtype=torch.int32, device=self.dev)
        self.idx_ffn = torch.empty(L, S, w.ffn_keep, **i32)                   # the sampled blueprints
        self.bufs["part"]["idx_ffn"] = self.idx_ffn
        ident = torch.arange(nb, **i32).expand(L, S, nb).contiguous()
        self._gather_idx_override, self._agg_pos_override = ident, ident      # every worker copies / returns every block
        self.h_mask = torch.zeros(S, w.d_ff, dtype=torch.uint8, device=self.dev)
        self.alpha_f = self.geo["part"].alpha_f = math.sqrt(nb / w.ffn_keep)  # the subnet's scale (Sec. 3.4)
        if self.has_attn:
            self.alpha_a = self.geo["part"].alpha_a = math.sqrt(H / w.head_keep)
            self.t_idx_head = torch.empty(L, S, w.head_keep, **i32)           # the sampled head blueprints
            self.t_pos_head = torch.empty(L, S, H, **i32)
            self.t_kv = [torch.empty(L, S, Hkv, **i32), torch.empty(L, S, **i32), torch.empty(L, S, **i32),
                         torch.empty(L, S, Hkv, **i32)]                       # kv_idx, kv_count, kv_cols, kv_pos (unused)
            # what gather and aggregate see: every worker holds every head / group at its own position
            self.idx_head.copy_(torch.arange(H, **i32).expand(L, S, H))
            self.pos_head.copy_(torch.arange(H, **i32).expand(L, S, H))
            self.kv_idx.copy_(torch.arange(Hkv, **i32).expand(L, S, Hkv))
            self.kv_pos.copy_(torch.arange(Hkv, **i32).expand(L, S, Hkv))
            self.kv_count.fill_(Hkv)
            self.kv_cols.fill_(Hkv * w.d_head)
            self.qkv_mask = torch.zeros(S, self.nq, dtype=torch.uint8, device=self.dev)
            self.qkv_count = torch.zeros(S, **i32)
            self.a_mask = torch.zeros(S, self.a_sub, dtype=torch.uint8, device=self.dev)
            self.a_masked = torch.empty(S, w.tokens, self.a_sub, dtype=torch.bfloat16, device=self.dev)

    def o_step(self, l: int, k: int, lr: Optional[float] = None):
        """The head mask multiplies the head outputs (Sec. 4.1) before the output projection sees them."""
        w = self.true_w
        B.twist_apply_col_mask(self.A[k], self.a_mask, self.a_masked, w.n_subnets, w.tokens, self.a_sub)
        self.launches += 1
        plain = self.A[k]
        self.A[k] = self.a_masked
        try:
            super().o_step(l, k, lr)
        finally:
            self.A[k] = plain

    def sample_masks(self, rnd: int):
        w = self.true_w
        with self._timed("sample_masks"):
            B.twist_sample_masks(w.seed_mask, rnd, 0, w.n_layers, B.KIND_FFN, w.n_ffn_blocks, w.n_subnets, w.ffn_keep,
                                 list(w.common_ffn), w.sample_mode, self.idx_ffn, self.cover_ffn, self.pos_ffn)
            self.launches += 2
            if self.has_attn:
                B.twist_sample_masks(w.seed_mask, rnd, 0, w.n_layers, B.KIND_HEAD, w.n_heads, w.n_subnets, w.head_keep,
                                     list(w.common_heads), w.sample_mode, self.t_idx_head, self.cover_head,
                                     self.t_pos_head)
                B.twist_kv_groups(self.t_idx_head, w.n_layers, w.n_subnets, w.head_keep, w.n_heads, w.n_kv_heads,
                                  w.d_head, self.t_kv[0], self.t_kv[1], self.t_kv[2], self.kv_cover, self.t_kv[3])
                self.launches += 4

    def gather_layer(self, l: int, which=("ffn", "attn")):
        super().gather_layer(l, which=which)
        w = self.true_w
        B.twist_hidden_mask(self.cover_ffn[l], w.n_ffn_blocks, w.ffn_block, 0, w.n_subnets, self.h_mask)
        self.launches += 1
        if self.has_attn:
            B.twist_qkv_col_mask(self.cover_head[l], self.kv_cover[l], w.n_heads, w.n_kv_heads, w.d_head, 0, w.n_subnets,
                                 self.qkv_mask, self.qkv_count)
            B.twist_hidden_mask(self.cover_head[l], w.n_heads, w.d_head, 0, w.n_subnets, self.a_mask)
            self.launches += 2

    def _qkv_loss_mask(self, l: int) -> dict:
        return dict(col_mask=self.qkv_mask, valid_cols=self.qkv_count)

    def _o_mask(self, l: int) -> dict:
        return dict(col_mask=self.a_mask)


class HybridRoundEngine(RoundEngine):
    """Hybrid TwIST (Sec. 4.1): worker 0 is the central model.  It keeps no slice: it trains its subnet in place on
    the full-width matrices under masks (an activation mask on the FFN block, a head mask on the attention blocks,
    as in MaskedRoundEngine), while workers 1 .. S-1 train gathered dense slices as in RoundEngine; the aggregator
    reads worker 0's rows from the full fp32 matrices (twist_aggregate_segment.central).  In exact arithmetic the
    round equals RoundEngine's.  (The full model's gate and up rows lie back to back, so a full-width layer is a
    valid w_gu operand.)  The central worker's batches of the attention blocks are full-width: Tq_c [1][T][(H + 2
    H_kv) d_head] (only the held columns are read), A_c [1][T][H d_head] (masked before the output projection)."""

    def __init__(self, w: Workload, device: str = "cuda", **kw):
        assert w.dtype == DTYPE_BF16 and w.n_subnets >= 2 and not w.shared_layers, "bf16 workloads without shared layers"
        super().__init__(w, device=device, keep_f32_full=True, **kw)
        assert self.fuse_loss or not self.has_attn, "the head mask of the QKV block acts in the fused loss"
        F, T, d = w.d_ff, w.tokens, w.d_model
        g, dev = self.g, self.dev
        bf = torch.bfloat16
        act = lambda width: torch.empty(1, T, width, dtype=bf, device=dev)
        self.c_pre, self.c_dpre, self.c_hh = act(g * F), act(g * F), act(F)
        self.c_mask = torch.zeros(1, F, dtype=torch.uint8, device=dev)
        f32 = lambda rows: torch.zeros(1, rows, d, dtype=torch.float32, device=dev)
        if self.adam:      # the central worker's moments are full-width like its weights; zeroed when its layer starts
            self.c_gu_m1, self.c_gu_m2, self.c_down_m1, self.c_down_m2 = f32(g * F), f32(g * F), f32(F), f32(F)
        if self.has_attn:
            H, Hkv, dh = w.n_heads, w.n_kv_heads, w.d_head
            self.c_nq, self.c_a = (H + 2 * Hkv) * dh, H * dh
            self.c_qkv_mask = torch.zeros(1, self.c_nq, dtype=torch.uint8, device=dev)
            self.c_qkv_count = torch.zeros(1, dtype=torch.int32, device=dev)
            self.c_a_mask = torch.zeros(1, self.c_a, dtype=torch.uint8, device=dev)
            self.c_a_masked, self.c_dqkv = act(self.c_a), act(self.c_nq)
            self.c_qkv_out = act(self.c_nq) if self.store_outputs else None
            self.c_da = act(self.c_a) if self.compute_dx else None
            self.Tq_c: List[torch.Tensor] = []
            self.A_c: List[torch.Tensor] = []
            if self.adam:
                self.c_qkv_m1, self.c_qkv_m2, self.c_o_m1, self.c_o_m2 = f32(self.c_nq), f32(self.c_nq), f32(self.c_a), f32(self.c_a)

    def _central_opt(self, k: int, *pairs):
        if not self.adam:
            return {}
        w = self.w
        kw = {"opt": B.adam(k + 1, w.beta1, w.beta2, w.adam_eps)}
        for arg, name in pairs:
            kw["m" + arg] = getattr(self, name + "_m1")
            kw["v" + arg] = getattr(self, name + "_m2")
        return kw

    def _others_opt(self, k: int, *pairs):
        return {key: (v if key == "opt" else v[1:]) for key, v in self._opt(k, *pairs).items()}

    def gather_layer(self, l: int, which=("ffn", "attn")):
        """Slices of workers 1 .. S-1 only; the central worker's masks for this layer."""
        w, d = self.w, self.w.d_model
        f, gf = self.f_sub, self.gf
        idx = self.idx_ffn[l, 1:]
        segs = []
        for m, off, dst, dst_m, stride in ([("gate", 0, self.w_gu, self.w_gu_m, gf)] if self.g == 2 else []) + [
                ("up", f if self.g == 2 else 0, self.w_gu, self.w_gu_m, gf), ("down", 0, self.w_down, self.w_down_m, f)]:
            segs.append(B.gather_segment(self.full[m][l], dst[1:], self._gather_master(dst_m[1:]), idx, None, w.ffn_keep,
                                         w.ffn_keep, w.ffn_block, 0, stride * d, off, w.n_ffn_blocks))
        if self.has_attn:
            H, Hkv, dh, hk = w.n_heads, w.n_kv_heads, w.d_head, w.head_keep
            qkv, ih, ik, ic = self.full["qkv"][l], self.idx_head[l, 1:], self.kv_idx[l, 1:], self.kv_count[l, 1:]
            q_dst, q_m = self.w_qkv[1:], self._gather_master(self.w_qkv_m[1:])
            segs.append(B.gather_segment(qkv, q_dst, q_m, ih, None, hk, hk, dh, 0, self.nq * d, 0, H))
            segs.append(B.gather_segment(qkv, q_dst, q_m, ik, ic, Hkv, self.kv_max, dh, H * dh, self.nq * d, self.a_sub, Hkv))
            segs.append(B.gather_segment(qkv, q_dst, q_m, ik, ic, Hkv, self.kv_max, dh, (H + Hkv) * dh, self.nq * d,
                                         self.a_sub + self.kv_max * dh, Hkv))
            segs.append(B.gather_segment(self.full["o"][l], self.w_o[1:], self._gather_master(self.w_o_m[1:]), ih, None,
                                         hk, hk, dh, 0, self.a_sub * d, 0, H))
        with self._timed("gather"):
            B.twist_gather_subnets(segs, w.n_subnets - 1, d, w.dtype)
            B.twist_hidden_mask(self.cover_ffn[l], w.n_ffn_blocks, w.ffn_block, 0, 1, self.c_mask)
            if self.has_attn:
                B.twist_qkv_col_mask(self.cover_head[l], self.kv_cover[l], w.n_heads, w.n_kv_heads, w.d_head, 0, 1,
                                     self.c_qkv_mask, self.c_qkv_count)
                B.twist_hidden_mask(self.cover_head[l], w.n_heads, w.d_head, 0, 1, self.c_a_mask)
                self.launches += 2
            for n in self.moment_names:        # a fresh worker state, also for the central worker
                getattr(self, n).zero_()
            if self.adam:
                for n in ("c_gu", "c_down") + (("c_qkv", "c_o") if self.has_attn else ()):
                    getattr(self, n + "_m1").zero_()
                    getattr(self, n + "_m2").zero_()
        self.launches += 2

    def ffn_step(self, l: int, k: int, lr: Optional[float] = None):
        w = self.w
        lr = w.lr if lr is None else lr
        S, T, d, F = w.n_subnets, w.tokens, w.d_model, w.d_ff
        central_opt = self._central_opt(k, ("_gu", "c_gu"), ("_down", "c_down"))
        others_opt = self._others_opt(k, ("_gu", "w_gu"), ("_down", "w_down"))
        # central worker: the full-width layer under its mask, updated in place
        c = self._ffn_args(w.ffn_kind, w.dtype, 1, T, d, F, self.alpha_f, lr, x=self.X[k][:1], w_gu=self.full_gu[l],
                       w_down=self.full["down"][l], w_gu_master=self.full_gu_f32[l],
                       w_down_master=self.full_f32["down"][l], pre=self.c_pre, hh=self.c_hh,
                       y=self.y[:1] if self.store_outputs else None, dy=self.dy[:1], dpre=self.c_dpre,
                       dx=self.dx[:1] if self.dx is not None else None, hidden_mask=self.c_mask,
                       tgt=self.Td[k][:1], loss=self.loss[l, 0, k][:1], loss_ws=self.ws, **central_opt)
        # workers 1 .. S-1: gathered slices
        o = self._ffn_args(w.ffn_kind, w.dtype, S - 1, T, d, w.f_sub, self.alpha_f, lr, x=self.X[k][1:], w_gu=self.w_gu[1:],
                       w_down=self.w_down[1:], w_gu_master=self.w_gu_m[1:], w_down_master=self.w_down_m[1:],
                       pre=self.pre[1:], hh=self.hh[1:], y=self.y[1:] if self.store_outputs else None, dy=self.dy[1:],
                       dpre=self.dpre[1:], dx=self.dx[1:] if self.dx is not None else None, tgt=self.Td[k][1:],
                       loss=self.loss[l, 0, k][1:], loss_ws=self.ws, **self._first(k), **others_opt)
        with self._timed("ffn_fwd"):
            B.twist_subnet_ffn_fwd(c)
            B.twist_subnet_ffn_fwd(o)
        with self._timed("ffn_bwd"):
            B.twist_subnet_ffn_bwd(c)
            B.twist_subnet_ffn_bwd(o)
        self.launches += 2 * (2 + 3 + (1 if self.compute_dx else 0))

    def qkv_step(self, l: int, k: int, lr: Optional[float] = None):
        w = self.w
        lr = w.lr if lr is None else lr
        S, T, d = w.n_subnets, w.tokens, w.d_model
        dx = lambda sl: self.dx[sl] if self.dx is not None else None
        c = self._proj_args(B.PROJ_QKV, w.dtype, 1, T, d, self.c_nq, 1.0, lr, in_=self.X[k][:1], w=self.full["qkv"][l],
                        w_master=self.full_f32["qkv"][l], out=self.c_qkv_out, d_out=self.c_dqkv, d_in=dx(slice(0, 1)),
                        tgt=self.Tq_c[k], loss=self.loss[l, 1, k][:1], loss_ws=self.ws, col_mask=self.c_qkv_mask,
                        valid_cols=self.c_qkv_count, **self._central_opt(k, ("", "c_qkv")))
        mask = {key: (v[1:] if key == "valid_cols" else v) for key, v in self._qkv_loss_mask(l).items()}
        o = self._proj_args(B.PROJ_QKV, w.dtype, S - 1, T, d, self.nq, 1.0, lr, in_=self.X[k][1:], w=self.w_qkv[1:],
                        w_master=self.w_qkv_m[1:], out=self.qkv_out[1:] if self.store_outputs else None,
                        d_out=self.dqkv[1:], d_in=dx(slice(1, None)), tgt=self.Tq[k][1:], loss=self.loss[l, 1, k][1:],
                        loss_ws=self.ws, **mask, **self._first(k), **self._others_opt(k, ("", "w_qkv")))
        with self._timed("qkv_fwd"):
            B.twist_subnet_attn_proj_fwd(c)
            B.twist_subnet_attn_proj_fwd(o)
        with self._timed("qkv_bwd"):
            B.twist_subnet_attn_proj_bwd(c)
            B.twist_subnet_attn_proj_bwd(o)
        self.launches += 2 * (1 + 1 + (1 if self.compute_dx else 0))

    def o_step(self, l: int, k: int, lr: Optional[float] = None):
        w = self.w
        lr = w.lr if lr is None else lr
        S, T, d = w.n_subnets, w.tokens, w.d_model
        B.twist_apply_col_mask(self.A_c[k], self.c_a_mask, self.c_a_masked, 1, T, self.c_a)     # Sec. 4.1: M * f(x)
        c = self._proj_args(B.PROJ_O, w.dtype, 1, T, d, self.c_a, self.alpha_a, lr, in_=self.c_a_masked, w=self.full["o"][l],
                        w_master=self.full_f32["o"][l], out=self.y[:1] if self.store_outputs else None,
                        d_out=self.dy[:1], d_in=self.c_da, tgt=self.Td[k][:1], loss=self.loss[l, 2, k][:1],
                        loss_ws=self.ws, col_mask=self.c_a_mask, **self._central_opt(k, ("", "c_o")))
        o = self._proj_args(B.PROJ_O, w.dtype, S - 1, T, d, self.a_sub, self.alpha_a, lr, in_=self.A[k][1:], w=self.w_o[1:],
                        w_master=self.w_o_m[1:], out=self.y[1:] if self.store_outputs else None, d_out=self.dy[1:],
                        d_in=self.da[1:] if self.da is not None else None, tgt=self.Td[k][1:],
                        loss=self.loss[l, 2, k][1:], loss_ws=self.ws, **self._first(k), **self._others_opt(k, ("", "w_o")))
        with self._timed("o_fwd"):
            B.twist_subnet_attn_proj_fwd(c)
            B.twist_subnet_attn_proj_fwd(o)
        with self._timed("o_bwd"):
            B.twist_subnet_attn_proj_bwd(c)
            B.twist_subnet_attn_proj_bwd(o)
        self.launches += 1 + 2 * (1 + 1 + (1 if self.compute_dx else 0))

    def aggregate_layer(self, l: int, live: int = 0xFFFFFFFF, which=("ffn", "attn")):
        w, d = self.w, self.w.d_model
        f, gf = self.f_sub, self.gf
        nb = w.n_ffn_blocks
        segs = []
        for m, off, sub, stride in ([("gate", 0, self.w_gu_m, gf)] if self.g == 2 else []) + [
                ("up", f if self.g == 2 else 0, self.w_gu_m, gf), ("down", 0, self.w_down_m, f)]:
            segs.append(B.aggregate_segment(self.full[m][l], self.full_f32[m][l], sub, self.cover_ffn[l], self.pos_ffn[l],
                                            nb, w.ffn_block, 0, stride * d, off, w.ffn_keep,
                                            central=self.full_f32[m][l], central_subnet=0))
        if self.has_attn:
            H, Hkv, dh = w.n_heads, w.n_kv_heads, w.d_head
            qf, qs = self.full_f32["qkv"][l], self.w_qkv_m
            c = dict(central=qf, central_subnet=0)
            segs.append(B.aggregate_segment(self.full["qkv"][l], qf, qs, self.cover_head[l], self.pos_head[l], H, dh, 0,
                                            self.nq * d, 0, self.head_keep, **c))
            segs.append(B.aggregate_segment(self.full["qkv"][l], qf, qs, self.kv_cover[l], self.kv_pos[l], Hkv, dh,
                                            H * dh, self.nq * d, self.a_sub, self.kv_max, **c))
            segs.append(B.aggregate_segment(self.full["qkv"][l], qf, qs, self.kv_cover[l], self.kv_pos[l], Hkv, dh,
                                            (H + Hkv) * dh, self.nq * d, self.a_sub + self.kv_max * dh, self.kv_max, **c))
            segs.append(B.aggregate_segment(self.full["o"][l], self.full_f32["o"][l], self.w_o_m, self.cover_head[l],
                                            self.pos_head[l], H, dh, 0, self.a_sub * d, 0, self.head_keep,
                                            central=self.full_f32["o"][l], central_subnet=0))
        with self._timed("aggregate"):
            B.twist_aggregate(segs, w.n_subnets, d, w.dtype, live)
        self.launches += 1


def shard_range(n_subnets: int, rank: int, world: int) -> Tuple[int, int]:
    """(first subnet, number of subnets) of `rank` when S subnets are spread evenly over `world` GPUs."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("rank %d of %d" % (rank, world))
    if n_subnets % world != 0:
        raise ValueError("%d subnets do not divide over %d GPUs" % (n_subnets, world))
    per = n_subnets // world
    return rank * per, per


class ShardedRoundEngine(RoundEngine):
    """The S subnets of a round spread over `world` GPUs, one process per GPU (Sec. 4.1: workers train their subnets in
    parallel and a server averages them; here every GPU is worker for S / world subnets and all of them are the server).

    Every GPU holds the whole model and samples the blueprints of all S subnets (the sampler is a pure function of
    (seed, round, layer, kind), so nothing is exchanged for that), gathers and trains only its own subnets
    subnet_begin .. subnet_begin + S / world - 1, and the aggregate runs in two halves around the one exchange of
    the round: twist_aggregate_partial (fp32 sums of this GPU's subnets, zeros elsewhere, in full-matrix geometry), an
    all-reduce (sum) of that buffer over the GPUs, twist_aggregate_finish (division by the global coverage counts,
    written to the fp32 model and its bf16 shadow).  After it every GPU holds the same new model.  `reduce` is the
    exchange: by default torch.distributed.all_reduce on the process group (NCCL), nothing when world == 1.
    The batches (X, Td, Tq, A) the caller loads are those of the GPU's own subnets."""

    def __init__(self, w: Workload, rank: int = 0, world: int = 1, reduce=None, device: str = "cuda", **kw):
        from dataclasses import replace
        self.global_w = w
        self.rank, self.world = rank, world
        self.subnet_begin, self.S_local = shard_range(w.n_subnets, rank, world)
        self.S_global = w.n_subnets
        super().__init__(replace(w, n_subnets=self.S_local), device=device, **kw)
        lw, dev = self.w, self.dev
        L, S, nb = lw.n_layers, self.S_global, lw.n_ffn_blocks
        i32 = dict(dtype=torch.int32, device=dev)
        own = slice(self.subnet_begin, self.subnet_begin + self.S_local)
        # blueprints and ranks of ALL subnets; what the base class reads are views of this GPU's subnets
        self.g_pos_ffn = torch.empty(L, S, nb, **i32)
        self.pos_ffn = self.g_pos_ffn[:, own]
        self.g_idx_ffn, self.g_idx_head = {}, {}
        if self.has_attn:
            H, Hkv = lw.n_heads, lw.n_kv_heads
            self.g_pos_head = torch.empty(L, S, H, **i32)
            self.g_kv_idx = torch.empty(L, S, Hkv, **i32)
            self.g_kv_count = torch.empty(L, S, **i32)
            self.g_kv_cols = torch.empty(L, S, **i32)
            self.g_kv_pos = torch.empty(L, S, Hkv, **i32)
            self.pos_head, self.kv_idx, self.kv_pos = self.g_pos_head[:, own], self.g_kv_idx[:, own], self.g_kv_pos[:, own]
            self.kv_count, self.kv_cols = self.g_kv_count[:, own], self.g_kv_cols[:, own]
        for kind, gm in self.geo.items():
            self._use_kind(kind)
            self.g_idx_ffn[kind] = torch.empty(L, S, gm.ffn_keep, **i32)
            self.bufs[kind]["idx_ffn"] = self.idx_ffn = self.g_idx_ffn[kind][:, own]
            if self.has_attn:
                self.g_idx_head[kind] = torch.empty(L, S, gm.head_keep, **i32)
                self.bufs[kind]["idx_head"] = self.idx_head = self.g_idx_head[kind][:, own]
        self._use_kind("part")
        # partial sums of one layer, every matrix back to back: one buffer, one exchange
        rows = {m: v.shape[1] for m, v in self.full.items()}
        self.part = torch.zeros(sum(rows.values()), lw.d_model, dtype=torch.float32, device=dev)
        self.part_of, at = {}, 0
        for m, r in rows.items():
            self.part_of[m] = self.part[at:at + r]
            at += r
        self.reduce = reduce if reduce is not None else self._all_reduce

    def _all_reduce(self, t: torch.Tensor):
        if self.world > 1:
            import torch.distributed as dist
            dist.all_reduce(t, op=dist.ReduceOp.SUM)

    def sample_masks(self, rnd: int):
        w, S = self.w, self.S_global
        with self._timed("sample_masks"):
            for l0, n, kind in self._layer_runs():
                self._use_kind(kind)
                sl = slice(l0, l0 + n)
                B.twist_sample_masks(w.seed_mask, rnd, l0, n, B.KIND_FFN, w.n_ffn_blocks, S, self.ffn_keep,
                                     list(w.common_ffn), w.sample_mode, self.g_idx_ffn[kind][sl], self.cover_ffn[sl],
                                     self.g_pos_ffn[sl])
                self.launches += 2
                if self.has_attn:
                    B.twist_sample_masks(w.seed_mask, rnd, l0, n, B.KIND_HEAD, w.n_heads, S, self.head_keep,
                                         list(w.common_heads), w.sample_mode, self.g_idx_head[kind][sl],
                                         self.cover_head[sl], self.g_pos_head[sl])
                    B.twist_kv_groups(self.g_idx_head[kind][sl], n, S, self.head_keep, w.n_heads, w.n_kv_heads,
                                      w.d_head, self.g_kv_idx[sl], self.g_kv_count[sl], self.g_kv_cols[sl],
                                      self.kv_cover[sl], self.g_kv_pos[sl])
                    self.launches += 4

    def aggregate_partial(self, l: int, live: int = 0xFFFFFFFF, which=("ffn", "attn")):
        """This GPU's fp32 sums of layer l into self.part."""
        self._use(l)
        w = self.w
        if w.dtype == DTYPE_BF16:
            segs = self._aggregate_segments(l, which, lambda m: self.full[m][l], lambda m: self.part_of[m])
        else:
            segs = self._aggregate_segments(l, which, lambda m: self.part_of[m], lambda m: None)
        with self._timed("aggregate"):
            B.twist_aggregate_partial(segs, self.S_local, self.subnet_begin, w.d_model, w.dtype, live)
        self.launches += 1

    def aggregate_finish(self, l: int, live: int = 0xFFFFFFFF, which=("ffn", "attn")):
        """The reduced sums in self.part divided by the coverage counts into the model."""
        self._use(l)
        w = self.w
        f32 = (lambda m: self.full_f32[m][l]) if self.full_f32 is not None else (lambda m: None)
        segs = self._aggregate_segments(l, which, lambda m: self.full[m][l], f32, central=lambda m: self.part_of[m])
        with self._timed("aggregate"):
            B.twist_aggregate_finish(segs, self.S_global, w.d_model, w.dtype, live)
        self.launches += 1

    def aggregate_layer(self, l: int, live: int = 0xFFFFFFFF, which=("ffn", "attn")):
        self.aggregate_partial(l, live, which)
        with self._timed("exchange"):
            self.reduce(self.part)
        self.aggregate_finish(l, live, which)


class StackEngine(RoundEngine):
    """One TwIST round in the chained (STACK) composition: every local step runs all layers,
    x <- x + alpha_a * O(core(QKV(LN_a(x)))),  x <- x + alpha_f * FFN(LN_f(x)),  with one loss on the final x
    (App. A, Transformer Layer Architecture; the two layer normalisations only when the workload asks for them).

    All layers' slices and saved activations are resident at once (the backward pass needs them), so
    this engine is for the stack-shaped workloads whose activations fit; the streamed RoundEngine
    covers the per-block workloads.  Like RoundEngine it only allocates buffers and calls the C ABI.
    The normalised activations are not kept: the backward pass forms them again from the saved inputs.
    """

    def __init__(self, w: Workload, n_seqs: int, seq_len: int, device: str = "cuda", keep_f32_full: bool = False):
        assert w.n_heads > 0 and w.dtype == DTYPE_BF16 and n_seqs * seq_len == w.tokens
        super().__init__(w, device=device, keep_f32_full=keep_f32_full, compute_dx=True, fuse_loss=False)
        self.n_seqs, self.seq_len = n_seqs, seq_len
        S, T, d, L = w.n_subnets, w.tokens, w.d_model, w.n_layers
        dev, bf = self.dev, torch.bfloat16
        for kind in self.geo:
            self._use_kind(kind)
        self._use_kind("part")
        # slices of every layer: the first layer of a kind uses the geometry's own buffers
        self.slices: List[Dict[str, torch.Tensor]] = []
        seen = set()
        for l in range(L):
            kind = self.kind_of(l)
            b = self.bufs[kind]
            names = [n for n in b if (n in _SLICES or n.endswith(("_m", "_m1", "_m2"))) and torch.is_tensor(b[n])]
            self.slices.append({n: (b[n] if kind not in seen else torch.empty_like(b[n])) for n in names})
            seen.add(kind)
        act = lambda width: torch.empty(S, T, width, dtype=bf, device=dev)
        geo = [self.geo[self.kind_of(l)] for l in range(L)]
        self.x = [act(d) for _ in range(L + 1)]
        self.x_mid = [act(d) for _ in range(L)]
        self.qkv_l = [act(geo[l].nq) for l in range(L)]
        self.a_l = [act(geo[l].a_sub) for l in range(L)]
        self.pre_l = [act(geo[l].gf) for l in range(L)]
        self.hh_l = [act(geo[l].f_sub) for l in range(L)]
        self.lse = [torch.empty(S, geo[l].head_keep, T, dtype=torch.float32, device=dev) for l in range(L)]
        self.delta = torch.empty(S, max(gm.head_keep for gm in geo), T, dtype=torch.float32, device=dev)
        self.grad = [act(d), act(d)]            # gradient w.r.t. the residual stream (ping-pong)
        self.stack_loss = torch.zeros(max(1, w.local_steps), S, dtype=torch.float32, device=dev)
        self.gqa = w.n_kv_heads != w.n_heads
        # layer normalisation (App. A): shared parameters, one copy per worker and layer, statistics per token
        self.ln = w.layer_norm
        if self.ln:
            f32 = lambda *shape: torch.empty(*shape, dtype=torch.float32, device=dev)
            self.full_ln = {n: f32(L, d) for n in LN_PARAMS}
            self.ln_w = [{n: f32(S, d) for n in LN_PARAMS} for _ in range(L)]
            self.ln_mom = [{n + t: torch.zeros(S, d, dtype=torch.float32, device=dev) for n in LN_PARAMS
                            for t in ("_m1", "_m2")} if self.adam else {} for _ in range(L)]
            self.ln_stat = [{n: f32(S, T) for n in ("mean_a", "rstd_a", "mean_f", "rstd_f")} for _ in range(L)]
            self.x_ln, self.d_ln = act(d), act(d)         # a normalised activation / the gradient w.r.t. one
            self.ln_ws = torch.empty(B.twist_layernorm_workspace_bytes(S, T, d), dtype=torch.uint8, device=dev)
            self.ln_zero_idx = torch.zeros(S, 1, dtype=torch.int32, device=dev)
            mask = (1 << S) - 1
            self.ln_cover = torch.tensor([mask - (1 << 32) if mask >= (1 << 31) else mask], dtype=torch.int32, device=dev)

    def _bind(self, l: int):
        self._use(l)
        for n, t in self.slices[l].items():
            setattr(self, n, t)

    def _core_args(self, l: int, **t):
        w = self.w
        extra = dict(head_idx=self.idx_head[l], kv_pos=self.kv_pos[l], kv_count=self.kv_count[l]) if self.gqa else {}
        return self._attn_core_args(w.dtype, w.n_subnets, self.n_seqs, self.seq_len, self.head_keep, self.kv_max, w.d_head,
                                w.n_heads, w.n_kv_heads, **extra, **t)

    # ------------------------------------------------------------------ layer normalisation
    def _ln_args(self, l: int, which: str, lr: float = 0.0, k: int = 0, **t):
        w = self.w
        p, st = self.ln_w[l], self.ln_stat[l]
        kw = {}
        if self.adam and lr != 0.0:
            m = self.ln_mom[l]
            kw = dict(opt=B.adam(k + 1, w.beta1, w.beta2, w.adam_eps), m_gamma=m[f"ln_{which}_g_m1"],
                      v_gamma=m[f"ln_{which}_g_m2"], m_beta=m[f"ln_{which}_b_m1"], v_beta=m[f"ln_{which}_b_m2"])
        return B.layernorm_args(w.dtype, w.n_subnets, w.tokens, w.d_model, w.ln_eps, lr, gamma=p[f"ln_{which}_g"],
                                beta=p[f"ln_{which}_b"], mean=st["mean_" + which], rstd=st["rstd_" + which], **kw, **t)

    def _ln_fwd(self, l: int, which: str, x, y):
        with self._timed("ln_fwd"):
            B.twist_layernorm_fwd(self._ln_args(l, which, x=x, y=y))
        self.launches += 1

    def _ln_bwd(self, l: int, which: str, k: int, lr: float, x, dy, dx, residual):
        with self._timed("ln_bwd"):
            B.twist_layernorm_bwd(self._ln_args(l, which, lr, k, x=x, dy=dy, dx=dx, dx_residual=residual, ws=self.ln_ws))
        self.launches += 3

    def gather_ln(self, l: int):
        """The shared normalisation parameters are broadcast: every worker gets a copy (Sec. 3.2)."""
        w, d = self.w, self.w.d_model
        segs = [B.gather_segment(self.full_ln[n][l], self.ln_w[l][n], None, self.ln_zero_idx, None, 1, 1, 1, 0, d, 0, 1)
                for n in LN_PARAMS]
        B.twist_gather_subnets(segs, w.n_subnets, d, B.FP32)
        for t in self.ln_mom[l].values():
            t.zero_()
        self.launches += 1

    def aggregate_ln(self, l: int, live: int = 0xFFFFFFFF):
        """Held by every worker: the aggregator's formula (Sec. 3.3) is the plain mean over the S copies."""
        w, d = self.w, self.w.d_model
        segs = [B.aggregate_segment(self.full_ln[n][l], None, self.ln_w[l][n], self.ln_cover, self.ln_zero_idx, 1, 1, 0,
                                    d, 0, 1) for n in LN_PARAMS]
        B.twist_aggregate(segs, w.n_subnets, d, B.FP32, live)
        self.launches += 1

    # ------------------------------------------------------------------ the chained local step
    def forward(self, k: int):
        w = self.w
        S, T, d = w.n_subnets, w.tokens, w.d_model
        self.x[0].copy_(self.X[k])
        for l in range(w.n_layers):
            self._bind(l)
            x_a = self.x[l]
            if self.ln:
                self._ln_fwd(l, "a", self.x[l], self.x_ln)
                x_a = self.x_ln
            with self._timed("qkv_fwd"):
                B.twist_subnet_attn_proj_fwd(self._proj_args(B.PROJ_QKV, w.dtype, S, T, d, self.nq, 1.0, 0.0, in_=x_a,
                                                         w=self.w_qkv, out=self.qkv_l[l]))
            with self._timed("core_fwd"):
                B.twist_attn_core_fwd(self._core_args(l, qkv=self.qkv_l[l], out=self.a_l[l], lse=self.lse[l]))
            with self._timed("o_fwd"):
                B.twist_subnet_attn_proj_fwd(self._proj_args(B.PROJ_O, w.dtype, S, T, d, self.a_sub, self.alpha_a, 0.0,
                                                         in_=self.a_l[l], w=self.w_o, out=self.x_mid[l],
                                                         out_residual=self.x[l]))
            x_f = self.x_mid[l]
            if self.ln:
                self._ln_fwd(l, "f", self.x_mid[l], self.x_ln)
                x_f = self.x_ln
            with self._timed("ffn_fwd"):
                B.twist_subnet_ffn_fwd(self._ffn_args(w.ffn_kind, w.dtype, S, T, d, self.f_sub, self.alpha_f, 0.0,
                                                  x=x_f, w_gu=self.w_gu, w_down=self.w_down, pre=self.pre_l[l],
                                                  hh=self.hh_l[l], y=self.x[l + 1], y_residual=self.x_mid[l]))
            self.launches += 5

    def backward(self, k: int, lr: Optional[float] = None):
        w = self.w
        lr = w.lr if lr is None else lr
        S, T, d = w.n_subnets, w.tokens, w.d_model
        g, g_mid = self.grad
        for l in reversed(range(w.n_layers)):
            self._bind(l)
            # FFN block.  With the normalisation: its input is formed again, its input gradient goes through the
            # normalisation's backward, which also adds the gradient arriving over the skip connection.
            x_f = self.x_mid[l]
            if self.ln:
                self._ln_fwd(l, "f", self.x_mid[l], self.x_ln)
                x_f = self.x_ln
            with self._timed("ffn_bwd"):
                B.twist_subnet_ffn_bwd(self._ffn_args(w.ffn_kind, w.dtype, S, T, d, self.f_sub, self.alpha_f, lr,
                                                  x=x_f, w_gu=self.w_gu, w_down=self.w_down,
                                                  w_gu_master=self.w_gu_m, w_down_master=self.w_down_m,
                                                  pre=self.pre_l[l], hh=self.hh_l[l], dy=g, dpre=self.dpre,
                                                  dx=self.d_ln if self.ln else g_mid,
                                                  dx_residual=None if self.ln else g, dw_gu=self.dw_gu,
                                                  dw_down=self.dw_down, **self._first(k),
                                                  **self._opt(k, ("_gu", "w_gu"), ("_down", "w_down"))))
            if self.ln:
                self._ln_bwd(l, "f", k, lr, self.x_mid[l], self.d_ln, g_mid, g)
            with self._timed("o_bwd"):
                B.twist_subnet_attn_proj_bwd(self._proj_args(B.PROJ_O, w.dtype, S, T, d, self.a_sub, self.alpha_a, lr,
                                                         in_=self.a_l[l], w=self.w_o, w_master=self.w_o_m, d_out=g_mid,
                                                         d_in=self.da, dw=self.dw_o, **self._first(k),
                                                         **self._opt(k, ("", "w_o"))))
            with self._timed("core_bwd"):
                B.twist_attn_core_bwd(self._core_args(l, qkv=self.qkv_l[l], out=self.a_l[l], lse=self.lse[l],
                                                      d_out=self.da, d_qkv=self.dqkv, delta=self.delta))
            x_a = self.x[l]
            if self.ln:
                self._ln_fwd(l, "a", self.x[l], self.x_ln)
                x_a = self.x_ln
            with self._timed("qkv_bwd"):
                B.twist_subnet_attn_proj_bwd(self._proj_args(B.PROJ_QKV, w.dtype, S, T, d, self.nq, 1.0, lr, in_=x_a,
                                                         w=self.w_qkv, w_master=self.w_qkv_m, d_out=self.dqkv,
                                                         d_in=self.d_ln if self.ln else g,
                                                         d_in_residual=None if self.ln else g_mid, dw=self.dw_qkv,
                                                         **self._first(k), **self._opt(k, ("", "w_qkv"))))
            if self.ln:
                self._ln_bwd(l, "a", k, lr, self.x[l], self.d_ln, g, g_mid)
            self.launches += 4 + 2 + 3 + 2

    def local_step(self, k: int, lr: Optional[float] = None):
        w = self.w
        self.forward(k)
        with self._timed("mse"):
            B.twist_mse_fwd_bwd(self.x[w.n_layers], self.Td[k], self.grad[0], self.stack_loss[k], w.n_subnets, w.tokens,
                                w.d_model, None, 0, 0, w.dtype, self.ws)
        self.launches += 2
        self.backward(k, lr)

    def _gather_all(self):
        for l in range(self.w.n_layers):
            self._bind(l)
            self.gather_layer(l)
            if self.ln:
                self.gather_ln(l)

    def extract(self, rnd: int):
        """Deployment (Sec. 4.2): sample blueprints as in training and gather every layer's dense slices; the S
        extracted subnets are then resident (self.slices) for forward-only inference."""
        self.sample_masks(rnd)
        self._gather_all()

    def evaluate(self, k: int) -> torch.Tensor:
        """Evaluation mode for subnets (Sec. 4.2): forward only through the whole stack of every extracted subnet on
        batch k with the subnets' own scales, no update.  An engine built with keep counts other than the training
        run's evaluates a mismatched subnet ratio.  Returns the losses [S] (device); callers average over workers."""
        w = self.w
        self.forward(k)
        B.twist_mse_fwd_bwd(self.x[w.n_layers], self.Td[k], self.grad[0], self.stack_loss[k], w.n_subnets, w.tokens,
                            w.d_model, None, 0, 0, w.dtype, self.ws)
        self.launches += 2
        return self.stack_loss[k]

    def run_round(self, rnd: int):
        """Resample, gather every layer, K local steps through the whole stack, aggregate every layer."""
        w = self.w
        self.sample_masks(rnd)
        self._gather_all()
        for k in range(w.local_steps):
            self.local_step(k)
        for l in range(w.n_layers):
            self._bind(l)
            self.aggregate_layer(l)
            if self.ln:
                self.aggregate_ln(l)
