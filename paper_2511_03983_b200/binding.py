"""Thin ctypes binding of the C ABI in include/twist.h (argument marshalling only).

Every function has the name of its C entry point.  Tensors are torch CUDA tensors
(torch is used for device memory and streams only); the binding passes their
data pointers and the current CUDA stream.  A non-zero status raises TwistError.
The shared library must exist: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtwist.so")

OK = 0
ERR_NULL, ERR_SHAPE, ERR_INFEASIBLE, ERR_BAD_INDEX, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_DEVICE_TIMEOUT = \
    -1, -2, -3, -4, -5, -6, -7, -8
FP32, BF16 = 0, 1
FFN_RELU, FFN_GELU, FFN_SWIGLU = 0, 1, 2
MODE_COVER, MODE_IID = 0, 1
KIND_FFN, KIND_HEAD = 0, 1
PROJ_QKV, PROJ_O = 0, 1
MAX_SEGMENTS = 8

EXPORTS = [
    "twist_abi_version", "twist_strerror", "twist_last_cuda_error", "twist_device_status", "twist_sample_masks",
    "twist_kv_groups", "twist_gather_subnets", "twist_aggregate", "twist_subnet_ffn_fwd", "twist_subnet_ffn_bwd",
    "twist_subnet_attn_proj_fwd", "twist_subnet_attn_proj_bwd", "twist_mse_workspace_bytes", "twist_mse_fwd_bwd",
    "twist_mse_fwd_bwd_noalloc", "twist_fused_loss_workspace_bytes", "twist_attn_core_fwd", "twist_attn_core_bwd",
    "twist_hidden_mask", "twist_selftest_wait", "twist_layernorm_workspace_bytes", "twist_layernorm_fwd",
    "twist_layernorm_bwd", "twist_qkv_col_mask", "twist_apply_col_mask", "twist_plan_create", "twist_plan_destroy",
    "twist_plan_stats", "twist_workspace_bytes", "twist_aggregate_partial", "twist_aggregate_finish",
]


class TwistError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__(f"{where}: status {status} ({detail})")


class GatherSegment(C.Structure):
    _fields_ = [("src", C.c_void_p), ("dst", C.c_void_p), ("dst_master", C.c_void_p), ("idx", C.c_void_p),
                ("count", C.c_void_p), ("idx_stride", C.c_int32), ("n_keep", C.c_int32), ("block_rows", C.c_int32),
                ("n_blocks", C.c_int32), ("src_row_offset", C.c_int64), ("dst_subnet_stride", C.c_int64),
                ("dst_row_offset", C.c_int64)]


class AggregateSegment(C.Structure):
    _fields_ = [("dst", C.c_void_p), ("dst_f32", C.c_void_p), ("sub", C.c_void_p), ("cover", C.c_void_p),
                ("pos", C.c_void_p), ("n_full", C.c_int32), ("block_rows", C.c_int32), ("dst_row_offset", C.c_int64),
                ("sub_subnet_stride", C.c_int64), ("sub_row_offset", C.c_int64), ("central", C.c_void_p),
                ("central_subnet", C.c_int32), ("n_keep", C.c_int32)]


class Optimizer(C.Structure):
    _fields_ = [("kind", C.c_int32), ("step", C.c_int32), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float)]


OPT_SGD, OPT_ADAM = 0, 1


def adam(step: int, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8) -> Optimizer:
    return Optimizer(OPT_ADAM, step, beta1, beta2, eps)


class FfnArgs(C.Structure):
    _fields_ = [("ffn_kind", C.c_int32), ("dtype", C.c_int32), ("n_subnets", C.c_int32), ("tokens", C.c_int32),
                ("d_model", C.c_int32), ("f_sub", C.c_int32), ("out_scale", C.c_float), ("lr", C.c_float),
                ("x", C.c_void_p), ("w_gu", C.c_void_p), ("w_down", C.c_void_p), ("w_gu_master", C.c_void_p),
                ("w_down_master", C.c_void_p), ("pre", C.c_void_p), ("hh", C.c_void_p), ("y", C.c_void_p),
                ("dy", C.c_void_p), ("dpre", C.c_void_p), ("dx", C.c_void_p), ("dw_gu", C.c_void_p),
                ("dw_down", C.c_void_p), ("tgt", C.c_void_p), ("loss", C.c_void_p), ("loss_ws", C.c_void_p),
                ("loss_ws_bytes", C.c_size_t), ("y_residual", C.c_void_p), ("dx_residual", C.c_void_p),
                ("opt", Optimizer), ("m_gu", C.c_void_p), ("v_gu", C.c_void_p), ("m_down", C.c_void_p),
                ("v_down", C.c_void_p), ("hidden_mask", C.c_void_p), ("plan", C.c_void_p),
                ("master_from_slice", C.c_int32)]


class ProjArgs(C.Structure):
    _fields_ = [("which", C.c_int32), ("dtype", C.c_int32), ("n_subnets", C.c_int32), ("tokens", C.c_int32),
                ("d_model", C.c_int32), ("n", C.c_int32), ("out_scale", C.c_float), ("lr", C.c_float),
                ("in_", C.c_void_p), ("w", C.c_void_p), ("w_master", C.c_void_p), ("out", C.c_void_p),
                ("d_out", C.c_void_p), ("d_in", C.c_void_p), ("dw", C.c_void_p), ("tgt", C.c_void_p),
                ("loss", C.c_void_p), ("loss_ws", C.c_void_p), ("loss_ws_bytes", C.c_size_t),
                ("valid_cols", C.c_void_p), ("seg_begin", C.c_int32), ("seg_width", C.c_int32),
                ("out_residual", C.c_void_p), ("d_in_residual", C.c_void_p), ("opt", Optimizer), ("m", C.c_void_p),
                ("v", C.c_void_p), ("col_mask", C.c_void_p), ("plan", C.c_void_p),
                ("master_from_slice", C.c_int32)]


class AttnCoreArgs(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("n_subnets", C.c_int32), ("n_seqs", C.c_int32), ("seq_len", C.c_int32),
                ("head_keep", C.c_int32), ("kv_max", C.c_int32), ("d_head", C.c_int32), ("n_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("qkv", C.c_void_p), ("out", C.c_void_p), ("lse", C.c_void_p),
                ("d_out", C.c_void_p), ("d_qkv", C.c_void_p), ("delta", C.c_void_p), ("head_idx", C.c_void_p),
                ("kv_pos", C.c_void_p), ("kv_count", C.c_void_p), ("plan", C.c_void_p)]


class Config(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("d_head", C.c_int32), ("d_ff", C.c_int32), ("ffn_kind", C.c_int32),
                ("n_subnets", C.c_int32), ("ffn_block", C.c_int32), ("ffn_keep", C.c_int32), ("head_keep", C.c_int32),
                ("sample_mode", C.c_int32), ("dtype", C.c_int32), ("tokens", C.c_int32), ("reserved", C.c_int32),
                ("seed", C.c_uint64)]


class Plan:
    """Owner of a twist_plan handle (the shapes of a workload and its cache of encoded tensor maps)."""

    def __init__(self, w):
        cfg = Config(C.sizeof(Config), w.n_layers, w.d_model, w.n_heads, w.n_kv_heads, w.d_head, w.d_ff, w.ffn_kind,
                     w.n_subnets, w.ffn_block, w.ffn_keep, w.head_keep, w.sample_mode, w.dtype, w.tokens, 0, w.seed_mask)
        self.handle = C.c_void_p()
        _check(lib().twist_plan_create(C.byref(cfg), C.byref(self.handle)), "twist_plan_create")

    @property
    def ptr(self) -> int:
        return self.handle.value

    def workspace_bytes(self) -> int:
        n = C.c_size_t(0)
        _check(lib().twist_workspace_bytes(self.handle, C.byref(n)), "twist_workspace_bytes")
        return n.value

    def stats(self):
        """(maps cached, cache hits, cache misses)"""
        a, b, c = C.c_uint64(0), C.c_uint64(0), C.c_uint64(0)
        _check(lib().twist_plan_stats(self.handle, C.byref(a), C.byref(b), C.byref(c)), "twist_plan_stats")
        return a.value, b.value, c.value

    def close(self):
        if self.handle and self.handle.value:
            lib().twist_plan_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class LayerNormArgs(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("n_subnets", C.c_int32), ("tokens", C.c_int32), ("d_model", C.c_int32),
                ("eps", C.c_float), ("lr", C.c_float), ("x", C.c_void_p), ("y", C.c_void_p), ("mean", C.c_void_p),
                ("rstd", C.c_void_p), ("gamma", C.c_void_p), ("beta", C.c_void_p), ("dy", C.c_void_p),
                ("dx", C.c_void_p), ("dx_residual", C.c_void_p), ("dgamma", C.c_void_p), ("dbeta", C.c_void_p),
                ("ws", C.c_void_p), ("ws_bytes", C.c_size_t), ("opt", Optimizer), ("m_gamma", C.c_void_p),
                ("v_gamma", C.c_void_p), ("m_beta", C.c_void_p), ("v_beta", C.c_void_p)]


_lib_handle = None


def lib() -> C.CDLL:
    """Loads libtwist.so (once).  Fails loudly when it has not been built."""
    global _lib_handle
    if _lib_handle is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2511_03983_b200.build` (there is no fallback)")
        h = C.CDLL(LIB_PATH)
        h.twist_abi_version.restype = C.c_uint32
        h.twist_strerror.restype = C.c_char_p
        h.twist_strerror.argtypes = [C.c_int32]
        h.twist_last_cuda_error.restype = C.c_char_p
        h.twist_device_status.argtypes = [C.POINTER(C.c_int32)]
        h.twist_selftest_wait.argtypes = [C.c_uint64, C.c_void_p]
        h.twist_sample_masks.argtypes = [C.c_uint64, C.c_uint64, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                         C.c_int32, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_void_p]
        h.twist_kv_groups.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        h.twist_hidden_mask.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
        h.twist_qkv_col_mask.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                         C.c_void_p, C.c_void_p, C.c_void_p]
        h.twist_plan_create.argtypes = [C.c_void_p, C.c_void_p]
        h.twist_plan_destroy.argtypes = [C.c_void_p]
        h.twist_plan_stats.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        h.twist_workspace_bytes.argtypes = [C.c_void_p, C.c_void_p]
        h.twist_apply_col_mask.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
        h.twist_gather_subnets.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
        h.twist_aggregate.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_uint32, C.c_void_p]
        h.twist_aggregate_partial.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_uint32,
                                              C.c_void_p]
        h.twist_aggregate_finish.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_uint32, C.c_void_p]
        h.twist_layernorm_workspace_bytes.restype = C.c_size_t
        h.twist_layernorm_workspace_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32]
        for name in ("twist_subnet_ffn_fwd", "twist_subnet_ffn_bwd", "twist_subnet_attn_proj_fwd",
                     "twist_subnet_attn_proj_bwd", "twist_attn_core_fwd", "twist_attn_core_bwd",
                     "twist_layernorm_fwd", "twist_layernorm_bwd"):
            getattr(h, name).argtypes = [C.c_void_p, C.c_void_p]
        h.twist_mse_workspace_bytes.restype = C.c_size_t
        h.twist_mse_workspace_bytes.argtypes = [C.c_int32]
        h.twist_fused_loss_workspace_bytes.restype = C.c_size_t
        h.twist_fused_loss_workspace_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32]
        h.twist_mse_fwd_bwd.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                        C.c_int32, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_size_t,
                                        C.c_void_p]
        h.twist_mse_fwd_bwd_noalloc.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                                C.c_int32, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
        for name in EXPORTS:
            f = getattr(h, name)
            if name not in ("twist_abi_version", "twist_strerror", "twist_last_cuda_error",
                            "twist_mse_workspace_bytes", "twist_fused_loss_workspace_bytes",
                            "twist_layernorm_workspace_bytes"):
                f.restype = C.c_int32
        _lib_handle = h
    return _lib_handle


def _check(status: int, where: str):
    if status != OK:
        h = lib()
        detail = h.twist_strerror(status).decode()
        if status == ERR_CUDA:
            detail += ": " + h.twist_last_cuda_error().decode()
        raise TwistError(status, where, detail)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def twist_abi_version() -> int:
    return lib().twist_abi_version()


def twist_device_status() -> int:
    code = C.c_int32(0)
    _check(lib().twist_device_status(C.byref(code)), "twist_device_status")
    return code.value


def twist_selftest_wait(limit_ns: int):
    """Runs the library's bounded waits on barriers nobody arrives at (test / bring-up only); afterwards
    twist_device_status() reports ERR_DEVICE_TIMEOUT once."""
    _check(lib().twist_selftest_wait(limit_ns, _stream()), "twist_selftest_wait")


def twist_sample_masks(seed, rnd, layer_begin, n_layers, kind, n_full, n_subnets, n_sub, common: Sequence[int],
                       sample_mode, idx, cover, pos):
    arr = (C.c_int32 * max(1, len(common)))(*common)
    _check(lib().twist_sample_masks(seed, rnd, layer_begin, n_layers, kind, n_full, n_subnets, n_sub,
                                    C.cast(arr, C.c_void_p) if len(common) else None, len(common), sample_mode,
                                    _ptr(idx), _ptr(cover), _ptr(pos), _stream()), "twist_sample_masks")


def twist_kv_groups(head_idx, n_layers, n_subnets, head_keep, n_heads, n_kv_heads, d_head, kv_idx, kv_count, kv_cols,
                    kv_cover, kv_pos):
    _check(lib().twist_kv_groups(_ptr(head_idx), n_layers, n_subnets, head_keep, n_heads, n_kv_heads, d_head,
                                 _ptr(kv_idx), _ptr(kv_count), _ptr(kv_cols), _ptr(kv_cover), _ptr(kv_pos), _stream()),
           "twist_kv_groups")


def gather_segment(src, dst, dst_master, idx, count, idx_stride, n_keep, block_rows, src_row_offset,
                   dst_subnet_stride, dst_row_offset, n_blocks) -> GatherSegment:
    """Marshals one twist_gather_segment.  src/dst/... may be tensors or raw device addresses (ints).
    n_blocks: blocks in the partitioned range of src (the range idx entries are checked against)."""
    a = lambda v: v if (v is None or isinstance(v, int)) else _ptr(v)
    return GatherSegment(a(src), a(dst), a(dst_master), a(idx), a(count), idx_stride, n_keep, block_rows, n_blocks,
                         src_row_offset, dst_subnet_stride, dst_row_offset)


def twist_gather_subnets(segs: Sequence[GatherSegment], n_subnets, d, dtype):
    arr = (GatherSegment * len(segs))(*segs)
    _check(lib().twist_gather_subnets(C.cast(arr, C.c_void_p), len(segs), n_subnets, d, dtype, _stream()),
           "twist_gather_subnets")


def aggregate_segment(dst, dst_f32, sub, cover, pos, n_full, block_rows, dst_row_offset, sub_subnet_stride,
                      sub_row_offset, n_keep, central=None, central_subnet=0) -> AggregateSegment:
    """Marshals one twist_aggregate_segment.  n_keep: blocks of the segment in a subnet's slice (the range the
    ranks in pos are checked against)."""
    a = lambda v: v if (v is None or isinstance(v, int)) else _ptr(v)
    return AggregateSegment(a(dst), a(dst_f32), a(sub), a(cover), a(pos), n_full, block_rows, dst_row_offset,
                            sub_subnet_stride, sub_row_offset, a(central), central_subnet, n_keep)


def twist_hidden_mask(cover, n_full, block_rows, subnet_begin, n_subnets, mask):
    _check(lib().twist_hidden_mask(_ptr(cover), n_full, block_rows, subnet_begin, n_subnets, _ptr(mask), _stream()),
           "twist_hidden_mask")


def twist_qkv_col_mask(head_cover, kv_cover, n_heads, n_kv_heads, d_head, subnet_begin, n_subnets, mask, count):
    _check(lib().twist_qkv_col_mask(_ptr(head_cover), _ptr(kv_cover), n_heads, n_kv_heads, d_head, subnet_begin,
                                    n_subnets, _ptr(mask), _ptr(count), _stream()), "twist_qkv_col_mask")


def twist_apply_col_mask(in_, mask, out, n_subnets, tokens, width):
    _check(lib().twist_apply_col_mask(_ptr(in_), _ptr(mask), _ptr(out), n_subnets, tokens, width, _stream()),
           "twist_apply_col_mask")


def twist_aggregate(segs: Sequence[AggregateSegment], n_subnets, d, dtype, live_subnets=0xFFFFFFFF):
    arr = (AggregateSegment * len(segs))(*segs)
    _check(lib().twist_aggregate(C.cast(arr, C.c_void_p), len(segs), n_subnets, d, dtype, live_subnets, _stream()),
           "twist_aggregate")


def twist_aggregate_partial(segs: Sequence[AggregateSegment], n_subnets, subnet_begin, d, dtype, live_subnets=0xFFFFFFFF):
    arr = (AggregateSegment * len(segs))(*segs)
    _check(lib().twist_aggregate_partial(C.cast(arr, C.c_void_p), len(segs), n_subnets, subnet_begin, d, dtype,
                                         live_subnets, _stream()), "twist_aggregate_partial")


def twist_aggregate_finish(segs: Sequence[AggregateSegment], n_subnets, d, dtype, live_subnets=0xFFFFFFFF):
    arr = (AggregateSegment * len(segs))(*segs)
    _check(lib().twist_aggregate_finish(C.cast(arr, C.c_void_p), len(segs), n_subnets, d, dtype, live_subnets, _stream()),
           "twist_aggregate_finish")


def _ws_bytes(ws) -> int:
    return 0 if ws is None else ws.numel() * ws.element_size()


def _plan_ptr(plan) -> Optional[int]:
    return None if plan is None else plan.ptr


def ffn_args(ffn_kind, dtype, n_subnets, tokens, d_model, f_sub, out_scale, lr=0.0, opt: Optional[Optimizer] = None,
             plan: Optional["Plan"] = None, master_from_slice: bool = False, **t) -> FfnArgs:
    """Marshals twist_ffn_args.  tgt / loss / loss_ws request the fused loss of the forward call; hidden_mask
    (uint8 [S][f_sub]) the activation mask of Masked TwIST."""
    names = ["x", "w_gu", "w_down", "w_gu_master", "w_down_master", "pre", "hh", "y", "dy", "dpre", "dx", "dw_gu",
             "dw_down", "tgt", "loss", "loss_ws"]
    moments = ["m_gu", "v_gu", "m_down", "v_down"]
    unknown = set(t) - set(names) - {"y_residual", "dx_residual", "hidden_mask"} - set(moments)
    assert not unknown, unknown
    a = FfnArgs(ffn_kind, dtype, n_subnets, tokens, d_model, f_sub, out_scale, lr, *[_ptr(t.get(n)) for n in names],
                _ws_bytes(t.get("loss_ws")), _ptr(t.get("y_residual")), _ptr(t.get("dx_residual")),
                opt if opt is not None else Optimizer(), *[_ptr(t.get(n)) for n in moments],
                _ptr(t.get("hidden_mask")), _plan_ptr(plan), int(master_from_slice))
    a._keepalive = list(t.values()) + [plan]      # the struct holds raw addresses: keep their owners alive with it
    return a


def twist_subnet_ffn_fwd(a: FfnArgs):
    _check(lib().twist_subnet_ffn_fwd(C.byref(a), _stream()), "twist_subnet_ffn_fwd")


def twist_subnet_ffn_bwd(a: FfnArgs):
    _check(lib().twist_subnet_ffn_bwd(C.byref(a), _stream()), "twist_subnet_ffn_bwd")


def proj_args(which, dtype, n_subnets, tokens, d_model, n, out_scale, lr=0.0, seg_begin=0, seg_width=0,
              opt: Optional[Optimizer] = None, plan: Optional["Plan"] = None, master_from_slice: bool = False,
              **t) -> ProjArgs:
    """Marshals twist_proj_args.  tgt / loss / loss_ws (and the optional column mask valid_cols,
    seg_begin, seg_width) request the fused loss of the forward call."""
    names = ["in_", "w", "w_master", "out", "d_out", "d_in", "dw", "tgt", "loss", "loss_ws"]
    unknown = set(t) - set(names) - {"valid_cols", "out_residual", "d_in_residual", "m", "v", "col_mask"}
    assert not unknown, unknown
    a = ProjArgs(which, dtype, n_subnets, tokens, d_model, n, out_scale, lr, *[_ptr(t.get(n)) for n in names],
                 _ws_bytes(t.get("loss_ws")), _ptr(t.get("valid_cols")), seg_begin, seg_width,
                 _ptr(t.get("out_residual")), _ptr(t.get("d_in_residual")), opt if opt is not None else Optimizer(),
                 _ptr(t.get("m")), _ptr(t.get("v")), _ptr(t.get("col_mask")), _plan_ptr(plan), int(master_from_slice))
    a._keepalive = list(t.values()) + [plan]
    return a


def twist_subnet_attn_proj_fwd(a: ProjArgs):
    _check(lib().twist_subnet_attn_proj_fwd(C.byref(a), _stream()), "twist_subnet_attn_proj_fwd")


def twist_subnet_attn_proj_bwd(a: ProjArgs):
    _check(lib().twist_subnet_attn_proj_bwd(C.byref(a), _stream()), "twist_subnet_attn_proj_bwd")


def attn_core_args(dtype, n_subnets, n_seqs, seq_len, head_keep, kv_max, d_head, n_heads=0, n_kv_heads=0,
                   plan: Optional["Plan"] = None, **t) -> AttnCoreArgs:
    names = ["qkv", "out", "lse", "d_out", "d_qkv", "delta", "head_idx", "kv_pos", "kv_count"]
    unknown = set(t) - set(names)
    assert not unknown, unknown
    a = AttnCoreArgs(dtype, n_subnets, n_seqs, seq_len, head_keep, kv_max, d_head, n_heads, n_kv_heads,
                     *[_ptr(t.get(n)) for n in names], _plan_ptr(plan))
    a._keepalive = list(t.values()) + [plan]
    return a


def twist_attn_core_fwd(a: AttnCoreArgs):
    _check(lib().twist_attn_core_fwd(C.byref(a), _stream()), "twist_attn_core_fwd")


def twist_attn_core_bwd(a: AttnCoreArgs):
    _check(lib().twist_attn_core_bwd(C.byref(a), _stream()), "twist_attn_core_bwd")


def layernorm_args(dtype, n_subnets, tokens, d_model, eps, lr=0.0, opt: Optional[Optimizer] = None, **t) -> LayerNormArgs:
    """Marshals twist_layernorm_args (tensors by keyword: x, y, mean, rstd, gamma, beta, dy, dx, dx_residual,
    dgamma, dbeta, ws, m_gamma, v_gamma, m_beta, v_beta)."""
    names = ["x", "y", "mean", "rstd", "gamma", "beta", "dy", "dx", "dx_residual", "dgamma", "dbeta", "ws"]
    moments = ["m_gamma", "v_gamma", "m_beta", "v_beta"]
    unknown = set(t) - set(names) - set(moments)
    assert not unknown, unknown
    a = LayerNormArgs(dtype, n_subnets, tokens, d_model, eps, lr, *[_ptr(t.get(n)) for n in names],
                      _ws_bytes(t.get("ws")), opt if opt is not None else Optimizer(), *[_ptr(t.get(n)) for n in moments])
    a._keepalive = list(t.values())
    return a


def twist_layernorm_workspace_bytes(n_subnets: int, tokens: int, d_model: int) -> int:
    return lib().twist_layernorm_workspace_bytes(n_subnets, tokens, d_model)


def twist_layernorm_fwd(a: LayerNormArgs):
    _check(lib().twist_layernorm_fwd(C.byref(a), _stream()), "twist_layernorm_fwd")


def twist_layernorm_bwd(a: LayerNormArgs):
    _check(lib().twist_layernorm_bwd(C.byref(a), _stream()), "twist_layernorm_bwd")


def twist_mse_workspace_bytes(n_subnets: int) -> int:
    return lib().twist_mse_workspace_bytes(n_subnets)


def twist_fused_loss_workspace_bytes(n_subnets: int, tokens: int, width: int) -> int:
    return lib().twist_fused_loss_workspace_bytes(n_subnets, tokens, width)


def twist_mse_fwd_bwd(y, tgt, dy, loss, n_subnets, tokens, width, valid_cols, seg_begin, seg_width, dtype, ws):
    _check(lib().twist_mse_fwd_bwd(_ptr(y), _ptr(tgt), _ptr(dy), _ptr(loss), n_subnets, tokens, width,
                                   _ptr(valid_cols), seg_begin, seg_width, dtype, _ptr(ws),
                                   ws.numel() * ws.element_size(), _stream()),
           "twist_mse_fwd_bwd")


def twist_mse_fwd_bwd_noalloc(y, tgt, dy, loss, n_subnets, tokens, width, valid_cols, seg_begin, seg_width, dtype):
    """Loss and gradient like twist_mse_fwd_bwd, but with the library's built-in scratch: for callers
    that must not (or cannot) allocate device memory.  At most 32 subnets; calls must not overlap on
    the GPU; make the first call on a device outside stream capture."""
    _check(lib().twist_mse_fwd_bwd_noalloc(_ptr(y), _ptr(tgt), _ptr(dy), _ptr(loss), n_subnets, tokens, width,
                                           _ptr(valid_cols), seg_begin, seg_width, dtype, _stream()),
           "twist_mse_fwd_bwd_noalloc")
