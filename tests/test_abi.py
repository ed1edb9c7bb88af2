"""The C-ABI library loads and exports every symbol include/twist.h declares; host-side
argument checks return the documented status codes without touching a GPU."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "twist.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(twist_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2511_03983_b200 import binding as B
    names = _declared()
    assert len(names) >= 14
    h = B.lib()
    for n in names:
        assert hasattr(h, n), n
    assert sorted(B.EXPORTS) == names
    assert B.twist_abi_version() == 3
    # every entry point that takes arguments declares their C types: a device address passed without them
    # would be truncated to 32 bits
    for n in names:
        if n not in ("twist_abi_version", "twist_last_cuda_error"):
            assert getattr(h, n).argtypes is not None, n


def test_status_strings():
    from paper_2511_03983_b200 import binding as B
    h = B.lib()
    assert h.twist_strerror(0) == b"ok"
    for code in range(-8, 0):
        assert len(h.twist_strerror(code)) > 3


def test_host_side_argument_checks():
    from paper_2511_03983_b200 import binding as B
    h = B.lib()
    dummy = C.c_void_p(0x1000)   # never dereferenced: every call below fails validation first
    # sampler: null, shape, unsupported, infeasible (size bound of Sec. 3.1), bad common list
    f = h.twist_sample_masks
    assert f(1, 0, 0, 1, 0, 12, 4, 6, None, 0, 0, None, dummy, dummy, None) == B.ERR_NULL
    assert f(1, 0, 0, 1, 0, 0, 4, 6, None, 0, 0, dummy, dummy, dummy, None) == B.ERR_SHAPE
    assert f(1, 0, 0, 1, 0, 20000, 4, 6000, None, 0, 0, dummy, dummy, dummy, None) == B.ERR_UNSUPPORTED
    assert f(1, 0, 0, 1, 0, 12, 33, 6, None, 0, 0, dummy, dummy, dummy, None) == B.ERR_UNSUPPORTED
    assert f(1, 0, 0, 1, 0, 11008, 2, 2752, None, 0, B.MODE_COVER, dummy, dummy, dummy, None) == B.ERR_INFEASIBLE
    assert f(1, 0, 0, 1, 0, 12, 4, 13, None, 0, B.MODE_IID, dummy, dummy, dummy, None) == B.ERR_INFEASIBLE
    bad = (C.c_int32 * 2)(5, 3)
    assert f(1, 0, 0, 1, 0, 12, 4, 6, C.cast(bad, C.c_void_p), 2, 0, dummy, dummy, dummy, None) == B.ERR_BAD_INDEX
    # gather / aggregate
    assert h.twist_gather_subnets(None, 1, 2, 64, B.BF16, None) == B.ERR_NULL
    seg = B.GatherSegment(0x1000, 0x2000, None, 0x3000, None, 4, 4, 1, 16, 0, 256, 0)
    arr = (B.GatherSegment * 1)(seg)
    assert h.twist_gather_subnets(C.cast(arr, C.c_void_p), 1, 2, 63, B.BF16, None) == B.ERR_SHAPE     # row not 16 B
    assert h.twist_gather_subnets(C.cast(arr, C.c_void_p), 9, 2, 64, B.BF16, None) == B.ERR_SHAPE     # too many segments
    seg0 = B.GatherSegment(0x1000, 0x2000, None, 0x3000, None, 4, 4, 1, 0, 0, 256, 0)     # source block count missing
    arr0 = (B.GatherSegment * 1)(seg0)
    assert h.twist_gather_subnets(C.cast(arr0, C.c_void_p), 1, 2, 64, B.BF16, None) == B.ERR_SHAPE
    assert h.twist_aggregate(None, 1, 2, 64, B.BF16, 3, None) == B.ERR_NULL
    ag = (B.AggregateSegment * 1)(B.AggregateSegment(0x1000, None, 0x2000, 0x3000, 0x4000, 8, 1, 0, 256, 0, None, 0, 0))
    assert h.twist_aggregate(C.cast(ag, C.c_void_p), 1, 2, 64, B.BF16, 3, None) == B.ERR_SHAPE   # slice block count missing
    # the aggregate in two halves (subnets spread over GPUs)
    ok_seg = lambda **kw: (B.AggregateSegment * 1)(B.AggregateSegment(**dict(dict(
        dst=0x1000, dst_f32=0x5000, sub=0x2000, cover=0x3000, pos=0x4000, n_full=8, block_rows=1, dst_row_offset=0,
        sub_subnet_stride=256, sub_row_offset=0, central=None, central_subnet=0, n_keep=4), **kw)))
    part = lambda seg, n, s0: h.twist_aggregate_partial(C.cast(seg, C.c_void_p), 1, n, s0, 64, B.BF16, 0xFFFFFFFF, None)
    assert part(ok_seg(), 4, 30) == B.ERR_SHAPE                          # subnets 30..33: beyond the 32 of a cover mask
    assert part(ok_seg(dst_f32=None), 4, 0) == B.ERR_NULL                # the partial sums are fp32: they need a buffer
    assert part(ok_seg(central=0x6000), 4, 0) == B.ERR_UNSUPPORTED       # no in-place worker on a shard
    fin = lambda seg: h.twist_aggregate_finish(C.cast(seg, C.c_void_p), 1, 8, 64, B.BF16, 0xFFFFFFFF, None)
    assert fin(ok_seg()) == B.ERR_NULL                                   # the reduced sums (central) are missing
    assert fin(ok_seg(central=0x6004)) == B.ERR_SHAPE                    # ... or not 16-byte aligned
    assert h.twist_selftest_wait(0, None) == B.ERR_SHAPE and h.twist_selftest_wait(10 ** 9, None) == B.ERR_SHAPE
    # local steps
    a = B.FfnArgs(B.FFN_SWIGLU, B.BF16, 2, 128, 64, 100, 1.0, 0.0)       # f_sub not a multiple of 8
    assert h.twist_subnet_ffn_fwd(C.byref(a), None) == B.ERR_SHAPE
    a = B.FfnArgs(B.FFN_SWIGLU, B.BF16, 2, 128, 64, 128, 1.0, 0.0)       # all pointers NULL
    assert h.twist_subnet_ffn_fwd(C.byref(a), None) == B.ERR_NULL
    assert h.twist_subnet_ffn_bwd(C.byref(a), None) == B.ERR_NULL
    p = B.ProjArgs(7, B.BF16, 2, 128, 64, 64, 1.0, 0.0)
    assert h.twist_subnet_attn_proj_fwd(C.byref(p), None) == B.ERR_SHAPE
    # mse workspace
    assert B.twist_mse_workspace_bytes(4) == 4 * 1024 * 4
    assert h.twist_mse_fwd_bwd(dummy, dummy, dummy, dummy, 2, 8, 64, None, 0, 0, B.BF16, None, 0, None) == B.ERR_WORKSPACE
    # attention core
    assert h.twist_attn_core_fwd(None, None) == B.ERR_NULL
    ac = B.AttnCoreArgs(B.FP32, 2, 1, 64, 2, 2, 64, 0, 0, 0x1000, 0x2000, 0x3000)
    assert h.twist_attn_core_fwd(C.byref(ac), None) == B.ERR_UNSUPPORTED                 # bf16 only
    ac = B.AttnCoreArgs(B.BF16, 2, 1, 64, 2, 2, 48, 0, 0, 0x1000, 0x2000, 0x3000)
    assert h.twist_attn_core_fwd(C.byref(ac), None) == B.ERR_UNSUPPORTED                 # head size
    ac = B.AttnCoreArgs(B.BF16, 2, 1, 64, 4, 2, 64, 0, 0, 0x1000, 0x2000, 0x3000)
    assert h.twist_attn_core_fwd(C.byref(ac), None) == B.ERR_SHAPE                       # kv_max != head_keep without sharing
    ac = B.AttnCoreArgs(B.BF16, 2, 1, 64, 2, 2, 64, 0, 0, 0x1000, 0x2000, None)
    assert h.twist_attn_core_fwd(C.byref(ac), None) == B.ERR_NULL                        # lse missing
    # skip connections are not combinable with the fused loss
    a = B.FfnArgs(B.FFN_SWIGLU, B.BF16, 2, 128, 64, 96, 1.0, 0.0, 0x1000, 0x1000, 0x1000, None, None, 0x1000, 0x1000,
                  0x1000, 0x1000, None, None, None, None, 0x1000, 0x1000, 0x1000, 1 << 30, 0x1000, None)
    assert h.twist_subnet_ffn_fwd(C.byref(a), None) == B.ERR_UNSUPPORTED
    # the activation mask of Masked TwIST exists in the bf16 path only
    a = B.FfnArgs(B.FFN_SWIGLU, B.FP32, 2, 128, 64, 96, 1.0, 0.0, 0x1000, 0x1000, 0x1000, None, None, 0x1000, 0x1000, 0x1000)
    a.hidden_mask = 0x1000
    assert h.twist_subnet_ffn_fwd(C.byref(a), None) == B.ERR_UNSUPPORTED


def test_plan_object_validates_its_configuration_and_sizes_the_scratch():
    from paper_2511_03983_b200 import binding as B
    from paper_2511_03983_b200 import inputs as I
    h = B.lib()
    for cfg in (2, 3, 4, 5):
        w = I.PRESETS[cfg]
        plan = B.Plan(w)
        need = plan.workspace_bytes()
        widths = [w.d_model] + ([(w.n_heads + 2 * w.n_kv_heads) * w.d_head] if w.n_heads else [])
        assert need >= B.twist_mse_workspace_bytes(w.n_subnets)
        assert need >= max(B.twist_fused_loss_workspace_bytes(w.n_subnets, w.tokens, x) for x in widths)
        assert need >= B.twist_layernorm_workspace_bytes(w.n_subnets, w.tokens, w.d_model)
        assert plan.stats() == (0, 0, 0)
        plan.close()
    good = B.Config(C.sizeof(B.Config), 2, 64, 4, 2, 16, 256, B.FFN_SWIGLU, 4, 1, 128, 2, B.MODE_COVER, B.BF16, 128, 0, 7)
    out = C.c_void_p()
    assert h.twist_plan_create(C.byref(good), C.byref(out)) == 0 and out.value
    assert h.twist_plan_destroy(out) == 0
    assert h.twist_plan_create(None, C.byref(out)) == B.ERR_NULL and h.twist_plan_destroy(None) == B.ERR_NULL
    import copy
    for field, value, want in (("struct_size", 8, B.ERR_SHAPE), ("n_subnets", 33, B.ERR_UNSUPPORTED),
                               ("ffn_keep", 257, B.ERR_INFEASIBLE), ("head_keep", 5, B.ERR_INFEASIBLE),
                               ("n_kv_heads", 3, B.ERR_SHAPE), ("tokens", 0, B.ERR_SHAPE), ("ffn_block", 3, B.ERR_SHAPE)):
        bad = copy.copy(good)
        setattr(bad, field, value)
        out = C.c_void_p()
        assert h.twist_plan_create(C.byref(bad), C.byref(out)) == want, field
        assert not out.value


def test_misaligned_pointers_are_refused_before_any_launch():
    """The kernels use 16-byte (the activation mask: 8-byte) vector accesses; a pointer that breaks the rule must
    come back as a status, never reach the device."""
    from paper_2511_03983_b200 import binding as B
    h = B.lib()
    ok = 0x10000
    names = ["x", "w_gu", "w_down", "w_gu_master", "w_down_master", "pre", "hh", "y", "dy", "dpre", "dx", "dw_gu",
             "dw_down", "tgt", "loss_ws", "y_residual", "dx_residual", "m_gu", "v_gu", "m_down", "v_down"]
    for n in names:
        a = B.FfnArgs(B.FFN_SWIGLU, B.BF16, 2, 128, 64, 96, 1.0, 0.0)
        for m in names:
            setattr(a, m, ok)
        setattr(a, n, ok + (8 if n != "x" else 2))
        assert h.twist_subnet_ffn_fwd(C.byref(a), None) == B.ERR_SHAPE, n
        assert h.twist_subnet_ffn_bwd(C.byref(a), None) == B.ERR_SHAPE, n
    a = B.FfnArgs(B.FFN_SWIGLU, B.BF16, 2, 128, 64, 96, 1.0, 0.0)
    for m in names:
        setattr(a, m, ok)
    a.hidden_mask = ok + 4                                   # byte mask: 8-byte rule
    assert h.twist_subnet_ffn_fwd(C.byref(a), None) == B.ERR_SHAPE
    pnames = ["in_", "w", "w_master", "out", "d_out", "d_in", "dw", "tgt", "loss_ws", "out_residual", "d_in_residual",
              "m", "v"]
    for n in pnames:
        p = B.ProjArgs(B.PROJ_O, B.BF16, 2, 128, 64, 64, 1.0, 0.0)
        for m in pnames:
            setattr(p, m, ok)
        setattr(p, n, ok + 4)
        assert h.twist_subnet_attn_proj_fwd(C.byref(p), None) == B.ERR_SHAPE, n
        assert h.twist_subnet_attn_proj_bwd(C.byref(p), None) == B.ERR_SHAPE, n


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2511_03983_b200 import binding as B
    monkeypatch.setattr(B, "_lib_handle", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(FileNotFoundError):
        B.lib()
