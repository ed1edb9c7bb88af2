"""Parity of the CUDA path (through the C ABI) with the CPU oracle on the same seeded inputs.

Bars: masks, index data and gather output bit-exact; aggregate within 1e-6 relative per
element; bf16 GEMM outputs and gradients within 2e-2 relative Frobenius error of the fp64
oracle (which mirrors the bf16 rounding points of stored tensors); fp32 path within 1e-4.
"""
import math
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import twist_oracle as o
from paper_2511_03983_b200 import inputs as I
from fp32_mirror import aggregate_f32

pytestmark = pytest.mark.gpu

GEMM_TOL = 2e-2
AGG_TOL = 1e-6


@pytest.fixture(scope="module")
def B():
    from paper_2511_03983_b200 import binding
    binding.lib()
    return binding


def dev(x, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(x))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def host(t):
    return t.detach().float().cpu().numpy().astype(np.float64) if t.is_floating_point() else t.detach().cpu().numpy()


def rel_fro(got, want):
    return float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-300))


def block_rel_max(got, want, bs=32):
    """Largest error of any bs x bs block, relative to the root-mean-square block norm of the expected matrix:
    a wrong or missing epilogue box at a ragged edge moves the whole-matrix Frobenius ratio by little, but
    makes this one O(1)."""
    M, N = want.shape
    pm, pn = (-M) % bs, (-N) % bs
    e = np.pad((got - want) ** 2, ((0, pm), (0, pn)))
    w = np.pad(want ** 2, ((0, pm), (0, pn)))
    eb = e.reshape((M + pm) // bs, bs, (N + pn) // bs, bs).sum(axis=(1, 3))
    wb = w.reshape((M + pm) // bs, bs, (N + pn) // bs, bs).sum(axis=(1, 3))
    full_blocks = max(1.0, (M * N) / (bs * bs))
    return float(np.sqrt(eb.max() / max(wb.sum() / full_blocks, 1e-300)))


def close(got, want, tol):
    """The Frobenius bar on the whole matrix and, so that no single tile can hide in it, 4x the bar on every
    32 x 32 block (bf16 rounding of one block scatters around the mean; 4x covers the spread of a small sample)."""
    return rel_fro(got, want) < tol and block_rel_max(got, want) < 4 * tol


def check_status(B):
    assert B.twist_device_status() == 0


# --------------------------------------------------------------------------------------------- sampler

def _gpu_masks(B, seed, rnd, layer_begin, n_layers, kind, n_full, S, n_sub, common, mode):
    idx = torch.full((n_layers, S, n_sub), -7, dtype=torch.int32, device="cuda")
    cover = torch.full((n_layers, n_full), -7, dtype=torch.int32, device="cuda")
    pos = torch.full((n_layers, S, n_full), -7, dtype=torch.int32, device="cuda")
    B.twist_sample_masks(seed, rnd, layer_begin, n_layers, kind, n_full, S, n_sub, common, mode, idx, cover, pos)
    torch.cuda.synchronize()
    return idx.cpu().numpy(), cover.cpu().numpy().view(np.uint32), pos.cpu().numpy()


@pytest.mark.parametrize("n_full,S,n_sub,common,mode,kind,n_layers", [
    (256, 2, 128, [], 0, 0, 1),            # config 1
    (3072, 4, 1536, [], 0, 0, 12),         # config 2 FFN
    (12, 4, 6, [], 0, 1, 12),              # config 2 heads
    (5632, 4, 2816, [], 0, 0, 3),          # config 3 FFN
    (32, 4, 16, [], 0, 1, 22),             # config 3 heads
    (11008, 8, 2752, [], 0, 0, 3),         # config 4 FFN
    (32, 8, 8, [], 0, 1, 32),              # config 4 heads
    (11008, 2, 2752, [], 1, 0, 2),         # config 5 cells (IID)
    (11008, 16, 8256, [], 1, 0, 2),
    (11008, 4, 5504, [], 1, 0, 1),
    (100, 7, 16, [3], 0, 0, 2), (12, 3, 6, [0, 7], 0, 1, 2), (40, 3, 17, [1, 2, 39], 1, 0, 2),   # common blocks
    (16384, 2, 8192, [], 0, 0, 1),         # maximum block count
    (7, 1, 7, [], 0, 0, 1), (1, 1, 1, [], 0, 1, 1), (33, 32, 2, [], 0, 0, 1),   # degenerate
])
def test_masks_bit_exact(B, n_full, S, n_sub, common, mode, kind, n_layers):
    seed, rnd, l0 = 3000 + n_full, 2, 5
    idx, cover, pos = _gpu_masks(B, seed, rnd, l0, n_layers, kind, n_full, S, n_sub, common, mode)
    for l in range(n_layers):
        A = o.sample_blueprint(n_full, S, n_sub, common, seed, rnd, l0 + l, kind, mode)
        assert np.array_equal(idx[l], A), (l,)
        c, _, p = o.cover_and_pos(A, n_full)
        assert np.array_equal(cover[l], c)
        assert np.array_equal(pos[l], p)
    check_status(B)


def test_kv_groups_bit_exact(B):
    H, Hkv, S, keep, L, dh = 32, 4, 4, 3, 6, 64       # few kept heads so that some groups are dropped
    idx, _, _ = _gpu_masks(B, 17, 0, 0, L, 1, H, S, keep, [], I.MODE_IID)
    t = lambda *s: torch.full(s, -7, dtype=torch.int32, device="cuda")
    kv_idx, kv_count, kv_cols, kv_cover, kv_pos = t(L, S, Hkv), t(L, S), t(L, S), t(L, Hkv), t(L, S, Hkv)
    B.twist_kv_groups(dev(idx), L, S, keep, H, Hkv, dh, kv_idx, kv_count, kv_cols, kv_cover, kv_pos)
    torch.cuda.synchronize()
    saw_ragged = False
    for l in range(L):
        want_idx, want_count = o.kv_groups(idx[l], H, Hkv)
        assert np.array_equal(kv_idx[l].cpu().numpy(), want_idx)
        assert np.array_equal(kv_count[l].cpu().numpy(), want_count)
        assert np.array_equal(kv_cols[l].cpu().numpy(), want_count * dh)
        c, _, p = o.cover_and_pos(want_idx, Hkv, counts=want_count)
        assert np.array_equal(kv_cover[l].cpu().numpy().view(np.uint32), c)
        assert np.array_equal(kv_pos[l].cpu().numpy(), p)
        saw_ragged |= bool(np.any(want_count < Hkv))
    assert saw_ragged


# --------------------------------------------------------------------------------------------- gather / aggregate

@pytest.mark.parametrize("dtype,d,n_full,S,n_sub,br", [
    (I.DTYPE_BF16, 4096, 512, 8, 128, 1), (I.DTYPE_BF16, 328, 300, 3, 101, 1), (I.DTYPE_BF16, 768, 12, 4, 6, 64),
    (I.DTYPE_FP32, 64, 256, 2, 128, 1), (I.DTYPE_FP32, 100, 37, 5, 9, 3), (I.DTYPE_BF16, 8, 5, 2, 3, 1),
    (I.DTYPE_BF16, 520, 200, 16, 150, 1),      # S = 16, keep 3/4: rows averaged over up to 16 subnets
    (I.DTYPE_BF16, 1024, 64, 32, 40, 2),       # the maximum subnet count
])
def test_gather_bit_exact_and_aggregate_parity(B, dtype, d, n_full, S, n_sub, br):
    td = torch.bfloat16 if dtype == I.DTYPE_BF16 else torch.float32
    W = I.normal(11, 1, (n_full * br + 5, d), 0.02, dtype)          # 5 extra rows: src_row_offset = 2
    A = o.sample_blueprint(n_full, S, n_sub, [], 5, 0, 0, 0, o.MODE_IID)
    cover, count, pos = o.cover_and_pos(A, n_full)
    Wd = dev(W, td)
    rows = n_sub * br
    pad_rows = 3                                                     # slice rows before the segment
    sub = torch.zeros(S, pad_rows + rows, d, dtype=td, device="cuda")
    master = torch.zeros(S, pad_rows + rows, d, dtype=torch.float32, device="cuda") if dtype == I.DTYPE_BF16 else None
    seg = B.gather_segment(Wd, sub, master, dev(A), None, n_sub, n_sub, br, 2, (pad_rows + rows) * d, pad_rows, n_full)
    B.twist_gather_subnets([seg], S, d, dtype)
    torch.cuda.synchronize()
    for s in range(S):
        want = o.gather_rows(W, A[s], br, row_offset=2)
        got = sub[s, pad_rows:].float().cpu().numpy()
        assert np.array_equal(got.view(np.uint32), want.astype(np.float32).view(np.uint32))
        assert torch.all(sub[s, :pad_rows] == 0)
        if master is not None:
            assert np.array_equal(master[s, pad_rows:].cpu().numpy().view(np.uint32), want.astype(np.float32).view(np.uint32))

    # "train": perturb the fp32 masters / slices with seeded noise, then aggregate
    noise = I.normal(12, 2, (S, pad_rows + rows, d), 0.01, I.DTYPE_FP32)
    trained = (master if master is not None else sub).float() + dev(noise)
    trained = trained.contiguous()
    saw_counts = set()
    for live in (0xFFFFFFFF, 0b101 & ((1 << S) - 1)):
        full = Wd.clone()
        full_f32 = torch.full((n_full * br + 5, d), 123.0, dtype=torch.float32, device="cuda") if dtype == I.DTYPE_BF16 else None
        seg = B.aggregate_segment(full, full_f32, trained, dev(cover.view(np.int32)), dev(pos), n_full, br, 2,
                                  (pad_rows + rows) * d, pad_rows, n_sub)
        B.twist_aggregate([seg], S, d, dtype, live)
        torch.cuda.synchronize()
        tr = trained.cpu().numpy().astype(np.float64)
        want = o.aggregate(W.astype(np.float64), [tr[s, pad_rows:] for s in range(S)], A, br, live_mask=live, row_offset=2)
        live_cnt = np.array([bin(int(c) & live).count("1") for c in cover])
        held_rows = np.repeat(live_cnt > 0, br)
        res = (full_f32 if full_f32 is not None else full).cpu().numpy().astype(np.float64)[2:2 + n_full * br]
        w_rows = want[2:2 + n_full * br]
        # relative to the mean magnitude of the averaged values (an fp32 sum that cancels cannot be
        # relatively exact in its own, much smaller, magnitude)
        mag = o.aggregate(np.abs(W.astype(np.float64)), [np.abs(tr[s, pad_rows:]) for s in range(S)], A, br,
                          live_mask=live, row_offset=2)[2:2 + n_full * br]
        err = np.abs(res[held_rows] - w_rows[held_rows]) / np.maximum(mag[held_rows], 1e-30)
        assert err.max() <= max(AGG_TOL, (live_cnt.max() + 1) * 2.0 ** -24), err.max()
        # and bit for bit the fp32 evaluation in the fixed order: running sum in ascending subnet index, one IEEE
        # division by the count (the kernel forms the quotient from a corrected reciprocal product)
        tr32 = trained.cpu().numpy()
        mirror = aggregate_f32(W, [tr32[s, pad_rows:] for s in range(S)], A, br, live_mask=live, row_offset=2)
        got32 = (full_f32 if full_f32 is not None else full).cpu().numpy()[2:2 + n_full * br]
        assert np.array_equal(got32[held_rows].view(np.uint32), mirror[2:2 + n_full * br][held_rows].view(np.uint32))
        saw_counts |= set(int(c) for c in live_cnt)
        if full_f32 is not None:      # untouched rows keep their values in both outputs; bf16 shadow = RNE(fp32 result)
            assert torch.all(full_f32[2:2 + n_full * br][torch.from_numpy(~held_rows).cuda()] == 123.0)
            assert torch.equal(full[2:2 + n_full * br][torch.from_numpy(held_rows).cuda()],
                               full_f32[2:2 + n_full * br][torch.from_numpy(held_rows).cuda()].to(torch.bfloat16))
        assert torch.equal(full[2:2 + n_full * br][torch.from_numpy(~held_rows).cuda()],
                           Wd[2:2 + n_full * br][torch.from_numpy(~held_rows).cuda()])
        assert torch.equal(full[:2], Wd[:2]) and torch.equal(full[2 + n_full * br:], Wd[2 + n_full * br:])
    assert max(saw_counts) >= min(S, 2)
    check_status(B)


def test_gather_ragged_counts_zero_fill(B):
    d, S, Hkv, dh = 64, 3, 4, 8
    W = I.normal(13, 1, (Hkv * dh, d), 0.02, I.DTYPE_BF16)
    kv_idx = np.array([[0, 2, -1, -1], [1, -1, -1, -1], [0, 1, 2, 3]], dtype=np.int32)
    kv_count = np.array([2, 1, 4], dtype=np.int32)
    sub = torch.full((S, Hkv * dh, d), 9.0, dtype=torch.bfloat16, device="cuda")
    master = torch.full((S, Hkv * dh, d), 9.0, dtype=torch.float32, device="cuda")
    seg = B.gather_segment(dev(W, torch.bfloat16), sub, master, dev(kv_idx), dev(kv_count), Hkv, Hkv, dh, 0, Hkv * dh * d, 0,
                           Hkv)
    B.twist_gather_subnets([seg], S, d, I.DTYPE_BF16)
    torch.cuda.synchronize()
    for s in range(S):
        n = kv_count[s] * dh
        want = o.gather_rows(W, kv_idx[s][: kv_count[s]], dh)
        assert np.array_equal(sub[s, :n].float().cpu().numpy(), want)
        assert torch.all(sub[s, n:] == 0) and torch.all(master[s, n:] == 0)


# --------------------------------------------------------------------------------------------- MSE glue

@pytest.mark.parametrize("dtype", [I.DTYPE_BF16, I.DTYPE_FP32])
def test_mse_parity(B, dtype):
    S, T, width = 3, 77, 72
    td = torch.bfloat16 if dtype == I.DTYPE_BF16 else torch.float32
    Y = I.normal(21, 1, (S, T, width), 1.0, dtype)
    Tg = I.normal(21, 2, (S, T, width), 1.0, dtype)
    ws = torch.empty(B.twist_mse_workspace_bytes(S), dtype=torch.uint8, device="cuda")
    for valid, seg_begin, seg_width in [(None, 0, 0), (np.array([8, 16, 24], dtype=np.int32), 24, 24),
                                        (np.array([72, 40, 8], dtype=np.int32), 0, 72)]:
        dy = torch.empty(S, T, width, dtype=td, device="cuda")
        loss = torch.empty(S, dtype=torch.float32, device="cuda")
        B.twist_mse_fwd_bwd(dev(Y, td), dev(Tg, td), dy, loss, S, T, width, None if valid is None else dev(valid),
                            seg_begin, seg_width, dtype, ws)
        torch.cuda.synchronize()
        for s in range(S):
            if valid is None:
                cols = np.arange(width)
            else:
                cols = np.array([c for c in range(width) if c < seg_begin or (c - seg_begin) % seg_width < valid[s]])
            want_loss, want_dy = o.mse(Y[s][:, cols].astype(np.float64), Tg[s][:, cols].astype(np.float64),
                                       lowp=dtype == I.DTYPE_BF16)
            got = host(dy[s])
            assert abs(loss[s].item() - want_loss) <= 1e-5 * want_loss
            assert rel_fro(got[:, cols], want_dy) < (1e-2 if dtype == I.DTYPE_BF16 else 1e-6)
            other = np.setdiff1d(np.arange(width), cols)
            assert np.all(got[:, other] == 0)


# --------------------------------------------------------------------------------------------- FFN / projections

def _ffn_case(B, kind, dtype, S, T, d, f, alpha, lr, seed, mask_keep=0):
    lowp = dtype == I.DTYPE_BF16
    td = torch.bfloat16 if lowp else torch.float32
    g = 2 if kind == I.FFN_SWIGLU else 1
    X = I.normal(seed, 1, (S, T, d), 1.0, dtype)
    Wgu = I.normal(seed, 2, (S, g * f, d), 0.05, dtype)
    Wd = I.normal(seed, 3, (S, f, d), 0.05, dtype)
    dY = I.normal(seed, 4, (S, T, d), 1e-3, dtype)
    t = lambda *s: torch.zeros(*s, dtype=td, device="cuda")
    w_gu, w_down = dev(Wgu, td), dev(Wd, td)
    m_gu, m_down = (w_gu.float(), w_down.float()) if lowp else (None, None)
    pre, hh, y, dpre, dx = t(S, T, g * f), t(S, T, f), t(S, T, d), t(S, T, g * f), t(S, T, d)
    dw_gu = torch.zeros(S, g * f, d, dtype=torch.float32, device="cuda")
    dw_down = torch.zeros(S, f, d, dtype=torch.float32, device="cuda")
    masks, extra = [None] * S, {}
    if mask_keep:          # Masked TwIST (Sec. 4.1): worker s sees only its active neurons of the full-width model
        rng = np.random.default_rng(seed)
        masks = [np.zeros(f, dtype=np.uint8) for _ in range(S)]
        for s in range(S):
            masks[s][rng.choice(f, mask_keep, replace=False)] = 1
        extra = dict(hidden_mask=dev(np.stack(masks)))
    a = B.ffn_args(kind, dtype, S, T, d, f, alpha, lr, x=dev(X, td), w_gu=w_gu, w_down=w_down, w_gu_master=m_gu,
                   w_down_master=m_down, pre=pre, hh=hh, y=y, dy=dev(dY, td), dpre=dpre, dx=dx, dw_gu=dw_gu,
                   dw_down=dw_down, **extra)
    B.twist_subnet_ffn_fwd(a)
    B.twist_subnet_ffn_bwd(a)
    torch.cuda.synchronize()
    check_status(B)
    tol = GEMM_TOL if lowp else 1e-4
    for s in range(S):
        Wg_s = Wgu[s, :f].astype(np.float64) if g == 2 else None
        Wu_s = Wgu[s, (g - 1) * f:].astype(np.float64)
        Wd_s = Wd[s].astype(np.float64)
        Xs, dYs = X[s].astype(np.float64), dY[s].astype(np.float64)
        Yw, saved = o.ffn_fwd(Xs, Wu_s, Wg_s, Wd_s, kind, alpha, lowp, hidden_mask=masks[s])
        dXw, dWu, dWg, dWd = o.ffn_bwd(dYs, Xs, saved, Wu_s, Wg_s, Wd_s, kind, alpha, lowp, hidden_mask=masks[s])
        if mask_keep:      # masked-out neurons: zero activation, exactly zero gradient rows, weights untouched
            off = np.flatnonzero(masks[s] == 0)
            rows = np.concatenate([off, off + f]) if g == 2 else off
            assert np.all(host(hh[s])[:, off] == 0)
            assert np.all(host(dw_gu[s])[rows] == 0) and np.all(host(dw_down[s])[off] == 0)
            assert np.array_equal(host(m_gu[s])[rows], Wgu[s][rows]) and np.array_equal(host(m_down[s])[off], Wd[s][off])
        pre_w = np.concatenate([saved["G"], saved["U"]], axis=1) if g == 2 else saved["U"]
        dWgu = np.concatenate([dWg, dWu], axis=0) if g == 2 else dWu
        assert close(host(pre[s]), pre_w, tol), ("pre", s)
        assert close(host(hh[s]), saved["Hh"], tol), ("hh", s)
        assert close(host(y[s]), Yw, tol), ("y", s)
        assert close(host(dx[s]), dXw, tol), ("dx", s)
        assert close(host(dw_gu[s]), dWgu, tol), ("dw_gu", s)
        assert close(host(dw_down[s]), dWd, tol), ("dw_down", s)
        if lr != 0:
            new_gu, new_gu_c = o.sgd(Wgu[s].astype(np.float64), dWgu, lr, lowp)
            new_d, new_d_c = o.sgd(Wd_s, dWd, lr, lowp)
            upd = host(m_gu[s] if lowp else w_gu[s]) - Wgu[s]
            assert close(upd, new_gu - Wgu[s], tol), ("sgd gu", s)
            upd = host(m_down[s] if lowp else w_down[s]) - Wd[s]
            assert close(upd, new_d - Wd[s], tol), ("sgd down", s)
            if lowp:   # compute copy is the nearest-even rounding of the device's own master
                assert torch.equal(w_gu[s], m_gu[s].to(torch.bfloat16))
                assert torch.equal(w_down[s], m_down[s].to(torch.bfloat16))


@pytest.mark.parametrize("kind", [I.FFN_RELU, I.FFN_GELU, I.FFN_SWIGLU])
def test_ffn_fp32_parity(B, kind):
    _ffn_case(B, kind, I.DTYPE_FP32, S=2, T=37, d=24, f=20, alpha=1.5, lr=0.5, seed=31)


@pytest.mark.parametrize("kind,S,T,d,f", [
    (I.FFN_SWIGLU, 2, 256, 256, 256),      # whole tiles
    (I.FFN_SWIGLU, 3, 200, 328, 344),      # ragged M, K and N tails, several tiles
    (I.FFN_GELU, 2, 333, 192, 520),
    (I.FFN_RELU, 2, 128, 64, 128),         # config-1 shape in bf16
    (I.FFN_SWIGLU, 1, 520, 1032, 688),     # > 4 k-blocks: the ring wraps; 3 n-tiles in dX
])
def test_ffn_bf16_parity(B, kind, S, T, d, f):
    _ffn_case(B, kind, I.DTYPE_BF16, S, T, d, f, alpha=2.0, lr=0.5, seed=41)


@pytest.mark.parametrize("kind,S,T,d,f,keep", [
    (I.FFN_SWIGLU, 2, 300, 264, 392, 96),      # ragged tiles, a quarter of the neurons active
    (I.FFN_GELU, 3, 130, 136, 264, 128),
    (I.FFN_RELU, 1, 257, 72, 520, 8),
])
def test_masked_twist_ffn_parity(B, kind, S, T, d, f, keep):
    """Masked TwIST (Sec. 4.1): the full-width model with an activation mask per worker, against the oracle's
    masked model; the scale is the one of a subnet with `keep` of f neurons (Sec. 3.4)."""
    _ffn_case(B, kind, I.DTYPE_BF16, S, T, d, f, o.act_scale(f, keep), 0.05, 33, mask_keep=keep)


def test_masked_twist_equals_the_gathered_subnet_on_the_gpu(B):
    """The same subnet once as a gathered dense slice and once as the masked full-width model: outputs and input
    gradients agree to rounding (the contraction merely runs over more, zeroed, terms)."""
    kind, T, d, F, keep = I.FFN_SWIGLU, 260, 136, 256, 64
    bf = torch.bfloat16
    rng = np.random.default_rng(3)
    kept = np.sort(rng.choice(F, keep, replace=False))
    X = I.normal(44, 1, (1, T, d), 1.0, I.DTYPE_BF16)
    Wgu = I.normal(44, 2, (1, 2 * F, d), 0.05, I.DTYPE_BF16)
    Wd = I.normal(44, 3, (1, F, d), 0.05, I.DTYPE_BF16)
    dY = I.normal(44, 4, (1, T, d), 1e-3, I.DTYPE_BF16)
    alpha = o.act_scale(F, keep)
    outs = []
    for masked in (True, False):
        f = F if masked else keep
        rows = np.arange(2 * F) if masked else np.concatenate([kept, kept + F])
        w_gu, w_down = dev(Wgu[:, rows], bf), dev(Wd[:, np.arange(F) if masked else kept], bf)
        t = lambda *s: torch.zeros(*s, dtype=bf, device="cuda")
        pre, hh, y, dpre, dx = t(1, T, 2 * f), t(1, T, f), t(1, T, d), t(1, T, 2 * f), t(1, T, d)
        extra = {}
        if masked:
            m = np.zeros((1, F), dtype=np.uint8)
            m[0, kept] = 1
            extra = dict(hidden_mask=dev(m))
        a = B.ffn_args(kind, I.DTYPE_BF16, 1, T, d, f, alpha, 0.0, x=dev(X, bf), w_gu=w_gu, w_down=w_down, pre=pre, hh=hh,
                       y=y, dy=dev(dY, bf), dpre=dpre, dx=dx, **extra)
        B.twist_subnet_ffn_fwd(a)
        B.twist_subnet_ffn_bwd(a)
        torch.cuda.synchronize()
        check_status(B)
        outs.append((host(y[0]), host(dx[0]), host(hh[0])[:, kept] if masked else host(hh[0])))
    (ym, dxm, hm), (yg, dxg, hg) = outs
    assert np.array_equal(hm, hg)                    # the kept activations are the same numbers
    assert rel_fro(ym, yg) < 4e-3 and rel_fro(dxm, dxg) < 4e-3     # one bf16 rounding apart at most


@pytest.mark.parametrize("dtype,S,T,d,n", [(I.DTYPE_FP32, 2, 33, 24, 16), (I.DTYPE_BF16, 2, 200, 328, 200),
                                           (I.DTYPE_BF16, 3, 384, 768, 1152), (I.DTYPE_BF16, 1, 130, 64, 72)])
def test_proj_parity(B, dtype, S, T, d, n):
    lowp = dtype == I.DTYPE_BF16
    td = torch.bfloat16 if lowp else torch.float32
    tol = GEMM_TOL if lowp else 1e-4
    lr = 0.5
    for which, alpha in ((B.PROJ_QKV, 1.0), (B.PROJ_O, 1.7)):
        w_in, w_out = (d, n) if which == B.PROJ_QKV else (n, d)
        Xin = I.normal(51, 1 + which, (S, T, w_in), 1.0, dtype)
        W = I.normal(51, 3 + which, (S, n, d), 0.05, dtype)
        dO = I.normal(51, 5 + which, (S, T, w_out), 1e-3, dtype)
        w = dev(W, td)
        m = w.float() if lowp else None
        out = torch.zeros(S, T, w_out, dtype=td, device="cuda")
        d_in = torch.zeros(S, T, w_in, dtype=td, device="cuda")
        dw = torch.zeros(S, n, d, dtype=torch.float32, device="cuda")
        a = B.proj_args(which, dtype, S, T, d, n, alpha, lr, in_=dev(Xin, td), w=w, w_master=m, out=out,
                        d_out=dev(dO, td), d_in=d_in, dw=dw)
        B.twist_subnet_attn_proj_fwd(a)
        B.twist_subnet_attn_proj_bwd(a)
        torch.cuda.synchronize()
        check_status(B)
        for s in range(S):
            Xs, Ws, dOs = (v[s].astype(np.float64) for v in (Xin, W, dO))
            if which == B.PROJ_QKV:
                want_out = o.qkv_fwd(Xs, Ws, lowp)
                want_din, want_dw = o.qkv_bwd(dOs, Xs, Ws, lowp)
            else:
                want_out = o.o_fwd(Xs, Ws, alpha, lowp)
                want_din, want_dw = o.o_bwd(dOs, Xs, Ws, alpha, lowp)
            assert close(host(out[s]), want_out, tol), (which, "out")
            assert close(host(d_in[s]), want_din, tol), (which, "d_in")
            assert close(host(dw[s]), want_dw, tol), (which, "dw")
            upd = host(m[s] if lowp else w[s]) - W[s]
            assert close(upd, -lr * want_dw, tol), (which, "sgd")


# --------------------------------------------------------------------------------------------- fused loss

@pytest.mark.parametrize("S,T,d,f", [(2, 200, 328, 344), (3, 520, 264, 136)])
def test_fused_loss_equals_standalone_loss_ffn(B, S, T, d, f):
    """The loss evaluated in the forward call's output kernel gives the gradient twist_mse_fwd_bwd gives on
    the stored output, bit for bit, and the same loss up to summation order; both match the oracle."""
    td, dtype, kind, alpha = torch.bfloat16, I.DTYPE_BF16, I.FFN_SWIGLU, 2.0
    X = I.normal(61, 1, (S, T, d), 1.0, dtype)
    Wgu = I.normal(61, 2, (S, 2 * f, d), 0.05, dtype)
    Wd = I.normal(61, 3, (S, f, d), 0.05, dtype)
    Tg = I.normal(61, 4, (S, T, d), 1.0, dtype)
    t = lambda *s: torch.zeros(*s, dtype=td, device="cuda")
    pre, hh, y, dy_a, dy_b = t(S, T, 2 * f), t(S, T, f), t(S, T, d), t(S, T, d), t(S, T, d)
    loss_a = torch.zeros(S, dtype=torch.float32, device="cuda")
    loss_b = torch.zeros(S, dtype=torch.float32, device="cuda")
    ws = torch.empty(B.twist_fused_loss_workspace_bytes(S, T, d), dtype=torch.uint8, device="cuda")
    common = dict(x=dev(X, td), w_gu=dev(Wgu, td), w_down=dev(Wd, td), pre=pre, hh=hh)
    B.twist_subnet_ffn_fwd(B.ffn_args(kind, dtype, S, T, d, f, alpha, 0.0, y=y, **common))
    B.twist_mse_fwd_bwd(y, dev(Tg, td), dy_a, loss_a, S, T, d, None, 0, 0, dtype, ws)
    y2 = t(S, T, d)
    B.twist_subnet_ffn_fwd(B.ffn_args(kind, dtype, S, T, d, f, alpha, 0.0, y=y2, dy=dy_b, tgt=dev(Tg, td), loss=loss_b,
                                      loss_ws=ws, **common))
    dy_c = t(S, T, d)     # the output need not be stored
    B.twist_subnet_ffn_fwd(B.ffn_args(kind, dtype, S, T, d, f, alpha, 0.0, y=None, dy=dy_c, tgt=dev(Tg, td),
                                      loss=loss_b, loss_ws=ws, **common))
    torch.cuda.synchronize()
    check_status(B)
    assert torch.equal(y, y2) and torch.equal(dy_a, dy_b) and torch.equal(dy_a, dy_c)
    assert torch.allclose(loss_a, loss_b, rtol=1e-5, atol=0)
    for s in range(S):
        Yw, _ = o.ffn_fwd(X[s].astype(np.float64), Wgu[s, f:].astype(np.float64), Wgu[s, :f].astype(np.float64),
                          Wd[s].astype(np.float64), kind, alpha, True)
        want_loss, want_dy = o.mse(Yw, Tg[s].astype(np.float64), True)
        assert abs(loss_b[s].item() - want_loss) <= 2e-2 * want_loss
        assert rel_fro(host(dy_b[s]), want_dy) < GEMM_TOL


def test_fused_loss_equals_standalone_loss_proj_with_column_mask(B):
    td, dtype = torch.bfloat16, I.DTYPE_BF16
    S, T, d = 3, 300, 200
    a_sub, kvw = 64, 48                   # [Q 64 | K 48 | V 48], valid K/V columns per subnet below
    n = a_sub + 2 * kvw
    valid = dev(np.array([48, 16, 32], dtype=np.int32))
    Xin = I.normal(71, 1, (S, T, d), 1.0, dtype)
    W = I.normal(71, 2, (S, n, d), 0.05, dtype)
    Tg = I.normal(71, 3, (S, T, n), 1.0, dtype)
    out = torch.zeros(S, T, n, dtype=td, device="cuda")
    d_a, d_b = torch.zeros_like(out), torch.zeros_like(out)
    loss_a = torch.zeros(S, dtype=torch.float32, device="cuda")
    loss_b = torch.zeros(S, dtype=torch.float32, device="cuda")
    ws = torch.empty(B.twist_fused_loss_workspace_bytes(S, T, max(n, d)), dtype=torch.uint8, device="cuda")
    for which, width, w_in, mask in ((B.PROJ_QKV, n, d, True), (B.PROJ_O, d, n, False)):
        xin = dev(Xin, td) if which == B.PROJ_QKV else dev(Tg, td)       # O projection: input of width n
        tg = dev(Tg, td) if which == B.PROJ_QKV else dev(Xin, td)
        o1 = torch.zeros(S, T, width, dtype=td, device="cuda")
        g1, g2 = torch.zeros_like(o1), torch.zeros_like(o1)
        kw = dict(valid_cols=valid, seg_begin=a_sub, seg_width=kvw) if mask else {}
        B.twist_subnet_attn_proj_fwd(B.proj_args(which, dtype, S, T, d, n, 1.3, 0.0, in_=xin, w=dev(W, td), out=o1))
        B.twist_mse_fwd_bwd(o1, tg, g1, loss_a, S, T, width, valid if mask else None, a_sub if mask else 0,
                            kvw if mask else 0, dtype, ws)
        torch.cuda.synchronize()
        B.twist_subnet_attn_proj_fwd(B.proj_args(which, dtype, S, T, d, n, 1.3, 0.0, in_=xin, w=dev(W, td), out=None,
                                                 d_out=g2, tgt=tg, loss=loss_b, loss_ws=ws, **kw))
        torch.cuda.synchronize()
        check_status(B)
        assert torch.equal(g1, g2), which
        assert torch.allclose(loss_a, loss_b, rtol=1e-5, atol=0), which


# --------------------------------------------------------------------------------------------- whole rounds

def _load_full(eng, w):
    td = torch.bfloat16 if w.dtype == I.DTYPE_BF16 else torch.float32
    mats = {"gate": I.MAT_GATE, "up": I.MAT_UP, "down": I.MAT_DOWN, "qkv": I.MAT_QKV, "o": I.MAT_O}
    full_np = []
    for l in range(w.n_layers):
        layer = {}
        for m in eng.full:
            layer[m] = I.weight(w, l, mats[m])
            eng.full[m][l].copy_(dev(layer[m], td))
        full_np.append(layer)
    return full_np


def _load_batches(eng, w, rnd):
    """Seeded batches of round rnd on the device and, for the oracle, on the host: store[(kind, k)] for the
    partitioned layers' widths, store[(kind, k, width)] for every width (shared layers have their own QKV / A widths)."""
    td = torch.bfloat16 if w.dtype == I.DTYPE_BF16 else torch.float32
    S = w.n_subnets
    eng.X, eng.Td = [], []
    store = {}
    for k in range(w.local_steps):
        for kind, dst in ((I.BATCH_X, eng.X), (I.BATCH_TGT_D, eng.Td)):
            arr = np.stack([I.batch(w, kind, rnd, s, k, w.d_model) for s in range(S)])
            store[(kind, k)] = store[(kind, k, w.d_model)] = arr
            dst.append(dev(arr, td))
    if eng.has_attn:
        for gk, gm in eng.geo.items():
            eng.batches[gk] = {"Tq": [], "A": []}
            for k in range(w.local_steps):
                for kind, width, name in ((I.BATCH_TGT_QKV, gm.nq, "Tq"), (I.BATCH_A, gm.a_sub, "A")):
                    arr = np.stack([I.batch(w, kind, rnd, s, k, width) for s in range(S)])
                    store[(kind, k, width)] = arr
                    if gk == "part":
                        store[(kind, k)] = arr
                    eng.batches[gk][name].append(dev(arr, td))
    if eng.has_attn and hasattr(eng, "Tq_c"):        # Hybrid TwIST: the central worker's full-width batches
        eng.Tq_c, eng.A_c = [], []
        for k in range(w.local_steps):
            for kind, width, dst in ((I.BATCH_TGT_QKV, eng.c_nq, eng.Tq_c), (I.BATCH_A, eng.c_a, eng.A_c)):
                arr = I.batch(w, kind + 4, rnd, 0, k, width)[None]
                store[("central", kind, k)] = arr
                dst.append(dev(arr, td))
    return store


def _run_round_and_compare(B, w, rnd=0, tol_dw=5e-2, engine_cls=None, **engine_kw):
    from paper_2511_03983_b200.engine import RoundEngine
    lowp = w.dtype == I.DTYPE_BF16
    eng = RoundEngine(w, keep_f32_full=True, **engine_kw) if engine_cls is None else engine_cls(w, **engine_kw)
    full_np = _load_full(eng, w)
    if eng.full_f32 is not None:       # the fp32 full model starts as the exact widening of the bf16 one
        for m in eng.full:
            eng.full_f32[m].copy_(eng.full[m].float())
    store = _load_batches(eng, w, rnd)
    before = {m: v.clone() for m, v in eng.full.items()}
    eng.run_round(rnd)
    torch.cuda.synchronize()
    check_status(B)
    ragged = eng.has_attn and w.n_kv_heads != w.n_heads
    w = getattr(eng, "true_w", w)
    for l in range(w.n_layers):
        bp = o.layer_blueprints(w, rnd, l)

        gm = eng.geo[eng.kind_of(l)]
        masked_attn = eng.has_attn and hasattr(eng, "true_w")      # full-width batches: the oracle sees the held columns

        def held_cols(bp, s, qkv):
            dh, H, Hkv = w.d_head, w.n_heads, w.n_kv_heads
            q = np.concatenate([np.arange(h * dh, (h + 1) * dh) for h in bp["head"][s]])
            if not qkv:
                return q
            groups = bp["kv_idx"][s][: bp["kv_count"][s]]
            kc = np.concatenate([np.arange((H + g) * dh, (H + g + 1) * dh) for g in groups])
            return np.concatenate([q, kc, kc + Hkv * dh])

        def get_batch(kind, rnd_, s, k, width, bp=bp, gm=gm):
            if s == 0 and ("central", kind, k) in store:
                return store[("central", kind, k)][0][:, held_cols(bp, s, kind == I.BATCH_TGT_QKV)]
            if masked_attn and kind in (I.BATCH_TGT_QKV, I.BATCH_A):
                full_width = gm.nq if kind == I.BATCH_TGT_QKV else gm.a_sub
                return store[(kind, k, full_width)][s][:, held_cols(bp, s, kind == I.BATCH_TGT_QKV)]
            if kind == I.BATCH_TGT_QKV and ragged:     # device layout [Q | K pad | V pad] -> oracle [Q | K | V]
                arr = store[(kind, k, gm.nq)][s]
                kc = bp["kv_count"][s] * w.d_head
                kvw = gm.kv_max * w.d_head
                return np.concatenate([arr[:, :gm.a_sub], arr[:, gm.a_sub:gm.a_sub + kc],
                                       arr[:, gm.a_sub + kvw:gm.a_sub + kvw + kc]], axis=1)
            return store[(kind, k, width)][s]

        full64 = {m: v.astype(np.float64) for m, v in full_np[l].items()}
        new, new_shadow, _, losses = o.round_blockwise_layer(w, full64, get_batch, rnd, l, lowp)
        assert np.array_equal(eng.bufs[eng.kind_of(l)]["idx_ffn"][l].cpu().numpy(), bp["ffn"])
        for m in eng.full:
            res = (eng.full_f32[m][l] if lowp else eng.full[m][l]).cpu().numpy().astype(np.float64)
            delta_w, delta_g = new[m] - full64[m], res - full64[m]
            # fp32: the update is ~1e-4 of the weight, so the fp32 storage of W bounds the accuracy of the
            # difference at ~1e-3; the weights themselves must agree to fp32 rounding.
            assert rel_fro(delta_g, delta_w) < (tol_dw if lowp else 1e-3), (l, m, rel_fro(delta_g, delta_w))
            if not lowp:
                assert np.max(np.abs(res - new[m])) <= 2e-7 * np.max(np.abs(new[m])), (l, m)
        for bi, name in enumerate(("ffn", "qkv", "o")[: 3 if eng.has_attn else 1]):
            got = eng.loss[l, bi, : w.local_steps].cpu().numpy()
            want = np.array([losses[s][name] for s in range(w.n_subnets)]).T
            assert np.allclose(got, want, rtol=2e-2 if lowp else 1e-4), (l, name)
    return eng, before


def test_config1_fp32_round_matches_oracle_everywhere(B):
    _run_round_and_compare(B, I.PRESETS[1])


@pytest.mark.parametrize("cfg,dims", [
    (2, dict(d_model=192, d_ff=528, d_head=16, tokens=200, n_layers=2, local_steps=2)),
    (3, dict(d_model=256, d_ff=688, d_head=8, tokens=256, n_layers=2, local_steps=2)),
    (4, dict(d_model=328, d_ff=1376, d_head=8, tokens=200, n_layers=1, local_steps=2)),
])
def test_scaled_twin_rounds_match_oracle(B, cfg, dims):
    w = I.scaled_twin(I.PRESETS[cfg], **dims)
    _run_round_and_compare(B, w)


@pytest.mark.parametrize("kind,mode", [(I.FFN_SWIGLU, I.MODE_COVER), (I.FFN_GELU, I.MODE_IID)])
def test_hybrid_twist_round_matches_the_oracle_round(B, kind, mode):
    """Hybrid TwIST (Sec. 4.1): worker 0 trains in place on the full-width model under its activation mask, the
    others on gathered slices; the round is the same function as the all-gathered round the oracle computes."""
    from paper_2511_03983_b200.engine import HybridRoundEngine
    w = replace(I.scaled_twin(I.PRESETS[5], d_model=136, d_ff=544, d_head=0, tokens=200, n_layers=2, local_steps=2),
                n_subnets=4, ffn_kind=kind, sample_mode=mode, lr=0.05)
    eng, before = _run_round_and_compare(B, w, engine_cls=HybridRoundEngine)
    assert any(not torch.equal(eng.full[m], before[m]) for m in before)        # the round did train


@pytest.mark.parametrize("eval_keep_ratio", [0.25, 0.5])
def test_deployment_extraction_and_evaluation_modes(B, eval_keep_ratio):
    """Sec. 4.2: a subnet extracted with the sampler's procedure at a subnet ratio that need not be the training one,
    evaluated forward-only with its own scale; the full model evaluated directly (no scale, no mask)."""
    from paper_2511_03983_b200.engine import RoundEngine
    base = I.scaled_twin(I.PRESETS[4], d_model=136, d_ff=544, d_head=8, tokens=200, n_layers=1, local_steps=1)
    w = replace(base, ffn_keep=int(base.n_ffn_blocks * eval_keep_ratio), sample_mode=I.MODE_IID)
    eng = RoundEngine(w)
    full_np = _load_full(eng, w)
    store = _load_batches(eng, w, 0)
    eng.sample_masks(0)
    eng.gather_layer(0)
    got = eng.evaluate_subnets(0, 0).cpu().numpy()
    got_full = eng.evaluate_full_ffn(0, 0).cpu().numpy()
    dense = eng.export_subnet(1)
    torch.cuda.synchronize()
    check_status(B)
    bp = o.layer_blueprints(w, 0, 0)
    alpha = o.act_scale(w.n_ffn_blocks, w.ffn_keep)
    F = w.d_ff
    for s in range(w.n_subnets):
        sl = {m: v.astype(np.float64) for m, v in o.gather_layer(w, full_np[0], bp, s).items()}
        X, Tg = store[(I.BATCH_X, 0)][s].astype(np.float64), store[(I.BATCH_TGT_D, 0)][s].astype(np.float64)
        Y, _ = o.ffn_fwd(X, sl["up"], sl["gate"], sl["down"], w.ffn_kind, alpha, True)
        want, _ = o.mse(Y, Tg, True)
        assert abs(got[0, s] - want) <= 2e-2 * want, (s, got[0, s], want)
        fm = {m: full_np[0][m].astype(np.float64) for m in ("up", "gate", "down")}
        Yf, _ = o.ffn_fwd(X, fm["up"], fm["gate"], fm["down"], w.ffn_kind, 1.0, True)
        want_f, _ = o.mse(Yf, Tg, True)
        assert abs(got_full[s] - want_f) <= 2e-2 * want_f, (s, got_full[s], want_f)
        if s == 1:      # the exported dense model is the gathered slice, bit for bit
            f = w.f_sub
            assert np.array_equal(host(dense["w_gu"][:f]), sl["gate"]) and np.array_equal(host(dense["w_gu"][f:]), sl["up"])
            assert np.array_equal(host(dense["w_down"]), sl["down"])
    assert F // w.ffn_block == w.n_ffn_blocks


@pytest.mark.parametrize("kind,mode", [(I.FFN_SWIGLU, I.MODE_COVER), (I.FFN_RELU, I.MODE_IID)])
def test_masked_twist_round_matches_the_oracle_round(B, kind, mode):
    """Masked TwIST (Sec. 4.1) as a whole round: every worker a full-width copy under its activation mask; the
    round is the same function as the gathered round the oracle computes."""
    from paper_2511_03983_b200.engine import MaskedRoundEngine
    w = replace(I.scaled_twin(I.PRESETS[5], d_model=136, d_ff=544, d_head=0, tokens=200, n_layers=2, local_steps=2),
                n_subnets=4, ffn_kind=kind, sample_mode=mode, lr=0.05)
    eng, before = _run_round_and_compare(B, w, engine_cls=MaskedRoundEngine, keep_f32_full=True)
    assert eng.w_gu.shape[1] == eng.g * w.d_ff            # nothing is physically smaller


def test_hybrid_twist_round_with_adam_matches_the_oracle_round(B):
    """Hybrid TwIST with the paper's optimiser: the central worker's moments are full-width and start at zero like
    the slices' moments; a masked neuron's zero gradient gives a zero Adam step."""
    from paper_2511_03983_b200.engine import HybridRoundEngine
    w = replace(I.scaled_twin(I.PRESETS[5], d_model=136, d_ff=544, d_head=0, tokens=200, n_layers=2, local_steps=3),
                n_subnets=4, sample_mode=I.MODE_COVER, optimizer="adam", lr=1e-3, beta1=0.9, beta2=0.99, adam_eps=3e-3)
    _run_round_and_compare(B, w, engine_cls=HybridRoundEngine)


def test_hidden_mask_from_cover_bits(B):
    cover = np.array([0b101, 0b010, 0, 0b111, 0b100], dtype=np.uint32)
    mask = torch.zeros(2, 15, dtype=torch.uint8, device="cuda")
    B.twist_hidden_mask(dev(cover.view(np.int32)), 5, 3, 1, 2, mask)
    torch.cuda.synchronize()
    want = np.array([[(c >> s) & 1 for c in cover for _ in range(3)] for s in (1, 2)], dtype=np.uint8)
    assert np.array_equal(mask.cpu().numpy(), want)


def test_scaled_twin_round_with_common_blocks_matches_oracle(B):
    """Common blocks (Sec. 3.1: blocks every subnet holds) in both partitioned kinds: their rows are averaged over
    all S workers; the cover construction of Algorithm 1 runs over the remaining blocks."""
    w = replace(I.scaled_twin(I.PRESETS[3], d_model=256, d_ff=688, d_head=8, tokens=256, n_layers=2, local_steps=2),
                common_ffn=(0, 5, 17, 400, 687), common_heads=(1, 30))
    eng, _ = _run_round_and_compare(B, w)
    cover = eng.cover_ffn.cpu().numpy().view(np.uint32)
    full_mask = (1 << w.n_subnets) - 1
    assert np.all(cover[:, list(w.common_ffn)] == full_mask)
    assert np.all(eng.cover_head.cpu().numpy().view(np.uint32)[:, list(w.common_heads)] == full_mask)


@pytest.mark.parametrize("engine_kw", [dict(fuse_loss=False), dict(store_outputs=False)])
def test_scaled_twin_round_with_standalone_loss_and_without_stored_outputs(B, engine_kw):
    w = I.scaled_twin(I.PRESETS[3], d_model=256, d_ff=688, d_head=8, tokens=256, n_layers=1, local_steps=2)
    _run_round_and_compare(B, w, **engine_kw)


def test_round_with_zero_lr_is_identity_on_the_bf16_model(B):
    from paper_2511_03983_b200.engine import RoundEngine
    w = replace(I.scaled_twin(I.PRESETS[4], d_model=128, d_ff=512, d_head=8, tokens=128, n_layers=1, local_steps=1),
                lr=0.0)
    eng = RoundEngine(w)
    _load_full(eng, w)
    _load_batches(eng, w, 0)
    before = {m: v.clone() for m, v in eng.full.items()}
    eng.run_round(0)
    torch.cuda.synchronize()
    for m in before:      # aggregation of identical (untrained) subnets is the identity
        assert torch.equal(before[m], eng.full[m]), m


# --------------------------------------------------------------------------------------------- Adam

def test_fused_adam_update_matches_the_oracle(B):
    """Two consecutive steps of the fused Adam update (FFN block).  The moments are linear /
    quadratic in the gradient, so they carry the 2e-2 bar; the weight step, which is close to a sign function of
    the gradient where the gradient is small, is checked exactly against the formula applied to the device's own
    moments."""
    bf, dtype, kind, alpha = torch.bfloat16, I.DTYPE_BF16, I.FFN_SWIGLU, 2.0
    S, T, d, f = 2, 200, 328, 344
    lr, b1, b2, eps = 1e-3, 0.9, 0.95, 1e-8
    X = I.normal(95, 1, (S, T, d), 1.0, dtype)
    Wgu = I.normal(95, 2, (S, 2 * f, d), 0.05, dtype)
    Wd = I.normal(95, 3, (S, f, d), 0.05, dtype)
    dY = I.normal(95, 4, (S, T, d), 1e-3, dtype)
    t = lambda *s: torch.zeros(*s, dtype=bf, device="cuda")
    w_gu, w_down = dev(Wgu, bf), dev(Wd, bf)
    m_gu, m_down = w_gu.float(), w_down.float()
    mom = {n: torch.zeros_like(m_gu if "gu" in n else m_down) for n in ("m_gu", "v_gu", "m_down", "v_down")}
    dw_gu = torch.zeros(S, 2 * f, d, dtype=torch.float32, device="cuda")
    dw_down = torch.zeros(S, f, d, dtype=torch.float32, device="cuda")
    pre, hh, y, dpre = t(S, T, 2 * f), t(S, T, f), t(S, T, d), t(S, T, 2 * f)
    x_dev, dy_dev = dev(X, bf), dev(dY, bf)          # kept alive: the argument struct holds raw pointers only
    for step in (1, 2):
        a = B.ffn_args(kind, dtype, S, T, d, f, alpha, lr, opt=B.adam(step, b1, b2, eps), x=x_dev, w_gu=w_gu,
                       w_down=w_down, w_gu_master=m_gu, w_down_master=m_down, pre=pre, hh=hh, y=y, dy=dy_dev,
                       dpre=dpre, dw_gu=dw_gu, dw_down=dw_down, **mom)
        before = {"gu": (m_gu.clone(), mom["m_gu"].clone(), mom["v_gu"].clone()),
                  "down": (m_down.clone(), mom["m_down"].clone(), mom["v_down"].clone())}
        B.twist_subnet_ffn_fwd(a)
        B.twist_subnet_ffn_bwd(a)
        torch.cuda.synchronize()
        check_status(B)
        for name, master, grad in (("gu", m_gu, dw_gu), ("down", m_down, dw_down)):
            w0, m0, v0 = (x.double().cpu().numpy() for x in before[name])
            g = grad.double().cpu().numpy()                       # the device's own gradient
            new, m1, v1, _ = o.adam(w0, m0, v0, g, step, lr, b1, b2, eps, True)
            assert rel_fro(host(mom["m_" + name]), m1) < 1e-5 and rel_fro(host(mom["v_" + name]), v1) < 1e-5
            assert rel_fro(host(master) - w0, new - w0) < 1e-3, (name, step)     # fp32 sqrt / divide vs fp64
        if step == 1:      # fresh moments against the oracle's own gradients: m = (1 - b1) g, v = (1 - b2) g^2
            for s in range(S):
                Wg_s, Wu_s, Wd_s = Wgu[s, :f].astype(np.float64), Wgu[s, f:].astype(np.float64), Wd[s].astype(np.float64)
                Xs, dYs = X[s].astype(np.float64), dY[s].astype(np.float64)
                _, saved = o.ffn_fwd(Xs, Wu_s, Wg_s, Wd_s, kind, alpha, True)
                _, dWu, dWg, dWd = o.ffn_bwd(dYs, Xs, saved, Wu_s, Wg_s, Wd_s, kind, alpha, True)
                dWgu = np.concatenate([dWg, dWu], axis=0)
                assert rel_fro(host(mom["m_down"][s]), (1 - b1) * dWd) < GEMM_TOL
                assert rel_fro(host(mom["v_down"][s]), (1 - b2) * dWd * dWd) < 2 * GEMM_TOL
                assert rel_fro(host(mom["m_gu"][s]), (1 - b1) * dWgu) < GEMM_TOL
                assert rel_fro(host(mom["v_gu"][s]), (1 - b2) * dWgu * dWgu) < 2 * GEMM_TOL


def test_scaled_twin_round_with_adam_matches_oracle(B):
    """A free-running BLOCKWISE round with Adam; eps is large against sqrt(v) here, so the step is nearly linear
    in the gradient and the 5e-2 bar on the weight change is meaningful (with a tiny eps the step is a sign
    function of gradients that are themselves only known to 2e-2)."""
    w = replace(I.scaled_twin(I.PRESETS[3], d_model=256, d_ff=688, d_head=8, tokens=256, n_layers=1, local_steps=3),
                optimizer="adam", lr=1e-3, beta1=0.9, beta2=0.99, adam_eps=3e-3)
    _run_round_and_compare(B, w)


def test_stack_round_with_adam_runs_and_matches_losses(B):
    from paper_2511_03983_b200.engine import StackEngine
    w = replace(I.scaled_twin(I.PRESETS[2], d_model=192, d_ff=528, d_head=16, tokens=192, n_layers=2, local_steps=3),
                optimizer="adam", lr=1e-3, adam_eps=3e-3)
    eng = StackEngine(w, 2, 96, keep_f32_full=True)
    full_np = _load_full(eng, w)
    store = {}
    for k in range(w.local_steps):
        for kind, dst in ((I.BATCH_X, eng.X), (I.BATCH_TGT_D, eng.Td)):
            arr = np.stack([I.batch(w, kind, 0, s, k, w.d_model) for s in range(w.n_subnets)])
            store[(kind, k)] = arr
            dst.append(dev(arr, torch.bfloat16))
    eng.run_round(0)
    torch.cuda.synchronize()
    check_status(B)
    full64 = [{m: v.astype(np.float64) for m, v in layer.items()} for layer in full_np]
    new, _, losses = o.round_stack(w, full64, lambda kind, rnd, s, k, width: store[(kind, k)][s], 0, 2, 96, True)
    assert np.allclose(eng.stack_loss[: w.local_steps].cpu().numpy(), np.array(losses).T, rtol=2e-2)
    for l in range(w.n_layers):
        for m in eng.full:
            res = eng.full_f32[m][l].cpu().numpy().astype(np.float64)
            assert rel_fro(res - full64[l][m], new[l][m] - full64[l][m]) < 5e-2, (l, m)


# --------------------------------------------------------------------------------------------- chained rounds

def test_two_chained_rounds_gather_the_previous_rounds_shadow(B):
    """Sec. 3 (overview of a round: aggregate, then resample and dispatch again): round 1 gathers the bf16 model that
    round 0's aggregate wrote.  Round 0 is compared as usual.  Round 1 is compared with the oracle's round started
    from the very bytes the device gathers (its own bf16 shadow), with round 1's blueprints and batches; and the
    oracle's own free-running shadow differs from the device's only by isolated one-ulp rounding flips."""
    from paper_2511_03983_b200.engine import RoundEngine
    # a learning rate at which one round moves the weights by a sizeable part of a bf16 ulp, so that the model the
    # second round gathers differs from the initial one in many elements
    w = replace(I.scaled_twin(I.PRESETS[4], d_model=328, d_ff=1376, d_head=8, tokens=200, n_layers=2, local_steps=2),
                lr=0.5)
    eng = RoundEngine(w, keep_f32_full=True)
    full_np = _load_full(eng, w)
    assert w.n_kv_heads == w.n_heads
    prev_bp = None
    oracle_shadow = [{m: v.astype(np.float64) for m, v in layer.items()} for layer in full_np]
    for rnd in (0, 1):
        store = _load_batches(eng, w, rnd)
        start = [{m: eng.full[m][l].float().cpu().numpy().astype(np.float64) for m in eng.full} for l in range(w.n_layers)]
        eng.run_round(rnd)
        torch.cuda.synchronize()
        check_status(B)
        get_batch = lambda kind, r, s, k, width: store[(kind, k)][s]
        for l in range(w.n_layers):
            new, new_shadow, bp, losses = o.round_blockwise_layer(w, start[l], get_batch, rnd, l, True)
            assert np.array_equal(eng.idx_ffn[l].cpu().numpy(), bp["ffn"])
            assert np.array_equal(eng.idx_head[l].cpu().numpy(), bp["head"])
            for m in eng.full:
                res = eng.full_f32[m][l].cpu().numpy().astype(np.float64)
                assert rel_fro(res - start[l][m], new[m] - start[l][m]) < 5e-2, (rnd, l, m)
                # the model the next round gathers is the nearest-even rounding of the fp32 result
                assert torch.equal(eng.full[m][l], eng.full_f32[m][l].to(torch.bfloat16))
            # the free-running oracle (its own shadow from round 0) against the device's shadow
            _, free_shadow, _, _ = o.round_blockwise_layer(w, oracle_shadow[l], get_batch, rnd, l, True)
            for m in eng.full:
                got = eng.full[m][l].float().cpu().numpy().astype(np.float64)
                differ = got != free_shadow[m]
                # one bf16 ulp at the magnitude of the weight (of the old one where the update nearly cancels it)
                ulp = np.maximum(np.abs(free_shadow[m]), np.abs(oracle_shadow[l][m])) * 2.0 ** -7 + 1e-30
                assert differ.mean() < (0.02 if rnd == 0 else 0.06), (rnd, l, m, differ.mean())
                # a rounding flip per round, plus (for weights much smaller than their update) the 2e-2-level
                # difference of the updates themselves
                bound = 2.0 * (rnd + 1) * ulp + 0.1 * np.abs(free_shadow[m] - oracle_shadow[l][m])
                assert np.all(np.abs(got - free_shadow[m])[differ] <= bound[differ]), (rnd, l, m)
            oracle_shadow[l] = free_shadow
        changed = np.mean([np.mean(eng.full[m][l].float().cpu().numpy() != full_np[l][m]) for m in eng.full
                           for l in range(w.n_layers)])
        assert changed > 0.02, changed                       # the gathered model is not the initial one
        if prev_bp is not None:       # the blueprints were resampled
            assert not np.array_equal(prev_bp, eng.idx_ffn.cpu().numpy())
        prev_bp = eng.idx_ffn.cpu().numpy().copy()


# --------------------------------------------------------------------------------------------- index validation, bounded waits

def test_gather_skips_out_of_range_indices_and_reports_them(B):
    d, n_full, S, n_sub = 64, 20, 2, 6
    W = I.normal(81, 1, (n_full, d), 0.02, I.DTYPE_BF16)
    A = np.array([[0, 3, 5, 7, 11, 19], [1, 2, 25, 8, -3, 13]], dtype=np.int32)      # 25 and -3 are not blocks
    sub = torch.full((S, n_sub, d), 9.0, dtype=torch.bfloat16, device="cuda")
    master = torch.full((S, n_sub, d), 9.0, dtype=torch.float32, device="cuda")
    seg = B.gather_segment(dev(W, torch.bfloat16), sub, master, dev(A), None, n_sub, n_sub, 1, 0, n_sub * d, 0, n_full)
    B.twist_gather_subnets([seg], S, d, I.DTYPE_BF16)
    assert B.twist_device_status() == B.ERR_BAD_INDEX
    assert B.twist_device_status() == 0                      # reading clears the word
    for s in range(S):
        for j in range(n_sub):
            if 0 <= A[s, j] < n_full:
                assert np.array_equal(sub[s, j].float().cpu().numpy(), W[A[s, j]])
                assert np.array_equal(master[s, j].cpu().numpy(), W[A[s, j]])
            else:                                            # canaries intact
                assert torch.all(sub[s, j] == 9.0) and torch.all(master[s, j] == 9.0)
    # a later, valid call is unaffected
    A_ok = np.array([[0, 3, 5, 7, 11, 19], [1, 2, 4, 8, 9, 13]], dtype=np.int32)
    seg = B.gather_segment(dev(W, torch.bfloat16), sub, master, dev(A_ok), None, n_sub, n_sub, 1, 0, n_sub * d, 0, n_full)
    B.twist_gather_subnets([seg], S, d, I.DTYPE_BF16)
    check_status(B)
    assert np.array_equal(sub[1, 2].float().cpu().numpy(), W[4])


def test_aggregate_skips_rows_with_bad_ranks_and_reports_them(B):
    d, n_full, S, n_sub = 32, 8, 2, 4
    A = np.array([[0, 2, 4, 6], [1, 2, 5, 6]], dtype=np.int32)
    cover, _, pos = o.cover_and_pos(A, n_full)
    pos = pos.copy()
    pos[1, 5] = 7            # subnet 1 holds block 5, but rank 7 is not a row of its 4-row slice
    pos[0, 4] = -1           # cover says subnet 0 holds block 4, the rank says it does not
    W = I.normal(82, 1, (n_full, d), 0.02, I.DTYPE_FP32)
    subs = I.normal(82, 2, (S, n_sub, d), 0.02, I.DTYPE_FP32)
    full = dev(W)
    seg = B.aggregate_segment(full, None, dev(subs), dev(cover.view(np.int32)), dev(pos), n_full, 1, 0, n_sub * d, 0, n_sub)
    B.twist_aggregate([seg], S, d, I.DTYPE_FP32)
    assert B.twist_device_status() == B.ERR_BAD_INDEX
    got = full.cpu().numpy()
    want = aggregate_f32(W, [subs[0], subs[1]], A, 1)
    for b in range(n_full):
        if b in (4, 5):
            assert np.array_equal(got[b], W[b])              # left as it was
        else:
            assert np.array_equal(got[b].view(np.uint32), want[b].view(np.uint32))
    check_status(B)


def test_attention_core_survives_bad_head_and_group_indices(B):
    S, n_seqs, N, H, Hkv, keep, dh = 1, 1, 64, 8, 2, 2, 16
    a, kvw = keep * dh, 2 * dh
    qkv = dev(I.normal(83, 1, (S, N, a + 2 * kvw), 1.0, I.DTYPE_BF16), torch.bfloat16)
    out = torch.zeros(S, N, a, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(S, keep, N, dtype=torch.float32, device="cuda")
    head_idx = dev(np.array([[1, 77]], dtype=np.int32))      # head 77 does not exist (8 heads)
    kv_pos = dev(np.array([[0, 9]], dtype=np.int32))         # position 9 does not exist (2 kept groups)
    args = B.attn_core_args(B.BF16, S, n_seqs, N, keep, 2, dh, H, Hkv, qkv=qkv, out=out, lse=lse, head_idx=head_idx,
                            kv_pos=kv_pos)
    B.twist_attn_core_fwd(args)
    assert B.twist_device_status() == B.ERR_BAD_INDEX
    assert torch.isfinite(out.float()).all()
    check_status(B)


def test_a_bounded_wait_that_runs_out_reports_a_timeout_and_leaves_the_device_usable(B):
    """The give-up path of the kernels' waits: barriers nobody arrives at, a limit of one millisecond.  The status
    word reports the time-out once; the next real launches run normally."""
    import time
    check_status(B)
    t0 = time.perf_counter()
    B.twist_selftest_wait(1_000_000)
    assert B.twist_device_status() == B.ERR_DEVICE_TIMEOUT      # synchronises
    assert time.perf_counter() - t0 < 5.0                       # gave up after the limit, not after the 2 s default
    assert B.twist_device_status() == 0                         # cleared by the read
    with pytest.raises(B.TwistError):
        B.twist_selftest_wait(10 ** 10)                         # limits beyond 0.1 s are refused
    _ffn_case(B, I.FFN_SWIGLU, I.DTYPE_BF16, S=2, T=256, d=256, f=256, alpha=2.0, lr=0.5, seed=41)
    check_status(B)


def test_blockwise_round_with_a_shared_layer_matches_the_oracle(B):
    """Sec. 5 Setup: some layers are shared (N_sub = N_full in both kinds): every worker holds and trains the whole
    layer, scale 1, and the aggregate is the plain mean over the S workers; the other layers are partitioned."""
    w = replace(I.scaled_twin(I.PRESETS[3], d_model=256, d_ff=688, d_head=8, tokens=256, n_layers=3, local_steps=2),
                shared_layers=(0, 2))
    eng, _ = _run_round_and_compare(B, w)
    full_mask = (1 << w.n_subnets) - 1
    cover = eng.cover_ffn.cpu().numpy().view(np.uint32)
    assert np.all(cover[0] == full_mask) and np.all(cover[2] == full_mask) and not np.all(cover[1] == full_mask)
    assert eng.bufs["shared"]["w_gu"].shape[1] == 2 * w.d_ff and eng.bufs["part"]["w_gu"].shape[1] == 2 * w.f_sub
    assert eng.geo["shared"].alpha_f == 1.0 and eng.geo["shared"].alpha_a == 1.0


# --------------------------------------------------------------------------------------------- layer normalisation

@pytest.mark.parametrize("S,T,d,adam", [(2, 77, 328, False), (3, 300, 768, True), (1, 130, 4096, False), (2, 9, 8, False)])
def test_layernorm_parity(B, S, T, d, adam):
    """App. A, Layer Normalization, forward and backward against the oracle: outputs and input gradients (bf16) to the
    bar of the other stored activations, statistics and parameter gradients (fp32 sums) much tighter, the
    optimiser step on gamma / b against the oracle's step on the device's own gradients."""
    bf = torch.bfloat16
    eps, lr = 1e-5, 0.05
    X = I.normal(91, 1, (S, T, d), 2.0, I.DTYPE_BF16) + np.float32(0.5)
    X = I.f32_from_bf16_bits(I.bf16_bits_from_f32(X))
    dY = I.normal(91, 2, (S, T, d), 1e-2, I.DTYPE_BF16)
    R = I.normal(91, 3, (S, T, d), 1e-2, I.DTYPE_BF16)
    g0 = (1.0 + I.normal(91, 4, (S, d), 0.2, I.DTYPE_FP32)).astype(np.float32)
    b0 = I.normal(91, 5, (S, d), 0.2, I.DTYPE_FP32)
    x, dy, r = dev(X, bf), dev(dY, bf), dev(R, bf)
    gamma, beta = dev(g0), dev(b0)
    y, dx = torch.zeros_like(x), torch.zeros_like(x)
    mean = torch.zeros(S, T, dtype=torch.float32, device="cuda")
    rstd = torch.zeros_like(mean)
    dg, db = torch.zeros_like(gamma), torch.zeros_like(gamma)
    ws = torch.empty(B.twist_layernorm_workspace_bytes(S, T, d), dtype=torch.uint8, device="cuda")
    mom = {n: torch.zeros_like(gamma) for n in ("m_gamma", "v_gamma", "m_beta", "v_beta")} if adam else {}
    opt = dict(opt=B.adam(1, 0.9, 0.99, 1e-3), **mom) if adam else {}
    a = B.layernorm_args(B.BF16, S, T, d, eps, lr, x=x, y=y, mean=mean, rstd=rstd, gamma=gamma, beta=beta, dy=dy, dx=dx,
                         dx_residual=r, dgamma=dg, dbeta=db, ws=ws, **opt)
    B.twist_layernorm_fwd(a)
    B.twist_layernorm_bwd(a)
    torch.cuda.synchronize()
    check_status(B)
    for s in range(S):
        Xs = X[s].astype(np.float64)
        Yw, saved = o.layer_norm_fwd(Xs, g0[s].astype(np.float64), b0[s].astype(np.float64), True, eps)
        assert close(host(y[s]), Yw, GEMM_TOL) if d >= 32 else rel_fro(host(y[s]), Yw) < GEMM_TOL
        assert np.allclose(mean[s].cpu().numpy(), Xs.mean(axis=1), rtol=1e-5, atol=1e-6)
        assert np.allclose(rstd[s].cpu().numpy(), saved["rstd"][:, 0], rtol=1e-5)
        dXw, dgw, dbw = o.layer_norm_bwd(dY[s].astype(np.float64), saved, g0[s].astype(np.float64), True,
                                         residual=R[s].astype(np.float64))
        assert rel_fro(host(dx[s]), dXw) < GEMM_TOL
        assert rel_fro(host(dx[s]) - R[s], dXw - R[s]) < 4 * GEMM_TOL        # the normalisation's own part of the sum
        assert rel_fro(host(dg[s]), dgw) < 1e-4 and rel_fro(host(db[s]), dbw) < 1e-4
        if adam:
            for name, p0, grad, m_, v_ in (("gamma", g0[s], dg[s], mom["m_gamma"][s], mom["v_gamma"][s]),
                                           ("beta", b0[s], db[s], mom["m_beta"][s], mom["v_beta"][s])):
                gdev = grad.double().cpu().numpy()
                new, m1, v1, _ = o.adam(p0.astype(np.float64), np.zeros(d), np.zeros(d), gdev, 1, lr, 0.9, 0.99, 1e-3, False)
                got = (gamma if name == "gamma" else beta)[s].double().cpu().numpy()
                assert rel_fro(got - p0, new - p0) < 1e-3, name
                assert rel_fro(host(m_), m1) < 1e-5 and rel_fro(host(v_), v1) < 1e-5
        else:
            assert rel_fro(host(gamma[s]) - g0[s], -lr * dgw) < 1e-3
            assert rel_fro(host(beta[s]) - b0[s], -lr * dbw) < 1e-3
    # in place: dx may overwrite dy
    dy2 = dy.clone()
    gamma.copy_(dev(g0)); beta.copy_(dev(b0))
    a2 = B.layernorm_args(B.BF16, S, T, d, eps, 0.0, x=x, mean=mean, rstd=rstd, gamma=gamma, beta=beta, dy=dy2, dx=dy2,
                          dx_residual=r, ws=ws)
    B.twist_layernorm_bwd(a2)
    torch.cuda.synchronize()
    assert torch.equal(dy2, dx)


@pytest.mark.parametrize("cfg,dims", [
    (4, dict(d_model=136, d_ff=544, d_head=8, tokens=200, n_layers=2, local_steps=2)),       # multi-head attention
    (3, dict(d_model=256, d_ff=688, d_head=8, tokens=256, n_layers=2, local_steps=1)),       # grouped-query: masked KV groups
])
def test_masked_twist_round_with_head_masks_matches_the_oracle_round(B, cfg, dims):
    """Masked TwIST (Sec. 4.1) with attention: FFN activations masked, and a head mask on the attention blocks (the
    dropped heads' columns out of the QKV block's loss, their outputs zero before the output projection, no gradient
    into them).  The round equals the gathered round the oracle computes; the rows of dropped heads keep their bytes
    in every worker's copy."""
    from paper_2511_03983_b200.engine import MaskedRoundEngine
    w = replace(I.scaled_twin(I.PRESETS[cfg], **dims), lr=0.05)
    eng, before = _run_round_and_compare(B, w, engine_cls=MaskedRoundEngine, keep_f32_full=True)
    assert eng.w_qkv.shape[1] == (w.n_heads + 2 * w.n_kv_heads) * w.d_head        # nothing is physically smaller
    # the last layer's worker copies: rows of heads a worker does not hold are bit-identical to the gathered model
    l = w.n_layers - 1
    bp = o.layer_blueprints(w, 0, l)
    for s in range(w.n_subnets):
        dropped = np.setdiff1d(np.arange(w.n_heads), bp["head"][s])
        rows = np.concatenate([np.arange(h * w.d_head, (h + 1) * w.d_head) for h in dropped])
        rt = torch.from_numpy(rows).cuda()
        assert torch.equal(eng.w_qkv_m[s][rt], before["qkv"][l][rt].float())
        assert torch.equal(eng.w_o_m[s][rt], before["o"][l][rt].float())


@pytest.mark.parametrize("cfg,dims,extra", [
    (4, dict(d_model=136, d_ff=544, d_head=8, tokens=200, n_layers=2, local_steps=2), dict(lr=0.05)),
    (3, dict(d_model=256, d_ff=688, d_head=8, tokens=256, n_layers=1, local_steps=2),
     dict(optimizer="adam", lr=1e-3, beta2=0.99, adam_eps=3e-3)),
])
def test_hybrid_twist_round_with_attention_matches_the_oracle_round(B, cfg, dims, extra):
    """Hybrid TwIST (Sec. 4.1) with attention blocks: the central worker trains the full-width projections in place
    under its head mask, the others train gathered slices; the aggregate takes the central worker's rows from the
    full fp32 matrices.  The round equals the all-gathered round of the oracle."""
    from paper_2511_03983_b200.engine import HybridRoundEngine
    w = replace(I.scaled_twin(I.PRESETS[cfg], **dims), **extra)
    eng, before = _run_round_and_compare(B, w, engine_cls=HybridRoundEngine)
    assert any(not torch.equal(eng.full[m], before[m]) for m in ("qkv", "o"))


def test_plan_caches_tensor_maps_and_changes_no_result(B):
    """The same FFN forward / backward on the same buffers without a plan, with a fresh plan, and with the warm plan:
    bit-identical results; the warm pass encodes no tensor map (every lookup hits)."""
    S, T, d, f = 2, 200, 328, 344
    plan = B.Plan(replace(I.PRESETS[5], n_subnets=S, tokens=T, d_model=d, d_ff=4 * f, ffn_keep=f))
    bf = torch.bfloat16
    t = lambda *shape: torch.zeros(*shape, dtype=bf, device="cuda")
    X = dev(I.normal(97, 1, (S, T, d), 1.0, I.DTYPE_BF16), bf)
    dY = dev(I.normal(97, 4, (S, T, d), 1e-3, I.DTYPE_BF16), bf)
    Wgu = dev(I.normal(97, 2, (S, 2 * f, d), 0.05, I.DTYPE_BF16), bf)
    Wd = dev(I.normal(97, 3, (S, f, d), 0.05, I.DTYPE_BF16), bf)
    buf = dict(w_gu=t(S, 2 * f, d), w_down=t(S, f, d), pre=t(S, T, 2 * f), hh=t(S, T, f), y=t(S, T, d),
               dpre=t(S, T, 2 * f), dx=t(S, T, d))
    buf["w_gu_master"] = torch.zeros(S, 2 * f, d, dtype=torch.float32, device="cuda")
    buf["w_down_master"] = torch.zeros(S, f, d, dtype=torch.float32, device="cuda")
    results, stats = [], []
    for use_plan in (None, plan, plan):
        buf["w_gu"].copy_(Wgu); buf["w_down"].copy_(Wd)
        buf["w_gu_master"].copy_(Wgu.float()); buf["w_down_master"].copy_(Wd.float())
        a = B.ffn_args(I.FFN_SWIGLU, I.DTYPE_BF16, S, T, d, f, 2.0, 0.5, plan=use_plan, x=X, dy=dY, **buf)
        B.twist_subnet_ffn_fwd(a)
        B.twist_subnet_ffn_bwd(a)
        torch.cuda.synchronize()
        check_status(B)
        results.append({k: v.clone() for k, v in buf.items()})
        stats.append(plan.stats())
    for k in buf:
        assert torch.equal(results[0][k], results[1][k]) and torch.equal(results[0][k], results[2][k]), k
    assert not torch.equal(results[0]["w_gu"], Wgu)                      # the step did train
    (c0, h0, m0), (c1, h1, m1), (c2, h2, m2) = stats
    assert (c0, h0, m0) == (0, 0, 0)                                     # calls without the plan leave it alone
    assert c1 > 0 and m1 == c1                                           # cold: every distinct map encoded once
    assert c2 == c1 and m2 == m1 and h2 - h1 == h1 + m1                  # warm: as many lookups, all of them hits
    plan.close()


@pytest.mark.parametrize("cfg,dims,world", [
    (4, dict(d_model=256, d_ff=1024, d_head=16, tokens=256, n_layers=2, local_steps=2), 2),
    (3, dict(d_model=256, d_ff=688, d_head=8, tokens=256, n_layers=2, local_steps=2), 4),
    (1, dict(), 2),
    (4, dict(d_model=256, d_ff=1024, d_head=16, tokens=256, n_layers=1, local_steps=1), 1),
])
def test_subnets_sharded_over_several_gpus_match_the_single_gpu_round(B, cfg, dims, world):
    """The S subnets of a round spread over `world` ranks (Sec. 4.1: workers in parallel, one server average), emulated
    here as `world` engines in one process whose partial-sum buffers the test adds up in place of the all-reduce.
    Every rank ends with the same model bit for bit; local training is bit-identical to the single-GPU round (same
    slices, same batches, same kernels: the losses say so); the new model equals the single-GPU one up to the fp32
    rounding of a differently associated sum, and the fp64 oracle within the aggregate's bound."""
    from paper_2511_03983_b200.engine import RoundEngine, ShardedRoundEngine, shard_range
    w = I.scaled_twin(I.PRESETS[cfg], **dims) if dims else I.PRESETS[cfg]
    lowp = w.dtype == I.DTYPE_BF16
    kw = dict(keep_f32_full=True) if lowp else {}
    ref = RoundEngine(w, **kw)
    full_np = _load_full(ref, w)
    if ref.full_f32 is not None:
        for m in ref.full:
            ref.full_f32[m].copy_(ref.full[m].float())
    _load_batches(ref, w, 0)
    start = {m: v.clone() for m, v in ref.full.items()}
    ref.run_round(0)
    ranks = []
    for r in range(world):
        e = ShardedRoundEngine(w, rank=r, world=world, reduce=lambda t: None, **kw)
        s0, n = shard_range(w.n_subnets, r, world)
        assert (e.subnet_begin, e.S_local) == (s0, n)
        for m in e.full:
            e.full[m].copy_(start[m])
            if e.full_f32 is not None:
                e.full_f32[m].copy_(start[m].float())
        own = slice(s0, s0 + n)
        e.X, e.Td = [t[own].contiguous() for t in ref.X], [t[own].contiguous() for t in ref.Td]
        if e.has_attn:
            for gk in e.geo:
                e.batches[gk] = {name: [t[own].contiguous() for t in ref.batches[gk][name]] for name in ("Tq", "A")}
        e.sample_masks(0)
        ranks.append(e)
    for l in range(w.n_layers):
        for e in ranks:                                  # each rank's local training, one after the other
            e.gather_layer(l)
            for k in range(w.local_steps):
                e.ffn_step(l, k)
                if e.has_attn:
                    e.qkv_step(l, k)
                    e.o_step(l, k)
            e.aggregate_partial(l)
        total = ranks[0].part.clone()                    # the exchange: sum over the ranks, the same bits everywhere
        for e in ranks[1:]:
            total += e.part
        for e in ranks:
            e.part.copy_(total)
            e.aggregate_finish(l)
    torch.cuda.synchronize()
    check_status(B)
    for e in ranks:
        s0 = e.subnet_begin
        assert torch.equal(e.loss, ref.loss[..., s0:s0 + e.S_local])           # the same local training
        assert torch.equal(e.cover_ffn, ref.cover_ffn)                         # the same blueprints on every rank
        for m in e.full:
            assert torch.equal(e.full[m], ranks[0].full[m]), m                 # one model after the round
            if e.full_f32 is not None:
                assert torch.equal(e.full_f32[m], ranks[0].full_f32[m]), m
    got = ranks[0].full_f32 if lowp else ranks[0].full
    want = ref.full_f32 if lowp else ref.full
    for m in got:
        assert not torch.equal(ranks[0].full[m], start[m])                     # the round did change the model
        g, r_ = got[m].double(), want[m].double()
        # differently associated fp32 sums of at most S terms, each of magnitude <= |mean| * count
        assert float((g - r_).abs().max()) <= 4 * w.n_subnets * 2.0 ** -24 * float(r_.abs().max()), m
        if lowp:                                                               # shadow = nearest-even rounding of fp32
            assert torch.equal(ranks[0].full[m], got[m].to(torch.bfloat16))
        if world == 1:                                                         # one GPU: the two halves are the aggregator
            assert torch.equal(got[m], want[m]) and torch.equal(ranks[0].full[m], ref.full[m]), m


def test_layer_step_captured_in_a_cuda_graph_replays_bit_identically(B):
    """A forward + backward FFN step with the fused loss, captured in a CUDA graph after an eager warm-up and replayed
    twice, gives the bits of the eager step.  Inside a capture the library's host-sequenced device counters are off
    (no wave synchronisation; the loss is finished by its own small launch), which changes no result; the contraction
    is long enough (2304, 3 waves of tiles) for the eager step to use both."""
    S, T, d, f = 4, 2560, 2304, 1280
    bf, dtype = torch.bfloat16, I.DTYPE_BF16
    t = lambda *shape: torch.zeros(*shape, dtype=bf, device="cuda")
    X = dev(I.normal(131, 1, (S, T, d), 1.0, dtype), bf)
    Tg = dev(I.normal(131, 4, (S, T, d), 1.0, dtype), bf)
    Wgu = dev(I.normal(131, 2, (S, 2 * f, d), 0.02, dtype), bf)
    Wd = dev(I.normal(131, 3, (S, f, d), 0.02, dtype), bf)
    out = dict(pre=t(S, T, 2 * f), hh=t(S, T, f), dy=t(S, T, d), dpre=t(S, T, 2 * f), dx=t(S, T, d),
               dw_gu=torch.zeros(S, 2 * f, d, dtype=torch.float32, device="cuda"),
               dw_down=torch.zeros(S, f, d, dtype=torch.float32, device="cuda"),
               loss=torch.zeros(S, dtype=torch.float32, device="cuda"))
    ws = torch.empty(B.twist_fused_loss_workspace_bytes(S, T, d), dtype=torch.uint8, device="cuda")
    a = B.ffn_args(I.FFN_SWIGLU, dtype, S, T, d, f, 2.0, 0.0, x=X, w_gu=Wgu, w_down=Wd, w_gu_master=Wgu.float(),
                   w_down_master=Wd.float(), y=None, tgt=Tg, loss_ws=ws, **out)

    def step():
        B.twist_subnet_ffn_fwd(a)
        B.twist_subnet_ffn_bwd(a)

    def snapshot():
        torch.cuda.synchronize()
        check_status(B)
        got = {k: v.clone() for k, v in out.items()}
        for v in out.values():
            v.zero_()
        return got

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step()                                       # eager, on the stream the capture will use
        eager = snapshot()
        assert float(eager["loss"].min()) > 0 and float(eager["dw_gu"].abs().max()) > 0
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            step()
        snapshot()                                   # capturing runs nothing: the outputs are still zero
        for _ in range(2):
            graph.replay()
            replayed = snapshot()
            for k in eager:
                assert torch.equal(eager[k], replayed[k]), k
        step()                                       # and eager launches work as before afterwards
        again = snapshot()
        for k in eager:
            assert torch.equal(eager[k], again[k]), k


def test_masters_created_by_the_first_update_equal_masters_written_by_the_gather(B):
    """The gather may leave the fp32 masters unwritten: the first weight update after it reads the bf16 slice, whose
    exact widening the master is.  Both ways give the same bits everywhere - full model, fp32 result, losses - for
    SGD and for Adam, with a learning rate and with lr = 0 (where the update only creates the masters)."""
    from paper_2511_03983_b200.engine import RoundEngine
    for extra in (dict(), dict(optimizer="adam", lr=1e-3, adam_eps=3e-3), dict(lr=0.0)):
        w = replace(I.scaled_twin(I.PRESETS[3], d_model=256, d_ff=688, d_head=8, tokens=256, n_layers=2, local_steps=2),
                    **extra)
        runs = []
        for lazy in (True, False):
            eng = RoundEngine(w, keep_f32_full=True, lazy_master=lazy)
            assert eng.lazy_master == lazy
            _load_full(eng, w)
            for m in eng.full:
                eng.full_f32[m].copy_(eng.full[m].float())
            for m in ("w_gu_m", "w_down_m", "w_qkv_m", "w_o_m"):       # whatever was there before must not matter
                getattr(eng, m).fill_(float("nan"))
            _load_batches(eng, w, 0)
            eng.run_round(0)
            torch.cuda.synchronize()
            check_status(B)
            runs.append(({m: v.clone() for m, v in eng.full.items()}, {m: v.clone() for m, v in eng.full_f32.items()},
                         eng.loss.clone(), eng.w_gu_m.clone()))
        for a, b in zip(runs[0][:2], runs[1][:2]):
            for m in a:
                assert torch.equal(a[m], b[m]), (extra, m)
        assert torch.equal(runs[0][2], runs[1][2]) and torch.equal(runs[0][3], runs[1][3])
        assert torch.isfinite(runs[0][3]).all()
