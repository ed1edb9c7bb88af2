"""Pins for the oracle's arithmetic against things other than itself: torch autograd on the
dense / masked full model, finite differences, the paper's closed forms (App. A), the
aggregator formula worked by hand, and the App. C byte model against Table 2.  CPU only."""
import os
from types import SimpleNamespace

import numpy as np
import pytest
import torch

from oracle import twist_oracle as o

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
KINDS = [o.FFN_RELU, o.FFN_GELU, o.FFN_SWIGLU]


def _rng(seed):
    return np.random.default_rng(seed)


def _torch_act(kind, pre_u, pre_g):
    if kind == o.FFN_RELU:
        return torch.relu(pre_u)
    if kind == o.FFN_GELU:
        return torch.nn.functional.gelu(pre_u)          # exact erf form
    return torch.nn.functional.silu(pre_g) * pre_u


def _dense_ffn_torch(kind, X, Wu, Wg, Wd, alpha, mask=None):
    """Textbook dense FFN with torch ops: y = alpha * (M * act(x W^T)) C."""
    Hh = _torch_act(kind, X @ Wu.T, X @ Wg.T if Wg is not None else None)
    if mask is not None:
        Hh = Hh * mask
    return alpha * (Hh @ Wd)


# ------------------------------------------------------------------ rounding helper

def test_round_bf16_matches_torch_conversion():
    x = _rng(0).standard_normal(20000).astype(np.float32) * 3
    ties = np.array([1.00390625, 1.01171875, -1.00390625, 0.0, 65280.0, 1e-30], dtype=np.float32)   # halfway cases
    x = np.concatenate([x, ties])
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(o.round_bf16(x.astype(np.float64)), want)


# ------------------------------------------------------------------ forward: dense special case

@pytest.mark.parametrize("kind", KINDS)
def test_ffn_forward_full_mask_is_the_dense_mlp(kind):
    r = _rng(1)
    X, Wu, Wg, Wd = r.standard_normal((9, 8)), r.standard_normal((16, 8)), r.standard_normal((16, 8)), \
        r.standard_normal((16, 8))
    Y, _ = o.ffn_fwd(X, Wu, Wg, Wd, kind, 1.0, lowp=False)
    want = _dense_ffn_torch(kind, *(torch.from_numpy(a) for a in (X, Wu, Wg, Wd)), 1.0).numpy()
    assert np.allclose(Y, want, rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ backward: autograd + finite differences

@pytest.mark.parametrize("kind", KINDS)
def test_ffn_backward_matches_autograd_and_finite_differences(kind):
    r = _rng(2)
    T, d, f = 4, 8, 16
    alpha = 1.7
    X, Wu, Wg, Wd, Tgt = (r.standard_normal(s) for s in [(T, d), (f, d), (f, d), (f, d), (T, d)])
    Y, saved = o.ffn_fwd(X, Wu, Wg, Wd, kind, alpha, lowp=False)
    loss, dY = o.mse(Y, Tgt, lowp=False)
    dX, dWu, dWg, dWd = o.ffn_bwd(dY, X, saved, Wu, Wg, Wd, kind, alpha, lowp=False)

    tX, tWu, tWg, tWd = (torch.tensor(a, requires_grad=True) for a in (X, Wu, Wg, Wd))
    tl = torch.mean((_dense_ffn_torch(kind, tX, tWu, tWg, tWd, alpha) - torch.from_numpy(Tgt)) ** 2)
    tl.backward()
    assert abs(loss - tl.item()) < 1e-12
    for got, want in [(dX, tX.grad), (dWu, tWu.grad), (dWd, tWd.grad)] + ([(dWg, tWg.grad)] if kind == 2 else []):
        assert np.allclose(got, want.numpy(), rtol=1e-9, atol=1e-12)

    # central finite differences on a few entries of every operand
    def loss_of(Xv, Wuv, Wgv, Wdv):
        Yv, _ = o.ffn_fwd(Xv, Wuv, Wgv, Wdv, kind, alpha, lowp=False)
        return o.mse(Yv, Tgt, lowp=False)[0]
    eps = 1e-6
    ops = [X, Wu, Wg, Wd]
    grads = [dX, dWu, dWg, dWd]
    for oi in range(4):
        if grads[oi] is None:
            continue
        for _ in range(6):
            idx = tuple(r.integers(0, n) for n in ops[oi].shape)
            if kind == o.FFN_RELU:   # keep away from the kink
                pass
            plus = [a.copy() for a in ops]
            minus = [a.copy() for a in ops]
            plus[oi][idx] += eps
            minus[oi][idx] -= eps
            fd = (loss_of(*plus) - loss_of(*minus)) / (2 * eps)
            assert abs(fd - grads[oi][idx]) <= 1e-6 * max(1.0, abs(fd)) + 1e-9, (kind, oi, idx, fd, grads[oi][idx])


def test_projection_backward_matches_autograd():
    r = _rng(3)
    T, d, n, a = 5, 8, 12, 6
    X, Wq, Tq = r.standard_normal((T, d)), r.standard_normal((n, d)), r.standard_normal((T, n))
    QKV = o.qkv_fwd(X, Wq, lowp=False)
    loss, dQ = o.mse(QKV, Tq, lowp=False)
    dX, dWq = o.qkv_bwd(dQ, X, Wq, lowp=False)
    tX, tW = torch.tensor(X, requires_grad=True), torch.tensor(Wq, requires_grad=True)
    torch.mean((tX @ tW.T - torch.from_numpy(Tq)) ** 2).backward()
    assert np.allclose(dX, tX.grad.numpy(), atol=1e-13) and np.allclose(dWq, tW.grad.numpy(), atol=1e-13)

    alpha = 2.0
    A, Wo, Td = r.standard_normal((T, a)), r.standard_normal((a, d)), r.standard_normal((T, d))
    Y = o.o_fwd(A, Wo, alpha, lowp=False)
    loss, dY = o.mse(Y, Td, lowp=False)
    dA, dWo = o.o_bwd(dY, A, Wo, alpha, lowp=False)
    tA, tW = torch.tensor(A, requires_grad=True), torch.tensor(Wo, requires_grad=True)
    tl = torch.mean((alpha * (tA @ tW) - torch.from_numpy(Td)) ** 2)
    tl.backward()
    assert abs(loss - tl.item()) < 1e-12
    assert np.allclose(dA, tA.grad.numpy(), atol=1e-13) and np.allclose(dWo, tW.grad.numpy(), atol=1e-13)


def test_mse_closed_form_and_valid_cols():
    Y = np.array([[1.0, 2.0, 5.0], [3.0, 4.0, 5.0]])
    Tg = np.array([[0.0, 0.0, 0.0], [1.0, 1.0, 0.0]])
    loss, dY = o.mse(Y, Tg, lowp=False)
    assert loss == pytest.approx((1 + 4 + 25 + 4 + 9 + 25) / 6)
    assert np.allclose(dY, 2 * (Y - Tg) / 6)
    loss, dY = o.mse(Y, Tg, lowp=False, valid_cols=2)
    assert loss == pytest.approx((1 + 4 + 4 + 9) / 4)
    assert np.allclose(dY[:, :2], 2 * (Y - Tg)[:, :2] / 4) and np.all(dY[:, 2] == 0)


# ------------------------------------------------------------------ masked == gathered (Masked TwIST, Sec. 4.1)

@pytest.mark.parametrize("kind", KINDS)
def test_masked_full_model_equals_gathered_slice(kind):
    r = _rng(4)
    T, d, F = 6, 8, 24
    kept = np.array(sorted(r.choice(F, 9, replace=False)))
    alpha = o.act_scale(F, len(kept))
    X, Wu, Wg, Wd, Tgt = (r.standard_normal(s) for s in [(T, d), (F, d), (F, d), (F, d), (T, d)])
    # gathered: physically smaller dense slice
    Y, saved = o.ffn_fwd(X, Wu[kept], Wg[kept], Wd[kept], kind, alpha, lowp=False)
    _, dY = o.mse(Y, Tgt, lowp=False)
    dX, dWu, dWg, dWd = o.ffn_bwd(dY, X, saved, Wu[kept], Wg[kept], Wd[kept], kind, alpha, lowp=False)
    # masked: y = M * f(x) on the full model, torch autograd
    mask = torch.zeros(F, dtype=torch.float64)
    mask[kept] = 1.0
    tX, tWu, tWg, tWd = (torch.tensor(a, requires_grad=True) for a in (X, Wu, Wg, Wd))
    tY = _dense_ffn_torch(kind, tX, tWu, tWg, tWd, alpha, mask)
    torch.mean((tY - torch.from_numpy(Tgt)) ** 2).backward()
    assert np.allclose(Y, tY.detach().numpy(), atol=1e-12)
    assert np.allclose(dX, tX.grad.numpy(), atol=1e-13)
    dropped = np.setdiff1d(np.arange(F), kept)
    for got, full in [(dWu, tWu.grad), (dWd, tWd.grad)] + ([(dWg, tWg.grad)] if kind == 2 else []):
        assert np.allclose(got, full.numpy()[kept], atol=1e-13)
        assert np.all(full.numpy()[dropped] == 0)


@pytest.mark.parametrize("kind", KINDS)
def test_oracle_hidden_mask_matches_autograd_of_the_masked_model(kind):
    """y = M * f(x) (Sec. 4.1) through the oracle's own mask option: forward, dX and every weight gradient equal
    torch autograd on the masked full model; rows of masked-out neurons get exactly zero gradient."""
    r = _rng(14)
    T, d, F = 5, 8, 16
    kept = np.array(sorted(r.choice(F, 6, replace=False)))
    alpha = o.act_scale(F, len(kept))
    X, Wu, Wg, Wd, Tgt = (r.standard_normal(s) for s in [(T, d), (F, d), (F, d), (F, d), (T, d)])
    m = np.zeros(F)
    m[kept] = 1.0
    Y, saved = o.ffn_fwd(X, Wu, Wg, Wd, kind, alpha, lowp=False, hidden_mask=m)
    _, dY = o.mse(Y, Tgt, lowp=False)
    dX, dWu, dWg, dWd = o.ffn_bwd(dY, X, saved, Wu, Wg, Wd, kind, alpha, lowp=False, hidden_mask=m)
    tX, tWu, tWg, tWd = (torch.tensor(a, requires_grad=True) for a in (X, Wu, Wg, Wd))
    tY = _dense_ffn_torch(kind, tX, tWu, tWg, tWd, alpha, torch.from_numpy(m))
    torch.mean((tY - torch.from_numpy(Tgt)) ** 2).backward()
    assert np.allclose(Y, tY.detach().numpy(), atol=1e-12)
    assert np.allclose(dX, tX.grad.numpy(), atol=1e-13)
    dropped = np.setdiff1d(np.arange(F), kept)
    for got, full in [(dWu, tWu.grad), (dWd, tWd.grad)] + ([(dWg, tWg.grad)] if kind == 2 else []):
        assert np.allclose(got, full.numpy(), atol=1e-13)
        assert np.all(got[dropped] == 0)
    # and the mask of all ones is the unmasked model
    Y1, _ = o.ffn_fwd(X, Wu, Wg, Wd, kind, alpha, lowp=False, hidden_mask=np.ones(F))
    Y0, _ = o.ffn_fwd(X, Wu, Wg, Wd, kind, alpha, lowp=False)
    assert np.array_equal(Y1, Y0)


# ------------------------------------------------------------------ aggregator (Sec. 3.3)

def test_aggregate_hand_example():
    full, subs, want = [], {}, []
    for line in open(os.path.join(GOLDEN, "aggregate_hand_example.txt")):
        p = line.split()
        if not p or p[0] == "#":
            continue
        if p[0] == "full":
            full.append([float(v) for v in p[1:]])
        elif p[0] == "sub":
            subs.setdefault(int(p[1]), []).append((int(p[2]), [float(v) for v in p[3:]]))
        elif p[0] == "want":
            want.append([float(v) for v in p[1:]])
    S = len(subs)
    blueprints = [np.array([row for row, _ in subs[s]]) for s in range(S)]
    slices = [np.array([v for _, v in subs[s]]) for s in range(S)]
    got = o.aggregate(np.array(full), slices, blueprints, 1)
    assert np.array_equal(got, np.array(want))


def test_aggregate_identity_disjoint_zero_coverage_and_live_mask():
    r = _rng(5)
    F, d, S = 40, 6, 4
    W = r.standard_normal((F, d))
    A = o.sample_blueprint(F, S, 16, [], 1, 0, 0, 0)
    # identical subnets (untrained slices) -> identity
    subs = [o.gather_rows(W, A[s], 1) for s in range(S)]
    assert np.allclose(o.aggregate(W, subs, A, 1), W, rtol=0, atol=1e-15)
    # disjoint subnets -> pure copy-back, no collisions
    Ad = o.sample_blueprint(F, S, 10, [], 1, 0, 0, 0)
    subs = [r.standard_normal((10, d)) for _ in range(S)]
    out = o.aggregate(W, subs, Ad, 1)
    for s in range(S):
        assert np.array_equal(out[Ad[s]], subs[s])
    # zero coverage keeps the old value; dropping a subnet removes it from numerator and denominator
    Ai = o.sample_blueprint(F, 2, 10, [], 1, 0, 0, 0, mode=o.MODE_IID)
    subs = [r.standard_normal((10, d)) for _ in range(2)]
    out = o.aggregate(W, subs, Ai, 1)
    uncovered = np.setdiff1d(np.arange(F), Ai.reshape(-1))
    assert len(uncovered) > 0 and np.array_equal(out[uncovered], W[uncovered])
    out0 = o.aggregate(W, subs, Ai, 1, live_mask=0b01)
    assert np.array_equal(out0[Ai[0]], subs[0])
    only1 = np.setdiff1d(Ai[1], Ai[0])
    assert np.array_equal(out0[only1], W[only1])
    # blocks of several rows
    Wb = r.standard_normal((12, d))
    outb = o.aggregate(Wb, [np.ones((6, d)), 3 * np.ones((6, d))], [np.array([0, 2]), np.array([2, 3])], 3)
    assert np.all(outb[0:3] == 1) and np.all(outb[6:9] == 2) and np.all(outb[9:12] == 3)
    assert np.array_equal(outb[3:6], Wb[3:6])


# ------------------------------------------------------------------ local training reduces to dense SGD

def _spec(**kw):
    base = dict(n_layers=1, d_model=8, n_heads=0, n_kv_heads=0, d_head=0, d_ff=16, ffn_kind=o.FFN_RELU,
                n_subnets=1, ffn_keep=16, head_keep=0, ffn_block=1, tokens=5, local_steps=3, lr=1e-2,
                sample_mode=o.MODE_COVER, seed_mask=1, common_ffn=(), common_heads=())
    base.update(kw)
    return SimpleNamespace(**base)


@pytest.mark.parametrize("kind", KINDS)
def test_single_full_subnet_round_is_dense_sgd(kind):
    r = _rng(6)
    spec = _spec(ffn_kind=kind, n_heads=4, n_kv_heads=4, d_head=2, head_keep=4)
    d, F, a = 8, 16, 8
    full = {"up": r.standard_normal((F, d)), "gate": r.standard_normal((F, d)), "down": r.standard_normal((F, d)),
            "qkv": r.standard_normal((3 * a, d)), "o": r.standard_normal((a, d))}
    batches = {}

    def get_batch(kind_, rnd, s, k, width):
        return batches.setdefault((kind_, k, width), _rng(100 + 10 * kind_ + k).standard_normal((spec.tokens, width)))

    new, _, bp, losses = o.round_blockwise_layer(spec, full, get_batch, 0, 0, lowp=False)
    assert np.array_equal(bp["ffn"][0], np.arange(F)) and np.array_equal(bp["head"][0], np.arange(4))

    # ordinary dense SGD on the full matrices with torch autograd (alpha = 1, full mask)
    t = {m: torch.tensor(v, requires_grad=True) for m, v in full.items()}
    for k in range(spec.local_steps):
        X, Td = torch.from_numpy(get_batch(0, 0, 0, k, d)), torch.from_numpy(get_batch(1, 0, 0, k, d))
        Tq, A = torch.from_numpy(get_batch(2, 0, 0, k, 3 * a)), torch.from_numpy(get_batch(3, 0, 0, k, a))
        l_ffn = torch.mean((_dense_ffn_torch(kind, X, t["up"], t["gate"], t["down"], 1.0) - Td) ** 2)
        l_qkv = torch.mean((X @ t["qkv"].T - Tq) ** 2)
        l_o = torch.mean((A @ t["o"] - Td) ** 2)
        (l_ffn + l_qkv + l_o).backward()
        assert losses[0]["ffn"][k] == pytest.approx(l_ffn.item(), rel=1e-12)
        assert losses[0]["qkv"][k] == pytest.approx(l_qkv.item(), rel=1e-12)
        assert losses[0]["o"][k] == pytest.approx(l_o.item(), rel=1e-12)
        with torch.no_grad():
            for m, v in t.items():
                if v.grad is not None:
                    v -= spec.lr * v.grad
                    v.grad = None
    for m in new:
        assert np.allclose(new[m], t[m].detach().numpy(), rtol=1e-11, atol=1e-13), m


def test_round_without_local_steps_is_the_identity():
    r = _rng(7)
    spec = _spec(ffn_kind=o.FFN_SWIGLU, n_subnets=3, ffn_keep=8, n_heads=8, n_kv_heads=2, d_head=2, head_keep=3,
                 local_steps=0)
    full = {"up": r.standard_normal((16, 8)), "gate": r.standard_normal((16, 8)), "down": r.standard_normal((16, 8)),
            "qkv": r.standard_normal(((8 + 4) * 2, 8)), "o": r.standard_normal((16, 8))}
    new, _, bp, _ = o.round_blockwise_layer(spec, full, None, 0, 0, lowp=False)
    for m in full:
        assert np.allclose(new[m], full[m], rtol=0, atol=1e-15), m


def test_round_with_two_subnets_averages_shared_rows_only():
    # K=1, S=2, overlapping subnets: rows held by one subnet take that subnet's SGD result,
    # shared rows take the mean of the two results (independent recomputation per subnet).
    r = _rng(8)
    spec = _spec(n_subnets=2, ffn_keep=10, local_steps=1, tokens=7)
    full = {"up": r.standard_normal((16, 8)), "down": r.standard_normal((16, 8))}
    data = {}

    def get_batch(kind_, rnd, s, k, width):
        return data.setdefault((kind_, s), _rng(50 + 7 * kind_ + s).standard_normal((spec.tokens, width)))

    new, _, bp, _ = o.round_blockwise_layer(spec, full, get_batch, 0, 0, lowp=False)
    alpha = float(np.sqrt(16 / 10))
    trained = []
    for s in range(2):
        rows = torch.from_numpy(bp["ffn"][s].astype(np.int64))
        tu, td = torch.tensor(full["up"], requires_grad=True), torch.tensor(full["down"], requires_grad=True)
        y = alpha * (torch.relu(torch.from_numpy(get_batch(0, 0, s, 0, 8)) @ tu[rows].T) @ td[rows])
        torch.mean((y - torch.from_numpy(get_batch(1, 0, s, 0, 8))) ** 2).backward()
        trained.append({"up": (tu - spec.lr * tu.grad).detach().numpy(), "down": (td - spec.lr * td.grad).detach().numpy()})
    in0, in1 = np.isin(np.arange(16), bp["ffn"][0]), np.isin(np.arange(16), bp["ffn"][1])
    for m in ("up", "down"):
        want = np.where((in0 & in1)[:, None], 0.5 * (trained[0][m] + trained[1][m]),
                        np.where(in0[:, None], trained[0][m], trained[1][m]))
        assert np.allclose(new[m], want, rtol=1e-12, atol=1e-14)


# ------------------------------------------------------------------ closed forms of App. A (He init)

def test_ffn_output_statistics_under_he_init():
    # E||y||^2 = E||x||^2 = d, Var(y_i) = 1, and E||y'||^2 / E||y||^2 = f'/F for a subset of neurons;
    # scaling by sqrt(F/f') restores the norm (Sec. 3.4).
    r = _rng(9)
    d, F, fsub, trials, T = 64, 256, 64, 40, 64
    full_sq, sub_sq, scaled_sq, comps = [], [], [], []
    for _ in range(trials):
        X = r.standard_normal((T, d))
        W = r.standard_normal((F, d)) * np.sqrt(2.0 / d)
        C = r.standard_normal((F, d)) * np.sqrt(1.0 / F)          # rows = neurons (C^ffn transposed)
        kept = r.choice(F, fsub, replace=False)
        Y, _ = o.ffn_fwd(X, W, None, C, o.FFN_RELU, 1.0, lowp=False)
        Ys, _ = o.ffn_fwd(X, W[kept], None, C[kept], o.FFN_RELU, 1.0, lowp=False)
        Ya, _ = o.ffn_fwd(X, W[kept], None, C[kept], o.FFN_RELU, o.act_scale(F, fsub), lowp=False)
        full_sq.append(np.mean(np.sum(Y * Y, axis=1)))
        sub_sq.append(np.mean(np.sum(Ys * Ys, axis=1)))
        scaled_sq.append(np.mean(np.sum(Ya * Ya, axis=1)))
        comps.append(Y.reshape(-1))
    full_sq, sub_sq, scaled_sq = np.mean(full_sq), np.mean(sub_sq), np.mean(scaled_sq)
    assert full_sq == pytest.approx(d, rel=0.05)
    assert np.var(np.concatenate(comps)) == pytest.approx(1.0, rel=0.05)
    assert sub_sq / full_sq == pytest.approx(fsub / F, rel=0.06)
    assert scaled_sq / full_sq == pytest.approx(1.0, rel=0.06)


def test_attention_output_projection_scales_with_kept_heads():
    # E||Y'_i||^2 = (H'/H) E||Y_i||^2 for statistically identical heads and C^attn ~ N(0, 1/(H d_head)).
    r = _rng(10)
    H, Hs, dh, d, T, trials = 12, 4, 16, 48, 64, 60
    full_sq, sub_sq = [], []
    for _ in range(trials):
        A = r.standard_normal((T, H * dh))
        C = r.standard_normal((H * dh, d)) * np.sqrt(1.0 / (H * dh))
        heads = np.sort(r.choice(H, Hs, replace=False))
        rows = o.block_rows_of(heads, dh)
        full_sq.append(np.mean(np.sum(o.o_fwd(A, C, 1.0, False) ** 2, axis=1)))
        sub_sq.append(np.mean(np.sum(o.o_fwd(A[:, rows], C[rows], 1.0, False) ** 2, axis=1)))
    assert np.mean(sub_sq) / np.mean(full_sq) == pytest.approx(Hs / H, rel=0.05)
    assert o.act_scale(H, Hs) == pytest.approx(np.sqrt(3.0))


# ------------------------------------------------------------------ byte model of App. C against Table 2

def test_parameter_model_matches_hand_counts_and_table2_slopes():
    counts = dict(l.split() for l in open(os.path.join(GOLDEN, "paper_gpt2_small_counts.txt")) if l[0] != "#")
    assert o.n_attn_params(768, 768) == int(counts["n_attn"])
    assert o.n_ffn_params(3072, 768) == int(counts["n_ffn"])
    comm = {}
    for line in open(os.path.join(GOLDEN, "paper_table2_comm.txt")):
        if line[0] != "#":
            setting, kept, tb = line.split()
            comm[(setting, int(kept))] = float(tb)
    # communication is proportional to the parameters moved: linear in the kept ratio, with per-2/12
    # slopes in the ratio N_ffn : N_attn, and `both` = attn + ffn
    slope = {s: (comm[(s, 10)] - comm[(s, 4)]) / 3 for s in ("attn", "ffn", "both")}
    assert slope["ffn"] / slope["attn"] == pytest.approx(o.n_ffn_params(3072, 768) / o.n_attn_params(768, 768), rel=0.01)
    assert slope["both"] == pytest.approx(slope["attn"] + slope["ffn"], rel=0.01)
    for s in ("attn", "ffn", "both"):
        assert comm[("ddp", 12)] - comm[(s, 10)] == pytest.approx(slope[s], rel=0.02)


def test_gather_is_the_concatenation_of_kept_blocks():
    W = np.arange(24 * 3, dtype=np.float64).reshape(24, 3)
    got = o.gather_rows(W, [1, 4], 2)
    assert np.array_equal(got, np.concatenate([W[2:4], W[8:10]]))
    got = o.gather_rows(W, [0, 2], 4, row_offset=8)
    assert np.array_equal(got, np.concatenate([W[8:12], W[16:20]]))


def test_lowp_mirror_stays_close_to_exact_and_is_bf16_representable():
    r = _rng(11)
    X = o.round_bf16(r.standard_normal((32, 64)))
    Wu, Wg, Wd = (o.round_bf16(r.standard_normal((48, 64)) * 0.02) for _ in range(3))
    Y, saved = o.ffn_fwd(X, Wu, Wg, Wd, o.FFN_SWIGLU, 2.0, lowp=True)
    Ye, _ = o.ffn_fwd(X, Wu, Wg, Wd, o.FFN_SWIGLU, 2.0, lowp=False)
    assert np.linalg.norm(Y - Ye) / np.linalg.norm(Ye) < 1e-2
    for a in (Y, saved["G"], saved["U"], saved["Hh"]):
        assert np.array_equal(o.round_bf16(a), a)


# ------------------------------------------------------------------ Adam (the optimiser of the paper's experiments)

def test_adam_steps_match_torch_optim_adam():
    r = _rng(40)
    w0 = r.standard_normal((5, 7))
    grads = [r.standard_normal((5, 7)) * s for s in (1.0, 1e-3, 5.0, 0.0, 2.0)]
    lr, b1, b2, eps = 3e-2, 0.9, 0.95, 1e-8
    wt = torch.from_numpy(w0.copy()).requires_grad_(True)
    opt = torch.optim.Adam([wt], lr=lr, betas=(b1, b2), eps=eps)
    w, m, v = w0.copy(), np.zeros_like(w0), np.zeros_like(w0)
    for t, g in enumerate(grads, start=1):
        wt.grad = torch.from_numpy(g.copy())
        opt.step()
        w, m, v, _ = o.adam(w, m, v, g, t, lr, b1, b2, eps, lowp=False)
        assert np.allclose(w, wt.detach().numpy(), rtol=1e-12, atol=1e-14), t


def test_blockwise_local_steps_with_adam_equal_torch_adam_on_the_dense_model():
    """S = 1 keeping everything, K = 3 steps with Adam = 3 torch.optim.Adam steps on the dense FFN block."""
    spec = SimpleNamespace(d_model=6, d_ff=10, ffn_block=1, ffn_keep=10, ffn_kind=o.FFN_GELU, n_heads=0, local_steps=3,
                           lr=1e-2, optimizer="adam", beta1=0.9, beta2=0.999, adam_eps=1e-8)
    r = _rng(41)
    sl = {"up": r.standard_normal((10, 6)) * 0.3, "down": r.standard_normal((10, 6)) * 0.3}
    batches = {(kind, k): r.standard_normal((9, 6)) for kind in (0, 1) for k in range(3)}
    tw = {m: torch.from_numpy(v.copy()).requires_grad_(True) for m, v in sl.items()}
    losses = o.local_steps_blockwise(spec, sl, lambda kind, rnd, s, k, w: batches[(kind, k)], 0, 0, lowp=False)
    opt = torch.optim.Adam(list(tw.values()), lr=1e-2, betas=(0.9, 0.999), eps=1e-8)
    for k in range(3):
        X, Tg = torch.from_numpy(batches[(0, k)]), torch.from_numpy(batches[(1, k)])
        loss = torch.mean((torch.nn.functional.gelu(X @ tw["up"].T) @ tw["down"] - Tg) ** 2)
        assert abs(loss.item() - losses["ffn"][k]) < 1e-12
        opt.zero_grad()
        loss.backward()
        opt.step()
    for m in sl:
        assert np.allclose(sl[m], tw[m].detach().numpy(), rtol=1e-9, atol=1e-12), m


def test_fp32_mirror_of_the_aggregator_agrees_with_the_float64_oracle():
    """tests/fp32_mirror.py (the fixed-order float32 evaluation the GPU result must equal bit for bit) against the
    float64 aggregator: same rows held, same untouched rows, and every averaged element within the rounding of
    count float32 additions and one division, (count + 1) 2^-24, relative to the mean magnitude of the values
    averaged.  A hand case fixes its order of operations."""
    from fp32_mirror import aggregate_f32
    rng = np.random.default_rng(3)
    n_full, S, n_sub, br, d = 40, 16, 30, 2, 24
    A = np.stack([np.sort(rng.choice(n_full, n_sub, replace=False)) for _ in range(S)])
    W = rng.standard_normal((n_full * br + 3, d)).astype(np.float32)
    subs = [rng.standard_normal((n_sub * br, d)).astype(np.float32) for _ in range(S)]
    for live in (None, 0b1010011):
        got = aggregate_f32(W, subs, A, br, live_mask=live, row_offset=3)
        want = o.aggregate(W.astype(np.float64), subs, A, br, live_mask=live, row_offset=3)
        mag = o.aggregate(np.abs(W).astype(np.float64), [np.abs(v) for v in subs], A, br, live_mask=live, row_offset=3)
        touched = np.any(want != W, axis=1)
        assert np.array_equal(got[~touched], W[~touched]) and touched[:3].sum() == 0
        assert np.max(np.abs(got[touched] - want[touched]) / mag[touched]) <= (S + 1) * 2.0 ** -24
    # order of operations: ((a + b) + c) / 3 in float32, not a + (b + c), not a product with a rounded 1/3
    a, b, c = np.float32(1.0), np.float32(2.0 ** -24), np.float32(2.0 ** -24)
    got = aggregate_f32(np.zeros((1, 1), np.float32), [np.full((1, 1), v, np.float32) for v in (a, b, c)],
                        [[0], [0], [0]], 1)
    assert got[0, 0] == np.float32((np.float32(a + b) + c) / np.float32(3.0)) == np.float32(1.0) / np.float32(3.0)
    assert got[0, 0] != np.float32(a + np.float32(b + c)) / np.float32(3.0)


# ------------------------------------------------------------------ layer normalisation (App. A)

def test_layer_norm_matches_torch_forward_and_autograd():
    r = _rng(31)
    T, d = 7, 12
    X, g, b = r.standard_normal((T, d)) * 2 + 0.5, r.standard_normal(d) + 1.0, r.standard_normal(d)
    dY, res = r.standard_normal((T, d)), r.standard_normal((T, d))
    Y, saved = o.layer_norm_fwd(X, g, b, lowp=False)
    tx, tg, tb = (torch.tensor(v, requires_grad=True) for v in (X, g, b))
    want = torch.nn.functional.layer_norm(tx, (d,), tg, tb, eps=o.LN_EPS)
    assert np.allclose(Y, want.detach().numpy(), rtol=1e-12, atol=1e-13)
    (want * torch.from_numpy(dY)).sum().backward()
    dX, dg, db = o.layer_norm_bwd(dY, saved, g, lowp=False)
    assert np.allclose(dX, tx.grad.numpy(), rtol=1e-10, atol=1e-12)
    assert np.allclose(dg, tg.grad.numpy(), rtol=1e-10, atol=1e-12)
    assert np.allclose(db, tb.grad.numpy(), rtol=1e-10, atol=1e-12)
    dXr, _, _ = o.layer_norm_bwd(dY, saved, g, lowp=False, residual=res)       # the skip connection's gradient
    assert np.allclose(dXr, dX + res, rtol=0, atol=1e-14)


def test_layer_norm_definition_and_finite_differences():
    """App. A, Layer Normalization: z = (x - mu) / sigma has zero mean and unit variance per token, and with the
    initial parameters (gamma = 1, b = 0: App. A, Initialization) the output is z itself; y is invariant to a
    shift and to a positive scaling of the token; the gradient passes a central-difference check."""
    r = _rng(32)
    T, d = 5, 16
    X = r.standard_normal((T, d)) * 3 + 1
    Y, saved = o.layer_norm_fwd(X, np.ones(d), np.zeros(d), lowp=False, eps=0.0)
    assert np.allclose(Y.mean(axis=1), 0, atol=1e-13) and np.allclose(Y.var(axis=1), 1, atol=1e-12)
    assert np.array_equal(Y, saved["z"])
    Y2, _ = o.layer_norm_fwd(4.0 * X + 7.0, np.ones(d), np.zeros(d), lowp=False, eps=0.0)
    assert np.allclose(Y, Y2, atol=1e-12)
    g, b, dY = r.standard_normal(d), r.standard_normal(d), r.standard_normal((T, d))
    f = lambda Z, gg, bb: float(np.sum(o.layer_norm_fwd(Z, gg, bb, False)[0] * dY))
    _, sv = o.layer_norm_fwd(X, g, b, False)
    dX, dg, db = o.layer_norm_bwd(dY, sv, g, False)
    eps = 1e-6
    for (i, j) in [(0, 0), (2, 5), (4, 15)]:
        Zp, Zm = X.copy(), X.copy()
        Zp[i, j] += eps; Zm[i, j] -= eps
        assert abs((f(Zp, g, b) - f(Zm, g, b)) / (2 * eps) - dX[i, j]) < 1e-6 * max(1.0, abs(dX[i, j]))
    for j in (0, 7):
        gp, gm = g.copy(), g.copy()
        gp[j] += eps; gm[j] -= eps
        assert abs((f(X, gp, b) - f(X, gm, b)) / (2 * eps) - dg[j]) < 1e-6 * max(1.0, abs(dg[j]))
        bp_, bm = b.copy(), b.copy()
        bp_[j] += eps; bm[j] -= eps
        assert abs((f(X, g, bp_) - f(X, g, bm)) / (2 * eps) - db[j]) < 1e-6 * max(1.0, abs(db[j]))


def test_layer_norm_parameter_count_is_two_d_model():
    """App. C: N_ln = 2 d_model per normalisation (gamma and b)."""
    d = 768
    _, saved = o.layer_norm_fwd(np.zeros((1, d)) + np.arange(d), np.ones(d), np.zeros(d), False)
    assert saved["z"].shape == (1, d) and np.ones(d).size + np.zeros(d).size == 2 * d


# ------------------------------------------------------------------ column-mask loss, masked attention worker (Sec. 4.1)

def test_mse_with_a_column_mask_and_with_no_valid_column():
    r = _rng(33)
    Y, Tg = r.standard_normal((6, 10)), r.standard_normal((6, 10))
    mask = np.array([1, 0, 0, 1, 1, 0, 1, 0, 0, 0])
    cols = np.flatnonzero(mask)
    loss, dY = o.mse(Y, Tg, False, col_mask=mask)
    assert loss == pytest.approx(np.mean((Y[:, cols] - Tg[:, cols]) ** 2), rel=1e-13)
    assert np.allclose(dY[:, cols], 2 * (Y[:, cols] - Tg[:, cols]) / (6 * len(cols))) and np.all(dY[:, mask == 0] == 0)
    l2, d2 = o.mse(Y[:, :4], Tg[:, :4], False, col_mask=np.ones(4))
    l3, d3 = o.mse(Y[:, :4], Tg[:, :4], False)
    assert l2 == l3 and np.array_equal(d2, d3)
    l0, d0 = o.mse(Y, Tg, False, col_mask=np.zeros(10))
    assert l0 == 0.0 and np.all(d0 == 0)


def test_head_masked_projections_equal_the_gathered_slices():
    """Sec. 4.1, Masked TwIST for attention: on the full-width projections with the dropped heads masked out (their
    query / key / value columns out of the loss; their head outputs zeroed before the output projection) the kept
    rows see the gathered subnet's outputs, losses and gradients, and the dropped rows get exactly zero gradient.
    Checked with torch autograd on the masked full matrices."""
    r = _rng(34)
    T, d, H, dh = 9, 10, 6, 4
    kept = np.array([1, 2, 5])
    rows = np.concatenate([np.arange(h * dh, (h + 1) * dh) for h in kept])
    qrows = np.concatenate([rows, H * dh + rows, 2 * H * dh + rows])          # Q, K, V rows of the kept heads
    Wqkv, Wo = r.standard_normal((3 * H * dh, d)), r.standard_normal((H * dh, d))
    X = r.standard_normal((T, d))
    Tq_full, A_full, Td = r.standard_normal((T, 3 * H * dh)), r.standard_normal((T, H * dh)), r.standard_normal((T, d))
    cmask = np.zeros(3 * H * dh); cmask[qrows] = 1
    amask = np.zeros(H * dh); amask[rows] = 1
    alpha = o.act_scale(H, len(kept))
    # gathered subnet
    out_g = o.qkv_fwd(X, Wqkv[qrows], False)
    loss_g, dq_g = o.mse(out_g, Tq_full[:, qrows], False)
    dx_g, dWq_g = o.qkv_bwd(dq_g, X, Wqkv[qrows], False)
    y_g = o.o_fwd(A_full[:, rows], Wo[rows], alpha, False)
    loss_o, dy = o.mse(y_g, Td, False)
    dA_g, dWo_g = o.o_bwd(dy, A_full[:, rows], Wo[rows], alpha, False)
    # masked full-width worker, by the oracle ...
    out_m = o.qkv_fwd(X, Wqkv, False)
    loss_m, dq_m = o.mse(out_m, Tq_full, False, col_mask=cmask)
    dx_m, dWq_m = o.qkv_bwd(dq_m, X, Wqkv, False)
    y_m = o.o_fwd(A_full * amask, Wo, alpha, False)
    _, dWo_m = o.o_bwd(dy, A_full * amask, Wo, alpha, False)
    assert loss_m == pytest.approx(loss_g, rel=1e-13) and np.allclose(dx_m, dx_g, atol=1e-14)
    assert np.allclose(dWq_m[qrows], dWq_g, atol=1e-14) and np.all(np.delete(dWq_m, qrows, axis=0) == 0)
    assert np.allclose(y_m, y_g, atol=1e-13)
    assert np.allclose(dWo_m[rows], dWo_g, atol=1e-14) and np.all(np.delete(dWo_m, rows, axis=0) == 0)
    # ... and by autograd on the masked model
    tq, to = torch.tensor(Wqkv, requires_grad=True), torch.tensor(Wo, requires_grad=True)
    tm = torch.from_numpy(cmask)
    lq = (((torch.from_numpy(X) @ tq.T - torch.from_numpy(Tq_full)) * tm) ** 2).sum() / (T * tm.sum())
    lo = torch.mean((alpha * ((torch.from_numpy(A_full) * torch.from_numpy(amask)) @ to) - torch.from_numpy(Td)) ** 2)
    (lq + lo).backward()
    assert lq.item() == pytest.approx(loss_m, rel=1e-12) and lo.item() == pytest.approx(loss_o, rel=1e-12)
    assert np.allclose(tq.grad.numpy(), dWq_m, atol=1e-13) and np.allclose(to.grad.numpy(), dWo_m, atol=1e-13)


# ------------------------------------------------------------------ shared layers (Sec. 5 Setup: N_sub = N_full)

def test_shared_layer_is_held_by_every_worker_and_averaged_over_all_of_them():
    r = _rng(35)
    spec = _spec(n_layers=2, n_subnets=3, ffn_keep=6, ffn_kind=o.FFN_GELU, n_heads=4, n_kv_heads=4, d_head=2,
                 head_keep=2, local_steps=1, tokens=6, shared_layers=(1,))
    assert o.layer_keeps(spec, 0) == (6, 2) and o.layer_keeps(spec, 1) == (16, 4)
    bp = o.layer_blueprints(spec, 0, 1)
    assert all(np.array_equal(row, np.arange(16)) for row in bp["ffn"])
    assert all(np.array_equal(row, np.arange(4)) for row in bp["head"])
    assert o.layer_blueprints(spec, 0, 0)["ffn"].shape == (3, 6)
    d, F, a = 8, 16, 8
    full = {"up": r.standard_normal((F, d)), "down": r.standard_normal((F, d)),
            "qkv": r.standard_normal((3 * a, d)), "o": r.standard_normal((a, d))}
    data = {}
    get_batch = lambda kd, rnd, s, k, width: data.setdefault((kd, s, width),
                                                             _rng(200 + 10 * kd + s).standard_normal((spec.tokens, width)))
    new, _, _, losses = o.round_blockwise_layer(spec, full, get_batch, 0, 1, lowp=False)
    # every worker trains the whole dense layer (scale 1) on its own batch; the aggregate is the plain mean
    mean = {m: np.zeros_like(v) for m, v in full.items()}
    for s in range(3):
        t = {m: torch.tensor(v, requires_grad=True) for m, v in full.items()}
        X, Td = torch.from_numpy(get_batch(0, 0, s, 0, d)), torch.from_numpy(get_batch(1, 0, s, 0, d))
        Tq, A = torch.from_numpy(get_batch(2, 0, s, 0, 3 * a)), torch.from_numpy(get_batch(3, 0, s, 0, a))
        l_ffn = torch.mean((_dense_ffn_torch(o.FFN_GELU, X, t["up"], None, t["down"], 1.0) - Td) ** 2)
        (l_ffn + torch.mean((X @ t["qkv"].T - Tq) ** 2) + torch.mean((A @ t["o"] - Td) ** 2)).backward()
        assert losses[s]["ffn"][0] == pytest.approx(l_ffn.item(), rel=1e-12)
        for m in full:
            mean[m] += (full[m] - spec.lr * t[m].grad.numpy()) / 3
    for m in full:
        assert np.allclose(new[m], mean[m], rtol=1e-11, atol=1e-13), m
