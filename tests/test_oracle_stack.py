"""Pins for the oracle's attention core and STACK composition against things other than itself:
torch's scaled_dot_product_attention and autograd on a dense / head-masked transformer written
with torch ops, finite differences, and the structural facts of App. A (a causal head's first
position copies V; uniform attention for equal keys).  CPU only."""
from types import SimpleNamespace

import numpy as np
import pytest
import torch

from oracle import twist_oracle as o


def _rng(seed):
    return np.random.default_rng(seed)


def _sdpa(Q, K, V):
    """[H, N, d] tensors -> causal attention with torch's own routine."""
    return torch.nn.functional.scaled_dot_product_attention(Q[None], K[None], V[None], is_causal=True)[0]


def _split(QKV, n_seqs, seq_len, dh, head_kv, kvw):
    """QKV [T, a + 2 kvw] -> per sequence (Q, K, V) as [H, N, dh] torch tensors, K/V expanded per head."""
    H = len(head_kv)
    a = H * dh
    out = []
    for b in range(n_seqs):
        r = QKV[b * seq_len:(b + 1) * seq_len]
        Q = torch.stack([r[:, h * dh:(h + 1) * dh] for h in range(H)])
        K = torch.stack([r[:, a + g * dh:a + (g + 1) * dh] for g in head_kv])
        V = torch.stack([r[:, a + kvw + g * dh:a + kvw + (g + 1) * dh] for g in head_kv])
        out.append((Q, K, V))
    return out


@pytest.mark.parametrize("head_kv,n_groups", [([0, 1, 2], 3), ([0, 0, 1, 1], 2), ([1, 1, 1], 2)])
def test_attention_core_forward_and_backward_match_torch_sdpa(head_kv, n_groups):
    r = _rng(3)
    n_seqs, N, dh = 2, 7, 4
    H = len(head_kv)
    kvw = n_groups * dh
    QKV = r.standard_normal((n_seqs * N, H * dh + 2 * kvw))
    dA = r.standard_normal((n_seqs * N, H * dh))
    A = o.attn_core_fwd(QKV, n_seqs, N, dh, head_kv, kvw, lowp=False)
    t = torch.from_numpy(QKV).requires_grad_(True)
    outs = []
    for Q, K, V in _split(t, n_seqs, N, dh, head_kv, kvw):
        O = _sdpa(Q, K, V)                                   # [H, N, dh]
        outs.append(torch.cat([O[h] for h in range(H)], dim=1))
    want = torch.cat(outs, dim=0)
    assert np.allclose(A, want.detach().numpy(), rtol=1e-10, atol=1e-12)
    (want * torch.from_numpy(dA)).sum().backward()
    dQKV = o.attn_core_bwd(dA, QKV, n_seqs, N, dh, head_kv, kvw, lowp=False)
    assert np.allclose(dQKV, t.grad.numpy(), rtol=1e-9, atol=1e-11)


def test_attention_core_backward_by_finite_differences():
    r = _rng(4)
    n_seqs, N, dh, head_kv, kvw = 1, 5, 3, [0, 0], 3
    QKV = r.standard_normal((N, 2 * dh + 2 * kvw))
    dA = r.standard_normal((N, 2 * dh))
    f = lambda Z: float(np.sum(o.attn_core_fwd(Z, n_seqs, N, dh, head_kv, kvw, False) * dA))
    g = o.attn_core_bwd(dA, QKV, n_seqs, N, dh, head_kv, kvw, False)
    eps = 1e-6
    for (i, j) in [(0, 0), (4, 1), (2, 7), (3, 10), (1, 6), (4, 11)]:
        Zp, Zm = QKV.copy(), QKV.copy()
        Zp[i, j] += eps
        Zm[i, j] -= eps
        assert abs((f(Zp) - f(Zm)) / (2 * eps) - g[i, j]) < 1e-6 * max(1.0, abs(g[i, j]))


def test_attention_core_structure_first_position_and_equal_keys():
    """Causal mask: position 0 attends only itself, so its output is its V row; with all keys
    equal the softmax is uniform and position n outputs the mean of V rows 0..n (App. A: head =
    softmax(Q K^T / sqrt(d)) V is a weighted sum of value vectors).  Sequences do not mix."""
    r = _rng(5)
    N, dh = 6, 4
    QKV = r.standard_normal((2 * N, 3 * dh))
    QKV[:, dh:2 * dh] = 1.0                                   # equal keys
    A = o.attn_core_fwd(QKV, 2, N, dh, [0], dh, False)
    V = QKV[:, 2 * dh:]
    for b in range(2):
        for n in range(N):
            assert np.allclose(A[b * N + n], V[b * N:b * N + n + 1].mean(axis=0), atol=1e-12)


# ------------------------------------------------------------------ STACK composition vs torch autograd

def _spec(**kw):
    base = dict(d_model=8, d_ff=12, ffn_block=1, ffn_keep=6, n_heads=4, n_kv_heads=2, head_keep=2, d_head=3,
                ffn_kind=o.FFN_SWIGLU, n_subnets=2, n_layers=2, local_steps=2, lr=0.05, sample_mode=o.MODE_COVER,
                seed_mask=17, common_ffn=(), common_heads=())
    base.update(kw)
    return SimpleNamespace(**base)


def _torch_act(kind, U, G):
    if kind == o.FFN_RELU:
        return torch.relu(U)
    if kind == o.FFN_GELU:
        return torch.nn.functional.gelu(U)
    return torch.nn.functional.silu(G) * U


def _torch_stack(spec, full, masks, X, n_seqs, N):
    """The chained layers written with torch ops on the FULL matrices with dropped neurons / heads
    masked out (Sec. 4.1: masked and gathered subnets compute the same function)."""
    H, Hkv, dh = spec.n_heads, spec.n_kv_heads, spec.d_head
    per = H // Hkv
    x = X
    ln = lambda v, g, b: torch.nn.functional.layer_norm(v, (v.shape[1],), g, b, eps=o.LN_EPS)
    for l, W in enumerate(full):
        ffn_keep, head_keep = o.layer_keeps(spec, l)
        alpha_f = (spec.d_ff / ffn_keep) ** 0.5
        alpha_a = (H / head_keep) ** 0.5
        x_in = x
        if "ln_a_g" in W:
            x = ln(x, W["ln_a_g"], W["ln_a_b"])
        qkv = x @ W["qkv"].T
        heads = []
        for b in range(n_seqs):
            r = qkv[b * N:(b + 1) * N]
            Q = torch.stack([r[:, h * dh:(h + 1) * dh] for h in range(H)])
            K = torch.stack([r[:, (H + h // per) * dh:(H + h // per + 1) * dh] for h in range(H)])
            V = torch.stack([r[:, (H + Hkv + h // per) * dh:(H + Hkv + h // per + 1) * dh] for h in range(H)])
            O = _sdpa(Q, K, V) * masks[l]["head"][:, None, None]
            heads.append(torch.cat([O[h] for h in range(H)], dim=1))
        x = x_in + alpha_a * (torch.cat(heads, dim=0) @ W["o"])
        x_f = ln(x, W["ln_f_g"], W["ln_f_b"]) if "ln_f_g" in W else x
        U = x_f @ W["up"].T
        G = x_f @ W["gate"].T if "gate" in W else None
        x = x + alpha_f * ((_torch_act(spec.ffn_kind, U, G) * masks[l]["ffn"]) @ W["down"])
    return x


@pytest.mark.parametrize("kind,hkv", [(o.FFN_SWIGLU, 2), (o.FFN_GELU, 4), (o.FFN_RELU, 1)])
def test_stack_local_steps_equal_masked_full_model_sgd_with_autograd(kind, hkv):
    """K local steps of a gathered subnet through the whole stack = K SGD steps of the masked full
    model under torch autograd, on the kept rows; dropped rows get zero gradient."""
    spec = _spec(ffn_kind=kind, n_kv_heads=hkv)
    r = _rng(6)
    L, d, F, H, dh = spec.n_layers, spec.d_model, spec.d_ff, spec.n_heads, spec.d_head
    n_seqs, N = 2, 5
    names = ["up", "down", "qkv", "o"] + (["gate"] if kind == o.FFN_SWIGLU else [])
    rows = {"up": F, "down": F, "gate": F, "qkv": (H + 2 * hkv) * dh, "o": H * dh}
    full = [{m: r.standard_normal((rows[m], d)) * 0.3 for m in names} for _ in range(L)]
    batches = {(kd, k): r.standard_normal((n_seqs * N, d)) for kd in (0, 1) for k in range(spec.local_steps)}
    get_batch = lambda kd, rnd, s, k, width: batches[(kd, k)]
    s = 1
    bps = [o.layer_blueprints(spec, 0, l) for l in range(L)]
    slices = [{m: v.astype(np.float64) for m, v in o.gather_layer(spec, full[l], bps[l], s).items()} for l in range(L)]
    head_kv = [o.head_kv_positions(bps[l], spec, s) for l in range(L)]
    losses = o.local_steps_stack(spec, slices, head_kv, get_batch, 0, s, n_seqs, N, lowp=False)

    # torch: masked full model, plain SGD
    tw = [{m: torch.from_numpy(v.copy()).requires_grad_(True) for m, v in full[l].items()} for l in range(L)]
    masks = []
    for l in range(L):
        fm = torch.zeros(F, dtype=torch.float64); fm[torch.from_numpy(bps[l]["ffn"][s].astype(np.int64))] = 1
        hm = torch.zeros(H, dtype=torch.float64); hm[torch.from_numpy(bps[l]["head"][s].astype(np.int64))] = 1
        masks.append({"ffn": fm, "head": hm})
    for k in range(spec.local_steps):
        y = _torch_stack(spec, tw, masks, torch.from_numpy(batches[(0, k)]), n_seqs, N)
        loss = torch.mean((y - torch.from_numpy(batches[(1, k)])) ** 2)
        assert abs(loss.item() - losses[k]) < 1e-10 * max(1.0, loss.item())
        loss.backward()
        with torch.no_grad():
            for W in tw:
                for v in W.values():
                    v -= spec.lr * v.grad
                    v.grad = None
    per = H // hkv
    for l in range(L):
        kept_f = bps[l]["ffn"][s]
        for m in ("up", "down") + (("gate",) if kind == o.FFN_SWIGLU else ()):
            got_full = tw[l][m].detach().numpy()
            assert np.allclose(slices[l][m], got_full[kept_f], rtol=1e-9, atol=1e-11), (l, m)
            dropped = np.setdiff1d(np.arange(F), kept_f)
            assert np.array_equal(got_full[dropped], full[l][m][dropped])
        heads = bps[l]["head"][s]
        q_rows = np.concatenate([np.arange(h * dh, (h + 1) * dh) for h in heads])
        groups = bps[l]["kv_idx"][s][: bps[l]["kv_count"][s]]
        k_rows = np.concatenate([np.arange((H + g) * dh, (H + g + 1) * dh) for g in groups])
        v_rows = k_rows + hkv * dh
        got_qkv = tw[l]["qkv"].detach().numpy()
        assert np.allclose(slices[l]["qkv"], got_qkv[np.concatenate([q_rows, k_rows, v_rows])], rtol=1e-9, atol=1e-11)
        assert np.allclose(slices[l]["o"], tw[l]["o"].detach().numpy()[q_rows], rtol=1e-9, atol=1e-11)
        dropped_heads = np.setdiff1d(np.arange(H), heads)
        if len(dropped_heads):
            dq = np.concatenate([np.arange(h * dh, (h + 1) * dh) for h in dropped_heads])
            assert np.array_equal(got_qkv[dq], full[l]["qkv"][dq])


def test_stack_round_with_one_full_subnet_is_dense_training():
    """S = 1 keeping everything: gather is the identity, alpha = 1, aggregation copies back: a STACK
    round equals K dense SGD steps (checked through the masked-model test's machinery above with
    all-ones masks)."""
    spec = _spec(n_subnets=1, ffn_keep=12, head_keep=4, n_kv_heads=4, ffn_kind=o.FFN_GELU, local_steps=1)
    r = _rng(7)
    L, d, F, H, dh = spec.n_layers, spec.d_model, spec.d_ff, spec.n_heads, spec.d_head
    n_seqs, N = 1, 4
    rows = {"up": F, "down": F, "qkv": 3 * H * dh, "o": H * dh}
    full = [{m: r.standard_normal((rows[m], d)) * 0.3 for m in rows} for _ in range(L)]
    X, Tg = r.standard_normal((N, d)), r.standard_normal((N, d))
    new, bps, losses = o.round_stack(spec, full, lambda kd, rnd, s, k, w: X if kd == 0 else Tg, 0, n_seqs, N, False)
    tw = [{m: torch.from_numpy(v.copy()).requires_grad_(True) for m, v in full[l].items()} for l in range(L)]
    ones = [{"ffn": torch.ones(F, dtype=torch.float64), "head": torch.ones(H, dtype=torch.float64)}] * L
    loss = torch.mean((_torch_stack(spec, tw, ones, torch.from_numpy(X), n_seqs, N) - torch.from_numpy(Tg)) ** 2)
    loss.backward()
    assert abs(loss.item() - losses[0][0]) < 1e-12
    for l in range(L):
        for m in rows:
            want = full[l][m] - spec.lr * tw[l][m].grad.numpy()
            assert np.allclose(new[l][m], want, rtol=1e-10, atol=1e-12), (l, m)


@pytest.mark.parametrize("shared", [(), (1,)])
def test_pre_ln_stack_equals_masked_full_model_with_layer_norm_under_autograd(shared):
    """App. A, Transformer Layer Architecture: LN -> attention -> skip -> LN -> FFN -> skip.  K local steps of a
    gathered subnet through the pre-LN stack = K SGD steps of the masked full model written with torch's own
    layer_norm, on the kept rows AND on the (shared, whole) normalisation parameters.  With a shared layer
    (N_sub = N_full, Sec. 5 Setup) that layer's slices are the whole matrices and its scales are 1."""
    spec = _spec(ffn_kind=o.FFN_SWIGLU, n_kv_heads=2, shared_layers=shared)
    r = _rng(16)
    L, d, F, H, dh, hkv = spec.n_layers, spec.d_model, spec.d_ff, spec.n_heads, spec.d_head, spec.n_kv_heads
    n_seqs, N = 2, 5
    rows = {"up": F, "down": F, "gate": F, "qkv": (H + 2 * hkv) * dh, "o": H * dh}
    full = []
    for _ in range(L):
        layer = {m: r.standard_normal((rows[m], d)) * 0.3 for m in rows}
        layer.update(ln_a_g=1 + 0.2 * r.standard_normal(d), ln_a_b=0.1 * r.standard_normal(d),
                     ln_f_g=1 + 0.2 * r.standard_normal(d), ln_f_b=0.1 * r.standard_normal(d))
        full.append(layer)
    batches = {(kd, k): r.standard_normal((n_seqs * N, d)) for kd in (0, 1) for k in range(spec.local_steps)}
    get_batch = lambda kd, rnd, s, k, width: batches[(kd, k)]
    s = 1
    bps = [o.layer_blueprints(spec, 0, l) for l in range(L)]
    slices = [{m: v.astype(np.float64) for m, v in o.gather_layer(spec, full[l], bps[l], s).items()} for l in range(L)]
    for l in range(L):
        assert all(m in slices[l] for m in o.LN_PARAMS)
        if l in shared:
            assert slices[l]["up"].shape[0] == F and slices[l]["o"].shape[0] == H * dh
    head_kv = [o.head_kv_positions(bps[l], spec, s) for l in range(L)]
    losses = o.local_steps_stack(spec, slices, head_kv, get_batch, 0, s, n_seqs, N, lowp=False)
    tw = [{m: torch.from_numpy(v.copy()).requires_grad_(True) for m, v in full[l].items()} for l in range(L)]
    masks = []
    for l in range(L):
        fm = torch.zeros(F, dtype=torch.float64); fm[torch.from_numpy(bps[l]["ffn"][s].astype(np.int64))] = 1
        hm = torch.zeros(H, dtype=torch.float64); hm[torch.from_numpy(bps[l]["head"][s].astype(np.int64))] = 1
        masks.append({"ffn": fm, "head": hm})
    for k in range(spec.local_steps):
        y = _torch_stack(spec, tw, masks, torch.from_numpy(batches[(0, k)]), n_seqs, N)
        loss = torch.mean((y - torch.from_numpy(batches[(1, k)])) ** 2)
        assert abs(loss.item() - losses[k]) < 1e-10 * max(1.0, loss.item())
        loss.backward()
        with torch.no_grad():
            for W in tw:
                for v in W.values():
                    v -= spec.lr * v.grad
                    v.grad = None
    for l in range(L):
        kept_f = bps[l]["ffn"][s]
        for m in ("up", "down", "gate"):
            assert np.allclose(slices[l][m], tw[l][m].detach().numpy()[kept_f], rtol=1e-9, atol=1e-11), (l, m)
        for m in o.LN_PARAMS:
            assert np.allclose(slices[l][m], tw[l][m].detach().numpy(), rtol=1e-9, atol=1e-11), (l, m)
            assert not np.allclose(slices[l][m], full[l][m])                       # they were trained
        heads = bps[l]["head"][s]
        q_rows = np.concatenate([np.arange(h * dh, (h + 1) * dh) for h in heads])
        assert np.allclose(slices[l]["o"], tw[l]["o"].detach().numpy()[q_rows], rtol=1e-9, atol=1e-11)


def test_round_stack_aggregates_the_normalisation_parameters_as_a_plain_mean():
    spec = _spec(ffn_kind=o.FFN_GELU, n_kv_heads=4, n_subnets=3, local_steps=1)
    r = _rng(17)
    L, d, F, H, dh = spec.n_layers, spec.d_model, spec.d_ff, spec.n_heads, spec.d_head
    n_seqs, N = 1, 4
    rows = {"up": F, "down": F, "qkv": 3 * H * dh, "o": H * dh}
    full = []
    for _ in range(L):
        layer = {m: r.standard_normal((rows[m], d)) * 0.3 for m in rows}
        layer.update(ln_a_g=np.ones(d), ln_a_b=np.zeros(d), ln_f_g=np.ones(d), ln_f_b=np.zeros(d))
        full.append(layer)
    data = {}
    get_batch = lambda kd, rnd, s, k, w: data.setdefault((kd, s), _rng(300 + 10 * kd + s).standard_normal((N, d)))
    new, bps, _ = o.round_stack(spec, full, get_batch, 0, n_seqs, N, False)
    for l in range(L):
        per_worker = []
        for s in range(spec.n_subnets):
            sl = [{m: v.astype(np.float64) for m, v in o.gather_layer(spec, full[j], bps[j], s).items()} for j in range(L)]
            hk = [o.head_kv_positions(bps[j], spec, s) for j in range(L)]
            o.local_steps_stack(spec, sl, hk, get_batch, 0, s, n_seqs, N, False)
            per_worker.append(sl[l])
        for m in o.LN_PARAMS:
            assert np.allclose(new[l][m], np.mean([pw[m] for pw in per_worker], axis=0), rtol=1e-13, atol=1e-15)
            assert new[l][m].shape == (d,)
