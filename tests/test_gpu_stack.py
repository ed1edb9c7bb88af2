"""Parity of the chained (STACK) composition with the CPU oracle: the attention core, the skip-connection
epilogues of the grouped GEMMs, and whole rounds of scaled-down twins of the stack-shaped workloads.
Tolerance: 2e-2 relative Frobenius error against the fp64 oracle that mirrors the bf16 rounding points."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import twist_oracle as o
from paper_2511_03983_b200 import inputs as I

pytestmark = pytest.mark.gpu

GEMM_TOL = 2e-2


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
    return t.detach().float().cpu().numpy().astype(np.float64)


def rel_fro(got, want):
    return float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-300))


# head_map: per subnet, (kept head ids, kept KV group list) under n_heads / n_kv_heads sharing; None = no sharing
@pytest.mark.parametrize("S,n_seqs,N,H,dh,gqa,ramp", [
    (2, 2, 64, 2, 64, None, 0.0),       # whole tiles, two threads per query
    (2, 3, 77, 3, 16, None, 0.0),       # ragged sequence length, one thread per query
    (1, 1, 200, 2, 128, None, 0.0),     # several key tiles, four threads per query
    (3, 2, 150, 4, 8, (8, 2), 0.0),     # grouped-query sharing: 8 heads in 2 groups, ragged group counts
    (2, 1, 130, 4, 32, (8, 4), 0.0),
    (2, 2, 300, 3, 64, None, 0.0),      # tensor-core path: three key blocks, ragged last block
    (2, 1, 333, 4, 64, (8, 2), 0.0),    # tensor-core path with grouped-query sharing
    (1, 2, 640, 2, 64, None, 6.0),      # keys grow along the sequence: the row maxima keep rising, so the
                                        # lazily updated reference maximum has to move several times
    (1, 1, 100, 2, 32, None, 6.0),
    (1, 2, 1, 1, 64, None, 0.0),        # tensor-core path, degenerate sizes: one token per sequence,
    (1, 1, 127, 1, 64, None, 0.0),      # one block minus a row,
    (2, 1, 129, 2, 64, None, 0.0),      # one block plus a row
])
def test_attention_core_parity(B, S, n_seqs, N, H, dh, gqa, ramp):
    bf = torch.bfloat16
    T = n_seqs * N
    if gqa is None:
        kv_max, head_kv = H, [np.arange(H)] * S
        extra, nh, nkv = {}, 0, 0
        kv_count = np.full(S, H, dtype=np.int32)
    else:
        nh, nkv = gqa
        per = nh // nkv
        rng = np.random.default_rng(5)
        head_idx = np.stack([np.sort(rng.choice(nh, H, replace=False)) for _ in range(S)]).astype(np.int32)
        head_idx[0] = np.arange(H)                      # subnet 0: heads of the first groups only (fewest groups)
        kv_idx, kv_count = o.kv_groups(head_idx, nh, nkv)
        _, _, kv_pos = o.cover_and_pos(kv_idx, nkv, counts=kv_count)
        kv_max = min(nkv, H)
        head_kv = [np.array([list(kv_idx[s][:kv_count[s]]).index(h // per) for h in head_idx[s]]) for s in range(S)]
        extra = dict(head_idx=dev(head_idx), kv_pos=dev(kv_pos.astype(np.int32)), kv_count=dev(kv_count))
        assert kv_count.min() < kv_max                  # the padding path is exercised
    a, kvw = H * dh, kv_max * dh
    nq = a + 2 * kvw
    QKV = I.normal(81, 1, (S, T, nq), 1.0, I.DTYPE_BF16)
    if ramp:
        pos = (np.arange(T) % N) / N
        QKV = QKV.copy()
        QKV[:, :, :a] *= 3.0
        QKV[:, :, a:a + kvw] *= (1.0 + ramp * pos)[None, :, None]
        QKV = I.f32_from_bf16_bits(I.bf16_bits_from_f32(QKV.astype(np.float32)))      # back onto the bf16 grid
    dA = I.normal(81, 2, (S, T, a), 1.0, I.DTYPE_BF16)
    qkv, d_out = dev(QKV, bf), dev(dA, bf)
    out = torch.zeros(S, T, a, dtype=bf, device="cuda")
    d_qkv = torch.full((S, T, nq), 7.0, dtype=bf, device="cuda")
    lse = torch.zeros(S, H, T, dtype=torch.float32, device="cuda")
    delta = torch.zeros(S, H, T, dtype=torch.float32, device="cuda")
    args = B.attn_core_args(B.BF16, S, n_seqs, N, H, kv_max, dh, nh, nkv, qkv=qkv, out=out, lse=lse, d_out=d_out,
                            d_qkv=d_qkv, delta=delta, **extra)
    B.twist_attn_core_fwd(args)
    B.twist_attn_core_bwd(args)
    torch.cuda.synchronize()
    assert B.twist_device_status() == 0
    for s in range(S):
        kc = int(kv_count[s]) * dh
        # oracle layout has no padding: [Q | K of the kept groups | V of the kept groups]
        Z = np.concatenate([QKV[s][:, :a], QKV[s][:, a:a + kc], QKV[s][:, a + kvw:a + kvw + kc]], axis=1).astype(np.float64)
        want = o.attn_core_fwd(Z, n_seqs, N, dh, head_kv[s], kc, lowp=True)
        assert rel_fro(host(out[s]), want) < GEMM_TOL, ("out", s)
        # teacher-forced backward: the oracle differentiates at the same inputs
        dZ = o.attn_core_bwd(dA[s].astype(np.float64), Z, n_seqs, N, dh, head_kv[s], kc, lowp=True)
        got = host(d_qkv[s])
        got_z = np.concatenate([got[:, :a], got[:, a:a + kc], got[:, a + kvw:a + kvw + kc]], axis=1)
        for name, cols in (("dq", slice(0, a)), ("dk", slice(a, a + kc)), ("dv", slice(a + kc, a + 2 * kc))):
            # a gradient that is exactly zero (one visible key: dS = P (dP - delta) = 0) is met up to the rounding of
            # delta, so the error is measured against the larger of its norm and a sliver of the incoming gradient's
            err = np.linalg.norm(got_z[:, cols] - dZ[:, cols])
            assert err < GEMM_TOL * max(np.linalg.norm(dZ[:, cols]), 1e-3 * np.linalg.norm(dA[s])), (name, s)
        assert np.all(got[:, a + kc:a + kvw] == 0) and np.all(got[:, a + kvw + kc:] == 0)     # padding columns
        # log-sum-exp of the first position of every sequence: a single score
        for b in range(n_seqs):
            for hq in range(H):
                g = head_kv[s][hq]
                q0 = Z[b * N, hq * dh:(hq + 1) * dh]
                k0 = Z[b * N, a + g * dh:a + (g + 1) * dh]
                assert abs(lse[s, hq, b * N].item() - q0 @ k0 / np.sqrt(dh)) < 1e-3 * max(1.0, abs(q0 @ k0))


def test_skip_connection_epilogues(B):
    """y = residual + alpha * hh W_down, dx = residual + dpre W_gu, O projection and QKV backward likewise."""
    bf, dtype = torch.bfloat16, I.DTYPE_BF16
    S, T, d, f, n = 2, 200, 328, 344, 136
    kind, alpha = I.FFN_SWIGLU, 1.7
    X = I.normal(91, 1, (S, T, d), 1.0, dtype)
    Wgu = I.normal(91, 2, (S, 2 * f, d), 0.05, dtype)
    Wd = I.normal(91, 3, (S, f, d), 0.05, dtype)
    R = I.normal(91, 4, (S, T, d), 1.0, dtype)
    dY = I.normal(91, 5, (S, T, d), 1e-2, dtype)
    R2 = I.normal(91, 6, (S, T, d), 1e-2, dtype)
    t = lambda *s: torch.zeros(*s, dtype=bf, device="cuda")
    pre, hh, y, dpre, dx = t(S, T, 2 * f), t(S, T, f), t(S, T, d), t(S, T, 2 * f), t(S, T, d)
    a = B.ffn_args(kind, dtype, S, T, d, f, alpha, 0.0, x=dev(X, bf), w_gu=dev(Wgu, bf), w_down=dev(Wd, bf), pre=pre,
                   hh=hh, y=y, dy=dev(dY, bf), dpre=dpre, dx=dx, y_residual=dev(R, bf), dx_residual=dev(R2, bf))
    B.twist_subnet_ffn_fwd(a)
    B.twist_subnet_ffn_bwd(a)
    W = I.normal(92, 1, (S, n, d), 0.05, dtype)
    Ain = I.normal(92, 2, (S, T, n), 1.0, dtype)
    dQ = I.normal(92, 3, (S, T, n), 1e-2, dtype)
    out, d_in = t(S, T, d), t(S, T, d)
    B.twist_subnet_attn_proj_fwd(B.proj_args(B.PROJ_O, dtype, S, T, d, n, alpha, 0.0, in_=dev(Ain, bf), w=dev(W, bf),
                                             out=out, out_residual=dev(R, bf)))
    B.twist_subnet_attn_proj_bwd(B.proj_args(B.PROJ_QKV, dtype, S, T, d, n, 1.0, 0.0, in_=dev(X, bf), w=dev(W, bf),
                                             d_out=dev(dQ, bf), d_in=d_in, d_in_residual=dev(R2, bf)))
    torch.cuda.synchronize()
    assert B.twist_device_status() == 0
    for s in range(S):
        f64 = lambda v: v[s].astype(np.float64)
        Yw, saved = o.ffn_fwd(f64(X), f64(Wgu)[f:], f64(Wgu)[:f], f64(Wd), kind, alpha, True, residual=f64(R))
        dXw, _, _, _ = o.ffn_bwd(f64(dY), f64(X), saved, f64(Wgu)[f:], f64(Wgu)[:f], f64(Wd), kind, alpha, True,
                                 residual=f64(R2))
        assert rel_fro(host(y[s]), Yw) < GEMM_TOL
        assert rel_fro(host(y[s]) - f64(R), Yw - f64(R)) < GEMM_TOL          # the block's own contribution
        assert rel_fro(host(dx[s]), dXw) < GEMM_TOL
        assert rel_fro(host(out[s]), o.o_fwd(f64(Ain), f64(W), alpha, True, residual=f64(R))) < GEMM_TOL
        assert rel_fro(host(d_in[s]), o.qkv_bwd(f64(dQ), f64(X), f64(W), True, residual=f64(R2))[0]) < GEMM_TOL


@pytest.mark.parametrize("cfg,dims,n_seqs,extra", [
    (2, dict(d_model=192, d_ff=528, d_head=16, tokens=192, n_layers=2, local_steps=2), 2, {}),     # GELU, 12 heads keep 6
    (3, dict(d_model=256, d_ff=688, d_head=8, tokens=200, n_layers=3, local_steps=2), 2, {}),      # SwiGLU, GQA 32 heads / 4 groups
    # the pre-LN layer of App. A (both layer normalisations, their parameters trained and averaged)
    # (a learning rate at which the change of gamma / b is well above the fp32 spacing of their values)
    (2, dict(d_model=192, d_ff=528, d_head=16, tokens=192, n_layers=2, local_steps=2), 2, dict(layer_norm=True, lr=1.0)),
    (3, dict(d_model=256, d_ff=688, d_head=8, tokens=200, n_layers=3, local_steps=2), 2,
     dict(layer_norm=True, optimizer="adam", lr=1e-2, adam_eps=3e-3)),
    # shared first and last layers (Sec. 5 Setup: N_sub = N_full there), with and without the normalisations
    (3, dict(d_model=256, d_ff=688, d_head=8, tokens=200, n_layers=3, local_steps=2), 2, dict(shared_layers=(0, 2))),
    (2, dict(d_model=192, d_ff=528, d_head=16, tokens=192, n_layers=3, local_steps=1), 2,
     dict(shared_layers=(2,), layer_norm=True, lr=1.0)),
])
def test_stack_round_of_a_scaled_twin_matches_the_oracle(B, cfg, dims, n_seqs, extra):
    from paper_2511_03983_b200.engine import StackEngine
    w = replace(I.scaled_twin(I.PRESETS[cfg], **dims), **extra)
    seq_len = w.tokens // n_seqs
    eng = StackEngine(w, n_seqs, seq_len, keep_f32_full=True)
    mats = {"gate": I.MAT_GATE, "up": I.MAT_UP, "down": I.MAT_DOWN, "qkv": I.MAT_QKV, "o": I.MAT_O}
    full_np = []
    for l in range(w.n_layers):
        layer = {m: I.weight(w, l, mats[m]) for m in eng.full}
        for m, v in layer.items():
            eng.full[m][l].copy_(dev(v, torch.bfloat16))
        if w.layer_norm:
            for n in I.LN_PARAMS:
                layer[n] = I.ln_param(w, l, n)
                eng.full_ln[n][l].copy_(dev(layer[n]))
        full_np.append(layer)
    store = {}
    for k in range(w.local_steps):
        for kind, dst in ((I.BATCH_X, eng.X), (I.BATCH_TGT_D, eng.Td)):
            arr = np.stack([I.batch(w, kind, 0, s, k, w.d_model) for s in range(w.n_subnets)])
            store[(kind, k)] = arr
            dst.append(dev(arr, torch.bfloat16))
    eng.run_round(0)
    torch.cuda.synchronize()
    assert B.twist_device_status() == 0
    full64 = [{m: v.astype(np.float64) for m, v in layer.items()} for layer in full_np]
    new, bps, losses = o.round_stack(w, full64, lambda kind, rnd, s, k, width: store[(kind, k)][s], 0, n_seqs, seq_len, True)
    got_loss = eng.stack_loss[: w.local_steps].cpu().numpy()
    want_loss = np.array(losses).T
    assert np.allclose(got_loss, want_loss, rtol=2e-2), (got_loss, want_loss)
    for l in range(w.n_layers):
        assert np.array_equal(eng.bufs[eng.kind_of(l)]["idx_ffn"][l].cpu().numpy(), bps[l]["ffn"])
        assert np.array_equal(eng.bufs[eng.kind_of(l)]["idx_head"][l].cpu().numpy(), bps[l]["head"])
        if l in w.shared_layers:
            assert bps[l]["ffn"].shape[1] == w.n_ffn_blocks and bps[l]["head"].shape[1] == w.n_heads
        for m in eng.full:
            res = eng.full_f32[m][l].cpu().numpy().astype(np.float64)
            dw, dg = new[l][m] - full64[l][m], res - full64[l][m]
            assert rel_fro(dg, dw) < 5e-2, (l, m, rel_fro(dg, dw))
        if w.layer_norm:
            for n in I.LN_PARAMS:
                res = eng.full_ln[n][l].cpu().numpy().astype(np.float64)
                dw, dg = new[l][n] - full64[l][n], res - full64[l][n]
                # stored in fp32: half a spacing of the values themselves is the floor of what a difference can show
                floor = 2.0 ** -24 * np.linalg.norm(np.maximum(np.abs(full64[l][n]), 2.0 ** -6)) / np.linalg.norm(dw)
                assert rel_fro(dg, dw) < 5e-2 + floor, (l, n, rel_fro(dg, dw), floor)


@pytest.mark.parametrize("mode", ["stack", "blockwise"])
def test_rounds_are_bit_reproducible(B, mode):
    """No kernel of the path uses atomics or an order that depends on scheduling (one writer per result, fixed
    summation orders): the same round from the same state gives the same bits - weights, masters and losses.
    The twin uses d_head = 64, so the STACK round runs the tensor-core attention kernels."""
    from paper_2511_03983_b200.engine import RoundEngine, StackEngine
    w = I.scaled_twin(I.PRESETS[3], d_model=256, d_ff=688, d_head=64, tokens=512, n_layers=2, local_steps=2)
    eng = StackEngine(w, 2, 256, keep_f32_full=True) if mode == "stack" else RoundEngine(w, keep_f32_full=True)
    mats = {"gate": I.MAT_GATE, "up": I.MAT_UP, "down": I.MAT_DOWN, "qkv": I.MAT_QKV, "o": I.MAT_O}
    init = {m: torch.stack([dev(I.weight(w, l, mats[m]), torch.bfloat16) for l in range(w.n_layers)]) for m in eng.full}
    for k in range(w.local_steps):
        widths = [(I.BATCH_X, w.d_model, eng.X), (I.BATCH_TGT_D, w.d_model, eng.Td)]
        if mode == "blockwise":
            widths += [(I.BATCH_TGT_QKV, eng.nq, eng.Tq), (I.BATCH_A, eng.a_sub, eng.A)]
        for kind, width, dst in widths:
            dst.append(dev(np.stack([I.batch(w, kind, 0, s, k, width) for s in range(w.n_subnets)]), torch.bfloat16))
    runs = []
    for _ in range(2):
        for m in eng.full:
            eng.full[m].copy_(init[m])
            eng.full_f32[m].copy_(init[m].float())
        eng.run_round(0)
        torch.cuda.synchronize()
        assert B.twist_device_status() == 0
        loss = eng.stack_loss if mode == "stack" else eng.loss
        runs.append(({m: v.clone() for m, v in eng.full.items()}, {m: v.clone() for m, v in eng.full_f32.items()},
                     loss.clone()))
    (a16, a32, la), (b16, b32, lb) = runs
    assert any(not torch.equal(a16[m], init[m]) for m in a16)          # the round did train
    for m in a16:
        assert torch.equal(a16[m], b16[m]) and torch.equal(a32[m], b32[m]), m
    assert torch.equal(la, lb)


@pytest.mark.parametrize("head_keep,ffn_ratio", [(16, 0.5), (24, 0.75)])
def test_extracted_subnets_forward_only_at_any_ratio(B, head_keep, ffn_ratio):
    """Sec. 4.2: subnets extracted with the sampler's procedure at a ratio that need not be the training one run
    forward only through the whole chained stack with their own scales; losses match the oracle's stack forward."""
    from paper_2511_03983_b200.engine import StackEngine
    base = I.scaled_twin(I.PRESETS[3], d_model=256, d_ff=688, d_head=8, tokens=200, n_layers=2, local_steps=1)
    w = replace(base, head_keep=head_keep, ffn_keep=int(base.n_ffn_blocks * ffn_ratio) // 8 * 8)
    n_seqs, seq_len = 2, 100
    eng = StackEngine(w, n_seqs, seq_len)
    mats = {"gate": I.MAT_GATE, "up": I.MAT_UP, "down": I.MAT_DOWN, "qkv": I.MAT_QKV, "o": I.MAT_O}
    full_np = []
    for l in range(w.n_layers):
        layer = {m: I.weight(w, l, mats[m]) for m in eng.full}
        for m, v in layer.items():
            eng.full[m][l].copy_(dev(v, torch.bfloat16))
        full_np.append(layer)
    X = np.stack([I.batch(w, I.BATCH_X, 0, s, 0, w.d_model) for s in range(w.n_subnets)])
    Tg = np.stack([I.batch(w, I.BATCH_TGT_D, 0, s, 0, w.d_model) for s in range(w.n_subnets)])
    eng.X.append(dev(X, torch.bfloat16))
    eng.Td.append(dev(Tg, torch.bfloat16))
    before = {m: v.clone() for m, v in eng.full.items()}
    eng.extract(0)
    got = eng.evaluate(0).cpu().numpy()
    torch.cuda.synchronize()
    assert B.twist_device_status() == 0
    for m in before:                                      # inference leaves the model alone
        assert torch.equal(before[m], eng.full[m])
    for s in range(w.n_subnets):
        bps = [o.layer_blueprints(w, 0, l) for l in range(w.n_layers)]
        layers = [{m: v.astype(np.float64) for m, v in o.gather_layer(w, full_np[l], bps[l], s).items()}
                  for l in range(w.n_layers)]
        head_kv = [o.head_kv_positions(bps[l], w, s) for l in range(w.n_layers)]
        out = o.stack_fwd(w, layers, head_kv, X[s].astype(np.float64), n_seqs, seq_len, True)
        y = out[0] if isinstance(out, tuple) else out
        want, _ = o.mse(y, Tg[s].astype(np.float64), True)
        assert abs(got[s] - want) <= 2e-2 * want, (s, got[s], want)
