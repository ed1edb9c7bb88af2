"""Parity at the full sizes of the 7B-shaped workload (S=8, T=32768, d=4096, F=11008 -> f'=2752,
8 of 32 heads) and of the TinyLlama-shaped one (S=4, T=32768, d=2048, F=5632 -> f'=2816, 16 of 32 heads in
4 KV groups), in the launch configuration bench.py times, on outputs the oracle can compute one
by one: sampled token rows of every activation, sampled weight rows of every fused-SGD update
(full-length contractions over all 32768 tokens), whole blueprints, whole gathered slices of
sampled subnets, and the whole aggregate.  Inputs are seeded draws made on the device; the oracle
reads the same bytes.  One layer, one local step."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from fp32_mirror import aggregate_f32
from oracle import twist_oracle as o
from paper_2511_03983_b200 import inputs as I

pytestmark = pytest.mark.gpu

TOL = 2e-2
SUBNETS = {4: (1, 6), 3: (0, 3), 2: (0, 2)}   # subnets whose activations / updates are checked, per workload
N_ROWS, N_WROWS = 40, 12  # sampled token rows, sampled weight rows


def rel_fro(got, want):
    return float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-300))


def f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


@pytest.fixture(scope="module", params=[4, 3, 2])
def setup(request):
    from paper_2511_03983_b200 import binding as B
    from paper_2511_03983_b200.engine import RoundEngine
    B.lib()
    w = replace(I.PRESETS[request.param], n_layers=1, local_steps=1)
    eng = RoundEngine(w, keep_f32_full=True, lazy_master=False)      # the tests below call the C ABI themselves
    gen = torch.Generator(device="cuda")
    gen.manual_seed(w.seed_w)
    for m, v in eng.full.items():
        v[0].copy_((torch.randn(v[0].shape, generator=gen, device="cuda") * 0.02).to(torch.bfloat16))
    gen.manual_seed(w.seed_x)
    S, T, d = w.n_subnets, w.tokens, w.d_model
    rnd = lambda width, std=1.0: (torch.randn(S, T, width, generator=gen, device="cuda") * std).to(torch.bfloat16)
    eng.X, eng.Td, eng.Tq, eng.A = [rnd(d)], [rnd(d)], [rnd(eng.nq)], [rnd(eng.a_sub)]
    full_np = {m: v[0].float().cpu().numpy() for m, v in eng.full.items()}
    eng.sample_masks(0)
    eng.gather_layer(0)
    torch.cuda.synchronize()
    bp = o.layer_blueprints(w, 0, 0)
    rng = np.random.default_rng(5)
    rows = np.sort(rng.choice(T, N_ROWS, replace=False))
    # the device pads K / V to the maximum group count; these workloads keep every group, so the layouts coincide
    assert np.all(bp["kv_count"] == eng.kv_max)
    yield dict(B=B, eng=eng, w=w, full=full_np, bp=bp, rows=rows, rng=rng, gen=gen, rnd=rnd, subnets=SUBNETS[request.param])
    del eng
    torch.cuda.empty_cache()


def test_blueprints_and_index_data_bit_exact(setup):
    eng, w, bp = setup["eng"], setup["w"], setup["bp"]
    assert np.array_equal(eng.idx_ffn[0].cpu().numpy(), bp["ffn"])
    assert np.array_equal(eng.idx_head[0].cpu().numpy(), bp["head"])
    c, _, p = o.cover_and_pos(bp["ffn"], w.n_ffn_blocks)
    assert np.array_equal(eng.cover_ffn[0].cpu().numpy().view(np.uint32), c)
    assert np.array_equal(eng.pos_ffn[0].cpu().numpy(), p)
    c, _, p = o.cover_and_pos(bp["head"], w.n_heads)
    assert np.array_equal(eng.cover_head[0].cpu().numpy().view(np.uint32), c)
    assert np.array_equal(eng.pos_head[0].cpu().numpy(), p)
    assert np.array_equal(eng.kv_idx[0].cpu().numpy(), bp["kv_idx"])
    assert np.array_equal(eng.kv_count[0].cpu().numpy(), bp["kv_count"])


def test_gathered_slices_bit_exact(setup):
    eng, w, bp, full = setup["eng"], setup["w"], setup["bp"], setup["full"]
    f = w.f_sub
    for s in setup["subnets"]:
        sl = o.gather_layer(w, full, bp, s)
        w_gu = np.concatenate([sl["gate"], sl["up"]]) if "gate" in sl else sl["up"]
        want = {"w_gu": w_gu, "w_down": sl["down"], "w_qkv": sl["qkv"], "w_o": sl["o"]}
        for name, arr in want.items():
            got16 = getattr(eng, name)[s].float().cpu().numpy()
            got32 = getattr(eng, name + "_m")[s].cpu().numpy()
            assert np.array_equal(got16.view(np.uint32), arr.view(np.uint32)), (s, name)
            assert np.array_equal(got32.view(np.uint32), arr.view(np.uint32)), (s, name, "master")


def _sl64(setup, s):
    sl = o.gather_layer(setup["w"], setup["full"], setup["bp"], s)
    return {m: v.astype(np.float64) for m, v in sl.items()}


def test_ffn_forward_backward_sampled(setup):
    B, eng, w, rows, rng = setup["B"], setup["eng"], setup["w"], setup["rows"], setup["rng"]
    S, T, d, f = w.n_subnets, w.tokens, w.d_model, w.f_sub
    lr = w.lr
    dY = setup["rnd"](d, 1e-4)
    a = B.ffn_args(w.ffn_kind, w.dtype, S, T, d, f, eng.alpha_f, lr, x=eng.X[0], w_gu=eng.w_gu, w_down=eng.w_down,
                   w_gu_master=eng.w_gu_m, w_down_master=eng.w_down_m, pre=eng.pre, hh=eng.hh, y=eng.y, dy=dY,
                   dpre=eng.dpre, dx=eng.dx)
    B.twist_subnet_ffn_fwd(a)
    B.twist_subnet_ffn_bwd(a)
    torch.cuda.synchronize()
    assert B.twist_device_status() == 0
    for s in setup["subnets"]:
        sl = _sl64(setup, s)
        X = f64(eng.X[0][s])
        dYs = f64(dY[s])
        # sampled token rows: every activation of the chain
        gated = "gate" in sl                      # SwiGLU: gate and up matrices; otherwise one matrix
        gate = sl["gate"] if gated else None
        Yw, saved = o.ffn_fwd(X[rows], sl["up"], gate, sl["down"], w.ffn_kind, eng.alpha_f, True)
        dXw, _, _, _ = o.ffn_bwd(dYs[rows], X[rows], saved, sl["up"], gate, sl["down"], w.ffn_kind, eng.alpha_f, True)
        r = torch.from_numpy(rows).cuda()
        pre_w = np.concatenate([saved["G"], saved["U"]], axis=1) if gated else saved["U"]
        assert rel_fro(f64(eng.pre[s][r]), pre_w) < TOL
        assert rel_fro(f64(eng.hh[s][r]), saved["Hh"]) < TOL
        assert rel_fro(f64(eng.y[s][r]), Yw) < TOL
        assert rel_fro(f64(eng.dx[s][r]), dXw) < TOL
        # sampled neurons: weight gradients with the full-length contraction over all T tokens; the
        # FFN is separable per neuron except for Y and dX, so restricting the slices to J is exact
        J = np.sort(rng.choice(f, N_WROWS, replace=False))
        gateJ = sl["gate"][J] if gated else None
        _, savedJ = o.ffn_fwd(X, sl["up"][J], gateJ, sl["down"][J], w.ffn_kind, eng.alpha_f, True)
        _, dWu, dWg, dWd = o.ffn_bwd(dYs, X, savedJ, sl["up"][J], gateJ, sl["down"][J], w.ffn_kind, eng.alpha_f, True)
        Jt = torch.from_numpy(J).cuda()
        upd_up = f64(eng.w_gu_m[s][Jt + (f if gated else 0)]) - sl["up"][J]
        upd_down = f64(eng.w_down_m[s][Jt]) - sl["down"][J]
        if gated:
            upd_gate = f64(eng.w_gu_m[s][Jt]) - sl["gate"][J]
            assert rel_fro(upd_gate, -lr * dWg) < TOL, (s, "gate")
        assert rel_fro(upd_up, -lr * dWu) < TOL, (s, "up")
        assert rel_fro(upd_down, -lr * dWd) < TOL, (s, "down")
        assert torch.equal(eng.w_gu[s][Jt], eng.w_gu_m[s][Jt].to(torch.bfloat16))


def test_projections_forward_backward_sampled(setup):
    B, eng, w, rows, rng = setup["B"], setup["eng"], setup["w"], setup["rows"], setup["rng"]
    S, T, d = w.n_subnets, w.tokens, w.d_model
    lr = w.lr
    dQ = setup["rnd"](eng.nq, 1e-4)
    dYo = setup["rnd"](d, 1e-4)
    aq = B.proj_args(B.PROJ_QKV, w.dtype, S, T, d, eng.nq, 1.0, lr, in_=eng.X[0], w=eng.w_qkv, w_master=eng.w_qkv_m,
                     out=eng.qkv_out, d_out=dQ, d_in=eng.dx)
    B.twist_subnet_attn_proj_fwd(aq)
    B.twist_subnet_attn_proj_bwd(aq)
    ao = B.proj_args(B.PROJ_O, w.dtype, S, T, d, eng.a_sub, eng.alpha_a, lr, in_=eng.A[0], w=eng.w_o, w_master=eng.w_o_m,
                     out=eng.y, d_out=dYo, d_in=eng.da)
    B.twist_subnet_attn_proj_fwd(ao)
    B.twist_subnet_attn_proj_bwd(ao)
    torch.cuda.synchronize()
    assert B.twist_device_status() == 0
    r = torch.from_numpy(rows).cuda()
    for s in setup["subnets"]:
        sl = _sl64(setup, s)
        X, A = f64(eng.X[0][s]), f64(eng.A[0][s])
        dQs, dYs = f64(dQ[s]), f64(dYo[s])
        assert rel_fro(f64(eng.qkv_out[s][r]), o.qkv_fwd(X[rows], sl["qkv"], True)) < TOL
        assert rel_fro(f64(eng.dx[s][r]), o.qkv_bwd(dQs[rows], X[rows], sl["qkv"], True)[0]) < TOL
        assert rel_fro(f64(eng.y[s][r]), o.o_fwd(A[rows], sl["o"], eng.alpha_a, True)) < TOL
        assert rel_fro(f64(eng.da[s][r]), o.o_bwd(dYs[rows], A[rows], sl["o"], eng.alpha_a, True)[0]) < TOL
        J = np.sort(rng.choice(eng.nq, N_WROWS, replace=False))
        _, dWq = o.qkv_bwd(dQs[:, J], X, sl["qkv"][J], True)
        assert rel_fro(f64(eng.w_qkv_m[s][torch.from_numpy(J).cuda()]) - sl["qkv"][J], -lr * dWq) < TOL
        J = np.sort(rng.choice(eng.a_sub, N_WROWS, replace=False))
        _, dWo = o.o_bwd(dYs, A[:, J], sl["o"][J], eng.alpha_a, True)
        assert rel_fro(f64(eng.w_o_m[s][torch.from_numpy(J).cuda()]) - sl["o"][J], -lr * dWo) < TOL


def test_aggregate_whole_layer(setup):
    eng, w, bp, full, gen = setup["eng"], setup["w"], setup["bp"], setup["full"], setup["gen"]
    S = w.n_subnets
    # seeded "trained" masters (the oracle reads the same bytes)
    for m in (eng.w_gu_m, eng.w_down_m, eng.w_qkv_m, eng.w_o_m):
        m.copy_(torch.randn(m.shape, generator=gen, device="cuda") * 0.02)
    eng.aggregate_layer(0)
    torch.cuda.synchronize()
    f, a_sub, dh, H, Hkv = w.f_sub, eng.a_sub, w.d_head, w.n_heads, w.n_kv_heads
    kvw = eng.kv_max * dh
    gu, down, qkv, wo = (t.cpu().numpy().astype(np.float64) for t in (eng.w_gu_m, eng.w_down_m, eng.w_qkv_m, eng.w_o_m))
    kvs = [bp["kv_idx"][s][: bp["kv_count"][s]] for s in range(S)]
    gated = "gate" in full
    cases = ([("gate", [gu[s, :f] for s in range(S)], bp["ffn"], 1, 0, slice(0, w.d_ff))] if gated else []) + [
        ("up", [gu[s, (f if gated else 0):] for s in range(S)], bp["ffn"], 1, 0, slice(0, w.d_ff)),
        ("down", [down[s] for s in range(S)], bp["ffn"], 1, 0, slice(0, w.d_ff)),
        ("qkv", [qkv[s, :a_sub] for s in range(S)], bp["head"], dh, 0, slice(0, H * dh)),
        ("qkv", [qkv[s, a_sub:a_sub + kvw] for s in range(S)], kvs, dh, H * dh, slice(H * dh, (H + Hkv) * dh)),
        ("qkv", [qkv[s, a_sub + kvw:] for s in range(S)], kvs, dh, (H + Hkv) * dh, slice((H + Hkv) * dh, (H + 2 * Hkv) * dh)),
        ("o", [wo[s] for s in range(S)], bp["head"], dh, 0, slice(0, H * dh)),
    ]
    for name, subs, blue, br, off, rows in cases:
        before = full[name].astype(np.float64)
        want = o.aggregate(before, subs, blue, br, row_offset=off)[rows]
        mag = o.aggregate(np.abs(before), [np.abs(v) for v in subs], blue, br, row_offset=off)[rows]
        got = eng.full_f32[name][0].cpu().numpy().astype(np.float64)[rows]
        held = np.any(want != before[rows], axis=1)
        assert held.any()
        err = np.abs(got[held] - want[held]) / np.maximum(mag[held], 1e-30)
        assert err.max() <= 1e-6, (name, err.max())
        # bit for bit the fp32 evaluation in the fixed order (ascending subnets, one IEEE division)
        mirror = aggregate_f32(full[name], [v.astype(np.float32) for v in subs], blue, br, row_offset=off)[rows]
        got32 = eng.full_f32[name][0].cpu().numpy()[rows]
        assert np.array_equal(got32[held].view(np.uint32), mirror[held].view(np.uint32)), name
        shadow = eng.full[name][0][rows]
        assert torch.equal(shadow[torch.from_numpy(held).cuda()],
                           eng.full_f32[name][0][rows][torch.from_numpy(held).cuda()].to(torch.bfloat16))


def test_fused_loss_at_full_size(setup):
    """The bench's forward call: loss and dY formed in the output epilogue, y not stored.  dY must equal, bit for
    bit, what the stand-alone loss kernel gives on the stored y; sampled rows of it and the loss match the oracle."""
    B, eng, w, rows = setup["B"], setup["eng"], setup["w"], setup["rows"]
    S, T, d, f = w.n_subnets, w.tokens, w.d_model, w.f_sub
    # earlier tests trained the slices and aggregated into the full model: restore the seeded model and gather again
    for m, v in setup["full"].items():
        eng.full[m][0].copy_(torch.from_numpy(v).to(torch.bfloat16))
    eng.gather_layer(0)
    common = dict(x=eng.X[0], w_gu=eng.w_gu, w_down=eng.w_down, pre=eng.pre, hh=eng.hh)
    loss_a = torch.zeros(S, dtype=torch.float32, device="cuda")
    loss_b = torch.zeros(S, dtype=torch.float32, device="cuda")
    dy_b = torch.empty_like(eng.dy)
    B.twist_subnet_ffn_fwd(B.ffn_args(w.ffn_kind, w.dtype, S, T, d, f, eng.alpha_f, 0.0, y=eng.y, **common))
    B.twist_mse_fwd_bwd(eng.y, eng.Td[0], eng.dy, loss_a, S, T, d, None, 0, 0, w.dtype, eng.ws)
    B.twist_subnet_ffn_fwd(B.ffn_args(w.ffn_kind, w.dtype, S, T, d, f, eng.alpha_f, 0.0, y=None, dy=dy_b, tgt=eng.Td[0],
                                      loss=loss_b, loss_ws=eng.ws, **common))
    torch.cuda.synchronize()
    assert B.twist_device_status() == 0
    assert torch.equal(eng.dy, dy_b)
    assert torch.allclose(loss_a, loss_b, rtol=1e-5, atol=0)
    r = torch.from_numpy(rows).cuda()
    for s in setup["subnets"]:
        sl = _sl64(setup, s)
        Yw, _ = o.ffn_fwd(f64(eng.X[0][s][r]), sl["up"], sl.get("gate"), sl["down"], w.ffn_kind, eng.alpha_f, True)
        want_dy = o.round_bf16(2.0 * (Yw - f64(eng.Td[0][s][r])) / (T * d))
        assert rel_fro(f64(dy_b[s][r]), want_dy) < TOL
        # the reduction: mean squared error over ALL T x d elements, recomputed in fp64 from the stored y
        diff = eng.y[s].double() - eng.Td[0][s].double()
        want_loss = float((diff * diff).sum().item()) / (T * d)
        assert abs(loss_b[s].item() - want_loss) <= 1e-5 * want_loss


@pytest.mark.parametrize("cfg", [2, 3])
def test_attention_core_at_stack_workload_sizes(cfg):
    """The softmax core at the full sizes of the stack-shaped workloads (8 x 1024 tokens, 6 of 12 heads; 16 x 2048
    tokens, 16 of 32 heads in 4 KV groups).  The oracle evaluates whole (subnet, sequence) pairs for the heads of a
    sampled KV position: every output row, dQ, and the dK / dV of that position summed over its heads."""
    from paper_2511_03983_b200 import binding as B
    B.lib()
    w = I.PRESETS[cfg]
    S, n_seqs, N, H, dh = w.n_subnets, w.n_seqs, w.tokens // w.n_seqs, w.head_keep, w.d_head
    T = w.tokens
    bp = o.layer_blueprints(w, 0, 0)
    gqa = w.n_kv_heads != w.n_heads
    kv_max = min(w.n_kv_heads, H)
    a, kvw = H * dh, kv_max * dh
    nq = a + 2 * kvw
    gen = torch.Generator(device="cuda")
    gen.manual_seed(77 + cfg)
    qkv = torch.randn(S, T, nq, generator=gen, device="cuda").to(torch.bfloat16)
    d_out = torch.randn(S, T, a, generator=gen, device="cuda").to(torch.bfloat16)
    out = torch.zeros(S, T, a, dtype=torch.bfloat16, device="cuda")
    d_qkv = torch.zeros(S, T, nq, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(S, H, T, dtype=torch.float32, device="cuda")
    delta = torch.zeros(S, H, T, dtype=torch.float32, device="cuda")
    extra = {}
    if gqa:
        _, _, kv_pos = o.cover_and_pos(bp["kv_idx"], w.n_kv_heads, counts=bp["kv_count"])
        extra = dict(head_idx=torch.from_numpy(bp["head"].astype(np.int32)).cuda(),
                     kv_pos=torch.from_numpy(kv_pos.astype(np.int32)).cuda(),
                     kv_count=torch.from_numpy(bp["kv_count"].astype(np.int32)).cuda())
    args = B.attn_core_args(B.BF16, S, n_seqs, N, H, kv_max, dh, w.n_heads, w.n_kv_heads, qkv=qkv, out=out, lse=lse,
                            d_out=d_out, d_qkv=d_qkv, delta=delta, **extra)
    B.twist_attn_core_fwd(args)
    B.twist_attn_core_bwd(args)
    torch.cuda.synchronize()
    assert B.twist_device_status() == 0
    rng = np.random.default_rng(11)
    for s, b in ((0, 0), (S - 1, n_seqs - 1)):
        head_kv = o.head_kv_positions(bp, w, s) if gqa else np.arange(H)
        g = int(rng.choice(np.unique(head_kv)))
        heads = [hq for hq in range(H) if head_kv[hq] == g]
        rows = slice(b * N, (b + 1) * N)
        # a sub-problem with only these heads and this one KV position
        qcols = np.concatenate([np.arange(hq * dh, (hq + 1) * dh) for hq in heads])
        kcols = np.arange(a + g * dh, a + (g + 1) * dh)
        vcols = kcols + kvw
        Z = f64(qkv[s, rows])[:, np.concatenate([qcols, kcols, vcols])]
        dA = f64(d_out[s, rows])[:, qcols]
        hk = [0] * len(heads)
        want = o.attn_core_fwd(Z, 1, N, dh, hk, dh, True)
        assert rel_fro(f64(out[s, rows])[:, qcols], want) < TOL
        dZ = o.attn_core_bwd(dA, Z, 1, N, dh, hk, dh, True)
        got = f64(d_qkv[s, rows])[:, np.concatenate([qcols, kcols, vcols])]
        nqh = len(qcols)
        assert rel_fro(got[:, :nqh], dZ[:, :nqh]) < TOL, "dq"
        assert rel_fro(got[:, nqh:nqh + dh], dZ[:, nqh:nqh + dh]) < TOL, "dk"
        assert rel_fro(got[:, nqh + dh:], dZ[:, nqh + dh:]) < TOL, "dv"


# ---------------------------------------------------------------------------------------------------------------
# The gather / aggregate sweep workload (7B FFN shapes, IID masks, 1024 tokens per subnet) at full block counts:
# the cell with rows no subnet holds (S = 2, keep 1/4), the cell with up to 16 subnets per row and the widest
# slices (S = 16, keep 3/4: f' = 8256), and the f' = 5504 cell (S = 4, keep 1/2).  One layer.
# ---------------------------------------------------------------------------------------------------------------

CELLS5 = [(2, 0.25), (16, 0.75), (4, 0.5)]


@pytest.fixture(scope="module", params=CELLS5, ids=lambda c: f"S{c[0]}-keep{c[1]}")
def cell(request):
    from paper_2511_03983_b200 import binding as B
    from paper_2511_03983_b200.engine import RoundEngine
    B.lib()
    S, keep = request.param
    base = I.PRESETS[5]
    w = replace(base, n_subnets=S, ffn_keep=int(np.floor(keep * base.n_ffn_blocks)), n_layers=1, local_steps=1,
                name=f"cfg5-S{S}-keep{keep}")
    eng = RoundEngine(w, keep_f32_full=True, lazy_master=False)      # the tests below call the C ABI themselves
    gen = torch.Generator(device="cuda")
    gen.manual_seed(w.seed_w + S)
    for m, v in eng.full.items():
        v[0].copy_((torch.randn(v[0].shape, generator=gen, device="cuda") * 0.02).to(torch.bfloat16))
    for m in eng.full:                    # the fp32 result starts as a recognisable value: untouched rows keep it
        eng.full_f32[m].fill_(123.0)
    T, d = w.tokens, w.d_model
    rnd = lambda width, std=1.0: (torch.randn(S, T, width, generator=gen, device="cuda") * std).to(torch.bfloat16)
    eng.X, eng.Td = [rnd(d)], [rnd(d)]
    full_np = {m: v[0].float().cpu().numpy() for m, v in eng.full.items()}
    eng.sample_masks(0)
    eng.gather_layer(0)
    torch.cuda.synchronize()
    bp = o.layer_blueprints(w, 0, 0)
    yield dict(B=B, eng=eng, w=w, full=full_np, bp=bp, gen=gen, rnd=rnd, rng=np.random.default_rng(7 + S))
    del eng
    torch.cuda.empty_cache()


def test_sweep_cell_blueprints_bit_exact(cell):
    eng, w, bp = cell["eng"], cell["w"], cell["bp"]
    assert np.array_equal(eng.idx_ffn[0].cpu().numpy(), bp["ffn"])
    c, count, p = o.cover_and_pos(bp["ffn"], w.n_ffn_blocks)
    assert np.array_equal(eng.cover_ffn[0].cpu().numpy().view(np.uint32), c)
    assert np.array_equal(eng.pos_ffn[0].cpu().numpy(), p)
    if w.n_subnets == 2:
        assert (count == 0).mean() > 0.4          # independent quarters leave (3/4)^2 of the blocks unheld
    if w.n_subnets == 16:
        assert count.max() == 16                  # some block is held by every subnet


def test_sweep_cell_gathered_slices_bit_exact(cell):
    eng, w, bp, full = cell["eng"], cell["w"], cell["bp"], cell["full"]
    for s in sorted({0, w.n_subnets - 1}):
        sl = o.gather_layer(w, full, bp, s)
        want = {"w_gu": np.concatenate([sl["gate"], sl["up"]]), "w_down": sl["down"]}
        for name, arr in want.items():
            got16 = getattr(eng, name)[s].float().cpu().numpy()
            got32 = getattr(eng, name + "_m")[s].cpu().numpy()
            assert np.array_equal(got16.view(np.uint32), arr.view(np.uint32)), (s, name)
            assert np.array_equal(got32.view(np.uint32), arr.view(np.uint32)), (s, name, "master")


def test_sweep_cell_ffn_forward_backward_sampled(cell):
    B, eng, w, rng = cell["B"], cell["eng"], cell["w"], cell["rng"]
    S, T, d, f = w.n_subnets, w.tokens, w.d_model, w.f_sub
    lr = w.lr
    dY = cell["rnd"](d, 1e-4)
    a = B.ffn_args(w.ffn_kind, w.dtype, S, T, d, f, eng.alpha_f, lr, x=eng.X[0], w_gu=eng.w_gu, w_down=eng.w_down,
                   w_gu_master=eng.w_gu_m, w_down_master=eng.w_down_m, pre=eng.pre, hh=eng.hh, y=eng.y, dy=dY,
                   dpre=eng.dpre, dx=eng.dx)
    B.twist_subnet_ffn_fwd(a)
    B.twist_subnet_ffn_bwd(a)
    torch.cuda.synchronize()
    assert B.twist_device_status() == 0
    rows = np.sort(rng.choice(T, N_ROWS, replace=False))
    r = torch.from_numpy(rows).cuda()
    for s in sorted({0, S - 1}):
        sl = {m: v.astype(np.float64) for m, v in o.gather_layer(w, cell["full"], cell["bp"], s).items()}
        X, dYs = f64(eng.X[0][s]), f64(dY[s])
        Yw, saved = o.ffn_fwd(X[rows], sl["up"], sl["gate"], sl["down"], w.ffn_kind, eng.alpha_f, True)
        dXw, _, _, _ = o.ffn_bwd(dYs[rows], X[rows], saved, sl["up"], sl["gate"], sl["down"], w.ffn_kind, eng.alpha_f, True)
        assert rel_fro(f64(eng.pre[s][r]), np.concatenate([saved["G"], saved["U"]], axis=1)) < TOL
        assert rel_fro(f64(eng.hh[s][r]), saved["Hh"]) < TOL
        assert rel_fro(f64(eng.y[s][r]), Yw) < TOL
        assert rel_fro(f64(eng.dx[s][r]), dXw) < TOL
        J = np.sort(np.concatenate([rng.choice(f, N_WROWS - 2, replace=False), [0, f - 1]]))     # incl. the ragged last tile
        J = np.unique(J)
        _, savedJ = o.ffn_fwd(X, sl["up"][J], sl["gate"][J], sl["down"][J], w.ffn_kind, eng.alpha_f, True)
        _, dWu, dWg, dWd = o.ffn_bwd(dYs, X, savedJ, sl["up"][J], sl["gate"][J], sl["down"][J], w.ffn_kind, eng.alpha_f, True)
        Jt = torch.from_numpy(J).cuda()
        assert rel_fro(f64(eng.w_gu_m[s][Jt]) - sl["gate"][J], -lr * dWg) < TOL, (s, "gate")
        assert rel_fro(f64(eng.w_gu_m[s][Jt + f]) - sl["up"][J], -lr * dWu) < TOL, (s, "up")
        assert rel_fro(f64(eng.w_down_m[s][Jt]) - sl["down"][J], -lr * dWd) < TOL, (s, "down")
        assert torch.equal(eng.w_gu[s][Jt], eng.w_gu_m[s][Jt].to(torch.bfloat16))


def test_sweep_cell_aggregate_whole_layer(cell):
    """The whole layer's aggregate.  The operation is independent per column, so the oracle (float64) and the fp32
    mirror evaluate every row on a sample of columns (all lanes and row spans of the kernel occur among them) and
    every column on a sample of rows: within 1e-6 of the oracle relative to the mean magnitude of the averaged
    values (the (count + 1) 2^-24 bound of the fp32 evaluation where count reaches 16), bit for bit equal to the fp32
    evaluation in the fixed order, and rows nobody holds untouched in both outputs."""
    eng, w, bp, full, gen, rng = cell["eng"], cell["w"], cell["bp"], cell["full"], cell["gen"], cell["rng"]
    S, f, d, F = w.n_subnets, w.f_sub, w.d_model, w.d_ff
    for m in (eng.w_gu_m, eng.w_down_m):
        m.copy_(torch.randn(m.shape, generator=gen, device="cuda") * 0.02)
    before16 = {m: eng.full[m][0].clone() for m in eng.full}
    eng.aggregate_layer(0)
    torch.cuda.synchronize()
    _, count, _ = o.cover_and_pos(bp["ffn"], w.n_ffn_blocks)
    held = count > 0
    cols = np.unique(np.concatenate([rng.choice(d, 254, replace=False), [0, d - 1]]))
    rows = np.unique(np.concatenate([rng.choice(F, 30, replace=False), [0, F - 1]]))
    ct, rt = torch.from_numpy(cols).cuda(), torch.from_numpy(rows).cuda()
    cases = [("gate", eng.w_gu_m[:, :f]), ("up", eng.w_gu_m[:, f:]), ("down", eng.w_down_m)]
    for name, master in cases:
        # (1) every row, sampled columns
        subs32 = master[:, :, ct].cpu().numpy()
        W0 = full[name][:, cols]
        want = o.aggregate(W0.astype(np.float64), [subs32[s].astype(np.float64) for s in range(S)], bp["ffn"], 1)
        mag = o.aggregate(np.abs(W0).astype(np.float64), [np.abs(subs32[s]).astype(np.float64) for s in range(S)],
                          bp["ffn"], 1)
        mirror = aggregate_f32(W0, [subs32[s] for s in range(S)], bp["ffn"], 1)
        got = eng.full_f32[name][0][:, ct].cpu().numpy()
        err = np.abs(got[held].astype(np.float64) - want[held]) / np.maximum(mag[held], 1e-30)
        assert err.max() <= max(1e-6, (count.max() + 1) * 2.0 ** -24), (name, err.max())
        assert np.array_equal(got[held].view(np.uint32), mirror[held].view(np.uint32)), name
        assert np.all(got[~held] == 123.0), name                                  # rows nobody holds: not written
        # (2) sampled rows, every column
        subs_r = []
        kept_rows = []
        for s in range(S):
            pos = np.searchsorted(bp["ffn"][s], rows)
            pos = np.where((pos < f) & (bp["ffn"][s][np.minimum(pos, f - 1)] == rows), pos, -1)
            kept_rows.append(pos)
        got_r = eng.full_f32[name][0][rt].cpu().numpy()
        for i, rr in enumerate(rows):
            holders = [s for s in range(S) if kept_rows[s][i] >= 0]
            if not holders:
                assert np.all(got_r[i] == 123.0)
                continue
            acc = np.zeros(d, dtype=np.float32)
            for s in holders:                                                     # ascending s, float32
                acc = acc + master[s, int(kept_rows[s][i])].cpu().numpy()
            assert np.array_equal(got_r[i].view(np.uint32), (acc / np.float32(len(holders))).view(np.uint32)), (name, rr)
        # the bf16 model: rounded result on held rows, previous bytes elsewhere
        ht = torch.from_numpy(held).cuda()
        assert torch.equal(eng.full[name][0][ht], eng.full_f32[name][0][ht].to(torch.bfloat16))
        assert torch.equal(eng.full[name][0][~ht], before16[name][~ht])
