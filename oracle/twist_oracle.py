"""CPU oracle for one TwIST training round.  TEST INFRASTRUCTURE ONLY.

A plain, slow, obviously-correct numpy implementation (float64 arithmetic) of
what the CUDA hot path computes: Algorithm 1 blueprints, dispatcher gather,
local forward/backward/SGD steps on the dense slices, and the aggregator's
coverage-normalised average.  It shares no code with the CUDA library and does
not import it; only tests, the smoke check and the bench's cpu_baseline leg may
call it.  The product path never routes through this module.

Every function cites the passage of the paper it follows.  TwIST is an
iteration, not a shortcut to a closed form, so each function takes the
algorithm's steps in the paper's order and notation.

Storage convention (a choice of this implementation, the paper fixes only mathematical
shapes in its Problem formulation): every partitioned matrix is stored with one
row per neuron / head-dimension and d_model contiguous, so a block is a run of
whole rows, contiguous in memory (block definition of Sec. 3.1):
    W_up, W_gate : [F, d]   (paper's W^ffn,  rows = hidden neurons)
    W_down       : [F, d]   (paper's C^ffn transposed, rows = hidden neurons)
    W_qkv        : [(H + 2 H_kv) d_head, d]  (transposed W^Q_h | W^K_h | W^V_h, head after head)
    W_o          : [H d_head, d]             (paper's C^attn as printed)

Parity pins: see tests/test_oracle_*.py.  The particular random stream of the
sampler (which blocks a given seed picks) is fixed by this file's hash, not by
the paper: "parity unpinned" for the stream itself; its distribution, its
post-conditions and every other function are pinned.  A whole round at scale has
no worked numeric example in the paper: "parity unpinned" beyond the per-step pins.
"""
from __future__ import annotations

import numpy as np
from scipy.special import erf

FFN_RELU, FFN_GELU, FFN_SWIGLU = 0, 1, 2
MODE_COVER, MODE_IID = 0, 1
KIND_FFN, KIND_HEAD = 0, 1
STREAM_PERM, STREAM_FILL = 0, 1

_U64 = np.uint64
_GOLDEN = _U64(0x9E3779B97F4A7C15)
_M1 = _U64(0xBF58476D1CE4E5B9)
_M2 = _U64(0x94D049BB133111EB)


# ----------------------------------------------------------------------------------------
# Counter-based integer hash used for every random draw of the sampler.
# The paper leaves the generator open (Algorithm 1 only names a routine that draws distinct
# blocks, and Sec. 3.1 asks for a uniform draw); this implementation fixes a 64-bit avalanche
# mixer (the published splitmix64 finaliser) applied to the counter tuple.
# ----------------------------------------------------------------------------------------

def mix64(z):
    """One avalanche round on uint64 (wrapping arithmetic)."""
    z = np.asarray(z, dtype=_U64)
    with np.errstate(over="ignore"):
        z = (z ^ (z >> _U64(30))) * _M1
        z = (z ^ (z >> _U64(27))) * _M2
        return z ^ (z >> _U64(31))


def block_keys(seed, rnd, layer, kind, stream, s, n_full):
    """Sort keys of blocks 0..n_full-1 for one (seed, round, layer, kind, stream, subnet).

    key(b) = (hash48 << 16) | b : the upper 48 bits are random, the lower 16 are the
    block index, so keys are distinct and "smallest key, ties by smaller b" is a
    plain integer order.  Requires n_full <= 65536.
    """
    assert 0 < n_full <= 65536
    with np.errstate(over="ignore"):
        h = mix64(_U64(seed) + _GOLDEN)
        h = mix64(h + _U64(rnd))
        h = mix64(h + _U64((layer << 16) | (kind << 8) | stream))
        h = mix64(h + _U64(s))
        b = np.arange(n_full, dtype=_U64)
        k = mix64(h + b)
    return (k & ~_U64(0xFFFF)) | b


def feasible(n_full, n_subnets, n_sub, n_common, mode=MODE_COVER):
    """Size constraints of Sec. 3.1: N_sub <= N_full and N_full - |C| <= S (N_sub - |C|).
    The IID mode (independent random subnets, no coverage guarantee) only needs
    |C| <= N_sub <= N_full."""
    if not (n_common <= n_sub <= n_full):
        return False
    if mode == MODE_COVER:
        return n_full - n_common <= n_subnets * (n_sub - n_common)
    return True


def sample_blueprint(n_full, n_subnets, n_sub, common, seed, rnd, layer, kind, mode=MODE_COVER):
    """Algorithm 1 ("Generate Training Subnet Blueprint"): returns A [S, N_sub], rows sorted.

    Steps, in the algorithm's order:
      1. every row starts with the common blocks C;
      2. the non-common blocks C' are enumerated -- here in a seeded uniformly random
         order (the text says subnets are generated uniformly at random) -- and the
         i-th goes to subnet i mod S, so every block is assigned at least once;
      3. each subnet s draws N_empty = N_sub - |filled_s| further distinct blocks
         uniformly from those it does not hold yet: the N_empty candidates with the
         smallest fill key of stream (s);
      4. each row is sorted.
    IID mode skips step 2 (used where N_sub is below the feasibility bound).
    """
    common = np.asarray(sorted(set(int(c) for c in common)), dtype=np.int64)
    if not feasible(n_full, n_subnets, n_sub, len(common), mode):
        raise ValueError("infeasible subnet size")
    is_common = np.zeros(n_full, dtype=bool)
    is_common[common] = True
    filled = np.zeros((n_subnets, n_full), dtype=bool)
    filled[:, common] = True                                            # step 1
    if mode == MODE_COVER:                                              # step 2
        kp = block_keys(seed, rnd, layer, kind, STREAM_PERM, 0, n_full)
        non_common = np.flatnonzero(~is_common)
        order = non_common[np.argsort(kp[non_common], kind="stable")]
        for i, b in enumerate(order):
            filled[i % n_subnets, b] = True
    A = np.zeros((n_subnets, n_sub), dtype=np.int32)
    for s in range(n_subnets):                                          # step 3
        n_empty = n_sub - int(filled[s].sum())
        assert n_empty >= 0
        kf = block_keys(seed, rnd, layer, kind, STREAM_FILL, s, n_full)
        cand = np.flatnonzero(~filled[s])
        chosen = cand[np.argsort(kf[cand], kind="stable")[:n_empty]]
        row = filled[s].copy()
        row[chosen] = True
        A[s] = np.flatnonzero(row)                                      # step 4 (ascending)
    return A


def cover_and_pos(A, n_full, counts=None):
    """Derived index data for the aggregator (Sec. 3.3): per block the bitmask of
    subnets holding it, the coverage count (the formula's denominator), and
    pos[s, b] = rank of b inside row A[s] (-1 if absent).  `counts[s]` limits row s
    to its first counts[s] entries (ragged KV-group rows)."""
    S = len(A)
    cover = np.zeros(n_full, dtype=np.uint32)
    pos = np.full((S, n_full), -1, dtype=np.int32)
    for s in range(S):
        row = np.asarray(A[s])[: (len(A[s]) if counts is None else counts[s])]
        cover[row] |= np.uint32(1 << s)
        pos[s, row] = np.arange(len(row), dtype=np.int32)
    count = np.array([bin(int(c)).count("1") for c in cover], dtype=np.int32)
    return cover, count, pos


def kv_groups(head_idx, n_heads, n_kv_heads):
    """Grouped-query attention (not in the paper, which is plain multi-head): KV group
    g = h // (H / H_kv) belongs to subnet s iff any of its query heads does.  Returns
    kv_idx [S, H_kv] (sorted kept groups, padded with -1) and kv_count [S]."""
    S = len(head_idx)
    per = n_heads // n_kv_heads
    kv_idx = np.full((S, n_kv_heads), -1, dtype=np.int32)
    kv_count = np.zeros(S, dtype=np.int32)
    for s in range(S):
        g = np.unique(np.asarray(head_idx[s]) // per)
        kv_idx[s, : len(g)] = g
        kv_count[s] = len(g)
    return kv_idx, kv_count


# ----------------------------------------------------------------------------------------
# Dispatcher (Sec. 3.2): kept blocks are concatenated into dense sub-matrices.
# ----------------------------------------------------------------------------------------

def block_rows_of(blocks, block_rows, row_offset=0):
    blocks = np.asarray(blocks, dtype=np.int64)
    return (row_offset + blocks[:, None] * block_rows + np.arange(block_rows)[None, :]).reshape(-1)


def gather_rows(W_full, blocks, block_rows, row_offset=0):
    """slice = rows of the kept blocks, in blueprint order, concatenated densely."""
    return W_full[block_rows_of(blocks, block_rows, row_offset)].copy()


# ----------------------------------------------------------------------------------------
# Rounding points of the bf16 data flow (weights, stored activations and stored
# activation gradients are bf16; every product-sum is accumulated wide).
# ----------------------------------------------------------------------------------------

def round_bf16(x):
    """float64 -> nearest bf16 (ties to even), returned as float64."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32).astype(np.float64)


def _q(x, lowp):
    return round_bf16(x) if lowp else np.asarray(x, dtype=np.float64)


def act_scale(n_full, n_sub):
    """Activation-shift correction of Sec. 3.4: sqrt(N_full / N_sub)."""
    return float(np.sqrt(n_full / n_sub))


# ----------------------------------------------------------------------------------------
# Layer normalisation (App. A, Layer Normalization): z = (x - mu) / sigma with mu, sigma the mean and the
# standard deviation of the d_model elements of a token, y = gamma * z + b.  The paper's formula has no
# stabiliser; sigma is taken as sqrt(var + eps) with a small eps (the usual convention; eps = 0 gives the
# printed formula).  gamma and b are shared parameters: every worker gets a copy and trains it.
# ----------------------------------------------------------------------------------------

LN_EPS = 1e-5


def layer_norm_fwd(X, gamma, beta, lowp, eps=LN_EPS):
    """Y [T, d] (stored precision) and what the backward pass needs: the normalised rows z and 1 / sigma."""
    mu = X.mean(axis=1, keepdims=True)
    var = ((X - mu) ** 2).mean(axis=1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + eps)
    z = (X - mu) * rstd
    return _q(gamma[None, :] * z + beta[None, :], lowp), {"z": z, "rstd": rstd}


def layer_norm_bwd(dY, saved, gamma, lowp, residual=None):
    """Exact chain rule through layer_norm_fwd: with dz = dY * gamma,
        dX = (dz - mean(dz) - z mean(dz * z)) / sigma,   dgamma = sum_t dY * z,   db = sum_t dY.
    `residual`: gradient arriving over the skip connection around the normalised block, added before dX is stored."""
    z, rstd = saved["z"], saved["rstd"]
    dz = dY * gamma[None, :]
    dX = rstd * (dz - dz.mean(axis=1, keepdims=True) - z * (dz * z).mean(axis=1, keepdims=True))
    return _q(_plus(dX, residual), lowp), np.sum(dY * z, axis=0), np.sum(dY, axis=0)


LN_PARAMS = ("ln_a_g", "ln_a_b", "ln_f_g", "ln_f_b")     # gamma / b of the attention and the FFN normalisation


# ----------------------------------------------------------------------------------------
# FFN block on a dense slice.  Paper (App. A, Feedforward): y = C relu(W x).
# GELU (exact, x Phi(x)) and SwiGLU (silu(gate) * up) are the workloads' variants.
# ----------------------------------------------------------------------------------------

def _sigmoid(z):
    return 1.0 / (1.0 + np.exp(-z))


def _act(pre, kind):
    if kind == FFN_RELU:
        return np.maximum(pre, 0.0)
    if kind == FFN_GELU:
        return 0.5 * pre * (1.0 + erf(pre / np.sqrt(2.0)))
    raise ValueError(kind)


def _act_grad(pre, kind):
    if kind == FFN_RELU:
        return (pre > 0.0).astype(np.float64)
    if kind == FFN_GELU:
        return 0.5 * (1.0 + erf(pre / np.sqrt(2.0))) + pre * np.exp(-0.5 * pre * pre) / np.sqrt(2.0 * np.pi)
    raise ValueError(kind)


def _plus(v, residual):
    return v if residual is None else v + residual


def ffn_fwd(X, W_up, W_gate, W_down, kind, alpha, lowp, residual=None, hidden_mask=None):
    """Y = alpha * act(X W_up^T) W_down  (MLP)  or  alpha * (silu(X W_gate^T) * (X W_up^T)) W_down.
    Returns Y [T, d] and the tensors kept for the backward pass (stored precision).
    `residual` (App. A, Transformer Layer Architecture, final output) is added before Y is stored.
    `hidden_mask` [f] of 0/1 (Sec. 4.1, Masked TwIST): the activations are multiplied by it, y = M * f(x)."""
    U = X @ W_up.T
    mask = 1.0 if hidden_mask is None else np.asarray(hidden_mask, dtype=np.float64)[None, :]
    if kind == FFN_SWIGLU:
        G = X @ W_gate.T
        Hh = mask * ((G * _sigmoid(G)) * U)
        saved = {"G": _q(G, lowp), "U": _q(U, lowp), "Hh": _q(Hh, lowp)}
    else:
        saved = {"U": _q(U, lowp), "Hh": _q(mask * _act(U, kind), lowp)}
    Y = _q(_plus(alpha * (saved["Hh"] @ W_down), residual), lowp)
    return Y, saved


def ffn_bwd(dY, X, saved, W_up, W_gate, W_down, kind, alpha, lowp, residual=None, hidden_mask=None):
    """Exact chain rule through ffn_fwd.  Returns dX and dW_up, dW_gate, dW_down ([f', d] each).
    `residual`: gradient arriving over the skip connection, added to dX before it is stored.
    `hidden_mask`: the mask of the forward pass; the gradient reaching the activations is multiplied by it."""
    dHh = alpha * (dY @ W_down.T)
    if hidden_mask is not None:
        dHh = dHh * np.asarray(hidden_mask, dtype=np.float64)[None, :]
    dW_down = alpha * (saved["Hh"].T @ dY)
    if kind == FFN_SWIGLU:
        G, U = saved["G"], saved["U"]
        sg = _sigmoid(G)
        dG = _q(dHh * U * (sg * (1.0 + G * (1.0 - sg))), lowp)
        dU = _q(dHh * (G * sg), lowp)
        dX = _q(_plus(dG @ W_gate + dU @ W_up, residual), lowp)
        return dX, dU.T @ X, dG.T @ X, dW_down
    dU = _q(dHh * _act_grad(saved["U"], kind), lowp)
    dX = _q(_plus(dU @ W_up, residual), lowp)
    return dX, dU.T @ X, None, dW_down


# ----------------------------------------------------------------------------------------
# Attention projections on a dense slice (App. A, Multi-Head Attention):
# Q_h = X W^Q_h (and K, V), Y_attn = Concat(heads) C^attn.
# ----------------------------------------------------------------------------------------

def qkv_fwd(X, W_qkv, lowp):
    return _q(X @ W_qkv.T, lowp)


def qkv_bwd(dQKV, X, W_qkv, lowp, residual=None):
    return _q(_plus(dQKV @ W_qkv, residual), lowp), dQKV.T @ X


def o_fwd(A, W_o, alpha, lowp, residual=None):
    return _q(_plus(alpha * (A @ W_o), residual), lowp)


def o_bwd(dY, A, W_o, alpha, lowp):
    return _q(alpha * (dY @ W_o.T), lowp), alpha * (A.T @ dY)


# ----------------------------------------------------------------------------------------
# Loss and optimiser of the local steps: mean squared error, plain SGD.
# ----------------------------------------------------------------------------------------

def mse(Y, Tgt, lowp, valid_cols=None, col_mask=None):
    """loss = mean over the T x width elements of (y - t)^2 (no 1/2); dY = 2 (y - t) / (T width).
    valid_cols restricts both to the leading columns, col_mask [width] of 0/1 to the columns it marks (zero
    gradient elsewhere; the mean runs over the valid elements).  No valid column: loss 0, gradient 0."""
    T, width = Y.shape
    if col_mask is not None:
        cols = np.flatnonzero(np.asarray(col_mask) != 0)
    else:
        cols = np.arange(width if valid_cols is None else valid_cols)
    diff = np.zeros_like(Y, dtype=np.float64)
    diff[:, cols] = Y[:, cols] - Tgt[:, cols]
    n = T * len(cols)
    if n == 0:
        return 0.0, diff
    return float(np.sum(diff * diff) / n), _q(2.0 * diff / n, lowp)


def sgd(master, dW, lr, lowp):
    """master <- master - lr dW; returns (new master, compute copy in stored precision)."""
    new = master - lr * dW
    return new, _q(new, lowp)


def adam(master, m, v, dW, step, lr, beta1, beta2, eps, lowp):
    """One Adam step (the optimiser of the paper's experiments, Sec. 5 Setup), in its standard form:
        m <- b1 m + (1 - b1) g,   v <- b2 v + (1 - b2) g^2,
        w <- w - lr (m / (1 - b1^t)) / (sqrt(v / (1 - b2^t)) + eps),        t = step = 1, 2, ...
    Returns (new master, new m, new v, compute copy in stored precision)."""
    m = beta1 * m + (1.0 - beta1) * dW
    v = beta2 * v + (1.0 - beta2) * dW * dW
    m_hat = m / (1.0 - beta1 ** step)
    v_hat = v / (1.0 - beta2 ** step)
    new = master - lr * m_hat / (np.sqrt(v_hat) + eps)
    return new, m, v, _q(new, lowp)


class _Optimizer:
    """Applies the workload's optimiser to a dict of masters.  Adam moments belong to the worker's copy of the
    slice: they start at zero when the slices are dispatched and are not aggregated (the paper exchanges
    parameters only)."""

    def __init__(self, spec):
        self.kind = getattr(spec, "optimizer", "sgd")
        self.spec = spec
        self.state = {}
        self.t = 0

    def begin_step(self):
        self.t += 1

    def update(self, key, master, dW, lowp):
        sp = self.spec
        if self.kind == "sgd":
            return sgd(master, dW, sp.lr, lowp)[0]
        m, v = self.state.get(key, (np.zeros_like(master), np.zeros_like(master)))
        new, m, v, _ = adam(master, m, v, dW, self.t, sp.lr, sp.beta1, sp.beta2, sp.adam_eps, lowp)
        self.state[key] = (m, v)
        return new


# ----------------------------------------------------------------------------------------
# Aggregator (Sec. 3.3): p <- sum_i p_i 1[p in W_i] / sum_i 1[p in W_i].
# ----------------------------------------------------------------------------------------

def aggregate(W_full, subs, blueprints, block_rows, live_mask=None, row_offset=0):
    """Average each partitioned row over the (live) subnets that hold it; rows held by
    no live subnet keep their value (the formula is 0/0 there).  Sum in ascending s."""
    out = np.array(W_full, dtype=np.float64, copy=True)
    acc = np.zeros_like(out)
    cnt = np.zeros(out.shape[0], dtype=np.int64)
    for s, (sub, blocks) in enumerate(zip(subs, blueprints)):
        if live_mask is not None and not (live_mask >> s) & 1:
            continue
        rows = block_rows_of(blocks, block_rows, row_offset)
        acc[rows] += np.asarray(sub, dtype=np.float64)[: len(rows)]
        cnt[rows] += 1
    held = cnt > 0
    out[held] = acc[held] / cnt[held][:, None]
    return out


# ----------------------------------------------------------------------------------------
# One round on one layer, BLOCKWISE composition: the FFN block, the QKV projection and
# the output projection of a layer are independent regression problems, each with its
# own N(0,1) inputs and targets.  Overview of a round: Sec. 3 (generate blueprints,
# dispatch, local training for the repartition interval, aggregate, resample).
# ----------------------------------------------------------------------------------------

def layer_keeps(spec, layer):
    """(N_sub for the FFN blocks, N_sub for the heads) of one layer.  A shared layer (Sec. 5 Setup: the first and
    the last two layers of the paper's runs) has N_sub = N_full in both kinds: every worker holds all of it."""
    if layer in getattr(spec, "shared_layers", ()):
        return spec.d_ff // spec.ffn_block, spec.n_heads
    return spec.ffn_keep, spec.head_keep


def layer_blueprints(spec, rnd, layer):
    """Blueprints of one layer for one round: FFN blocks, heads, KV groups."""
    out = {}
    ffn_keep, head_keep = layer_keeps(spec, layer)
    out["ffn"] = sample_blueprint(spec.d_ff // spec.ffn_block, spec.n_subnets, ffn_keep, spec.common_ffn,
                                  spec.seed_mask, rnd, layer, KIND_FFN, spec.sample_mode)
    if spec.n_heads:
        out["head"] = sample_blueprint(spec.n_heads, spec.n_subnets, head_keep, spec.common_heads,
                                       spec.seed_mask, rnd, layer, KIND_HEAD, spec.sample_mode)
        out["kv_idx"], out["kv_count"] = kv_groups(out["head"], spec.n_heads, spec.n_kv_heads)
    return out


def gather_layer(spec, full, bp, s):
    """Dense slices of subnet s for one layer (full: dict gate/up/down/qkv/o -> [rows, d])."""
    sl = {}
    sl["up"] = gather_rows(full["up"], bp["ffn"][s], spec.ffn_block)
    sl["down"] = gather_rows(full["down"], bp["ffn"][s], spec.ffn_block)
    if spec.ffn_kind == FFN_SWIGLU:
        sl["gate"] = gather_rows(full["gate"], bp["ffn"][s], spec.ffn_block)
    if spec.n_heads:
        dh, H, Hkv = spec.d_head, spec.n_heads, spec.n_kv_heads
        kv = bp["kv_idx"][s][: bp["kv_count"][s]]
        sl["qkv"] = np.concatenate([gather_rows(full["qkv"], bp["head"][s], dh),
                                    gather_rows(full["qkv"], kv, dh, H * dh),
                                    gather_rows(full["qkv"], kv, dh, (H + Hkv) * dh)], axis=0)
        sl["o"] = gather_rows(full["o"], bp["head"][s], dh)
    for m in LN_PARAMS:          # shared parameters are broadcast whole (Sec. 3.2)
        if m in full:
            sl[m] = np.array(full[m], copy=True)
    return sl


def local_steps_blockwise(spec, sl, get_batch, rnd, s, lowp):
    """K local SGD steps of subnet s on its slices `sl` (masters, float64; updated in
    place).  get_batch(kind, rnd, s, k, width) -> [T, width].  Returns the losses
    {block: [K]}.  Batch kinds: 0 X, 1 target of width d, 2 target of QKV width, 3 A."""
    d = spec.d_model
    alpha_f = act_scale(spec.d_ff, sl["up"].shape[0])          # N_full / N_sub of this layer (Sec. 3.4)
    losses = {"ffn": [], "qkv": [], "o": []}
    opt = _Optimizer(spec)
    for k in range(spec.local_steps):
        opt.begin_step()
        X = get_batch(0, rnd, s, k, d).astype(np.float64)
        Td = get_batch(1, rnd, s, k, d).astype(np.float64)
        cw = {m: _q(v, lowp) for m, v in sl.items()}            # compute copies
        Y, saved = ffn_fwd(X, cw["up"], cw.get("gate"), cw["down"], spec.ffn_kind, alpha_f, lowp)
        loss, dY = mse(Y, Td, lowp)
        _, dWu, dWg, dWd = ffn_bwd(dY, X, saved, cw["up"], cw.get("gate"), cw["down"], spec.ffn_kind, alpha_f, lowp)
        losses["ffn"].append(loss)
        sl["up"] = opt.update("up", sl["up"], dWu, lowp)
        sl["down"] = opt.update("down", sl["down"], dWd, lowp)
        if dWg is not None:
            sl["gate"] = opt.update("gate", sl["gate"], dWg, lowp)
        if spec.n_heads:
            alpha_a = act_scale(spec.n_heads * spec.d_head, sl["o"].shape[0])
            nq = sl["qkv"].shape[0]
            Tq = get_batch(2, rnd, s, k, nq).astype(np.float64)
            QKV = qkv_fwd(X, cw["qkv"], lowp)
            loss, dQKV = mse(QKV, Tq, lowp)
            _, dWq = qkv_bwd(dQKV, X, cw["qkv"], lowp)
            losses["qkv"].append(loss)
            sl["qkv"] = opt.update("qkv", sl["qkv"], dWq, lowp)
            A = get_batch(3, rnd, s, k, sl["o"].shape[0]).astype(np.float64)
            Yo = o_fwd(A, cw["o"], alpha_a, lowp)
            loss, dYo = mse(Yo, Td, lowp)
            _, dWo = o_bwd(dYo, A, cw["o"], alpha_a, lowp)
            losses["o"].append(loss)
            sl["o"] = opt.update("o", sl["o"], dWo, lowp)
    return losses


def aggregate_layer(spec, full, slices, bp):
    """Aggregator over all partitioned matrices of one layer; returns the new full dict."""
    S = spec.n_subnets
    new = {}
    for m in ("up", "down") + (("gate",) if spec.ffn_kind == FFN_SWIGLU else ()):
        new[m] = aggregate(full[m], [slices[s][m] for s in range(S)], bp["ffn"], spec.ffn_block)
    for m in LN_PARAMS:          # held by every subnet: the aggregator formula is the plain mean over S
        if m in full:
            new[m] = aggregate(np.asarray(full[m])[None, :], [slices[s][m][None, :] for s in range(S)], [[0]] * S, 1)[0]
    if spec.n_heads:
        dh, H, Hkv = spec.d_head, spec.n_heads, spec.n_kv_heads
        a_sub = len(bp["head"][0]) * dh
        kvs = [bp["kv_idx"][s][: bp["kv_count"][s]] for s in range(S)]
        qkv = aggregate(full["qkv"], [slices[s]["qkv"][:a_sub] for s in range(S)], bp["head"], dh)
        qkv = aggregate(qkv, [slices[s]["qkv"][a_sub:a_sub + len(kvs[s]) * dh] for s in range(S)], kvs, dh,
                        row_offset=H * dh)
        qkv = aggregate(qkv, [slices[s]["qkv"][a_sub + len(kvs[s]) * dh:] for s in range(S)], kvs, dh,
                        row_offset=(H + Hkv) * dh)
        new["qkv"] = qkv
        new["o"] = aggregate(full["o"], [slices[s]["o"] for s in range(S)], bp["head"], dh)
    return new


def round_blockwise_layer(spec, full, get_batch, rnd, layer, lowp):
    """One full round on one layer: blueprint -> gather -> K local steps per subnet ->
    aggregate.  Returns (new full weights of the layer, blueprints, losses per subnet)."""
    bp = layer_blueprints(spec, rnd, layer)
    slices, losses = [], []
    for s in range(spec.n_subnets):
        sl = {m: np.asarray(v, dtype=np.float64) for m, v in gather_layer(spec, full, bp, s).items()}
        losses.append(local_steps_blockwise(spec, sl, get_batch, rnd, s, lowp))
        slices.append(sl)
    new = aggregate_layer(spec, full, slices, bp)
    if lowp:   # the stored full model is bf16; the next round's gather reads the rounded shadow
        new_shadow = {m: round_bf16(v) for m, v in new.items()}
    else:
        new_shadow = new
    return new, new_shadow, bp, losses


# ----------------------------------------------------------------------------------------
# Attention core on the kept heads (App. A, Multi-Head Attention):
#   head_h = softmax(Q_h K_h^T / sqrt(d_head)) V_h,
# applied per sequence with a causal mask (the workloads are causal language-model shapes:
# position n attends positions <= n).  Grouped-query attention (an extension): kept head hq
# reads the K/V columns of its KV group, head_kv[hq] = position of that group among the
# subnet's kept groups.
# Layout of QKV [T, a' + 2 kvw]: Q of the kept heads, then K of the kept groups, then V.
# ----------------------------------------------------------------------------------------

def _causal_softmax(scores):
    n = scores.shape[0]
    masked = np.where(np.tril(np.ones((n, n), dtype=bool)), scores, -np.inf)
    masked = masked - masked.max(axis=1, keepdims=True)
    e = np.exp(masked)
    return e / e.sum(axis=1, keepdims=True)


def attn_core_fwd(QKV, n_seqs, seq_len, d_head, head_kv, kv_width, lowp):
    """A [T, a'] = concatenated heads; T = n_seqs * seq_len rows, sequence after sequence."""
    H = len(head_kv)
    a = H * d_head
    A = np.zeros((n_seqs * seq_len, a), dtype=np.float64)
    for b in range(n_seqs):
        rows = slice(b * seq_len, (b + 1) * seq_len)
        for hq in range(H):
            g = int(head_kv[hq])
            Q = QKV[rows, hq * d_head:(hq + 1) * d_head]
            K = QKV[rows, a + g * d_head:a + (g + 1) * d_head]
            V = QKV[rows, a + kv_width + g * d_head:a + kv_width + (g + 1) * d_head]
            P = _causal_softmax(Q @ K.T / np.sqrt(d_head))
            A[rows, hq * d_head:(hq + 1) * d_head] = P @ V
    return _q(A, lowp)


def attn_core_bwd(dA, QKV, n_seqs, seq_len, d_head, head_kv, kv_width, lowp):
    """Exact chain rule through attn_core_fwd: with P the softmax and dP = dO V^T,
    dV = P^T dO,  dS = P * (dP - rowsum(dP * P)),  dQ = dS K / sqrt(d),  dK = dS^T Q / sqrt(d);
    heads that share a KV group add up in dK and dV."""
    H = len(head_kv)
    a = H * d_head
    dQKV = np.zeros_like(QKV, dtype=np.float64)
    for b in range(n_seqs):
        rows = slice(b * seq_len, (b + 1) * seq_len)
        for hq in range(H):
            g = int(head_kv[hq])
            qc = slice(hq * d_head, (hq + 1) * d_head)
            kc = slice(a + g * d_head, a + (g + 1) * d_head)
            vc = slice(a + kv_width + g * d_head, a + kv_width + (g + 1) * d_head)
            Q, K, V, dO = QKV[rows, qc], QKV[rows, kc], QKV[rows, vc], dA[rows, qc]
            P = _causal_softmax(Q @ K.T / np.sqrt(d_head))
            dP = dO @ V.T
            dS = P * (dP - np.sum(dP * P, axis=1, keepdims=True))
            dQKV[rows, qc] += dS @ K / np.sqrt(d_head)
            dQKV[rows, kc] += dS.T @ Q / np.sqrt(d_head)
            dQKV[rows, vc] += P.T @ dO
    return _q(dQKV, lowp)


# ----------------------------------------------------------------------------------------
# STACK composition: the chained transformer of App. A (Transformer Layer Architecture),
# without layer normalisation, biases and embeddings (not on this path):
#   x <- x + alpha_a * Concat(heads) C^attn ;  x <- x + alpha_f * FFN(x)   for every layer,
# one MSE loss on the final x.  alpha = sqrt(N_full / N_sub) scales each block's output
# before the residual addition (Sec. 3.4).
# ----------------------------------------------------------------------------------------

def head_kv_positions(bp, spec, s):
    """Position of each kept head's KV group among subnet s's kept groups."""
    per = spec.n_heads // spec.n_kv_heads
    groups = list(bp["kv_idx"][s][: bp["kv_count"][s]])
    return np.array([groups.index(h // per) for h in bp["head"][s]], dtype=np.int64)


def stack_fwd(spec, layers, head_kv, X0, n_seqs, seq_len, lowp):
    """layers[l] = compute copies {gate, up, down, qkv, o} of one subnet; head_kv[l] as above.
    Returns the final x and what the backward pass needs per layer."""
    x, saved = X0, []
    for l, W in enumerate(layers):
        alpha_f = act_scale(spec.d_ff, W["up"].shape[0])                        # per layer: N_full / N_sub
        alpha_a = act_scale(spec.n_heads * spec.d_head, W["o"].shape[0])
        kvw = (W["qkv"].shape[0] - W["o"].shape[0]) // 2
        sv = {"x": x, "kvw": kvw}
        if "ln_a_g" in W:            # pre-LN layer (App. A, Transformer Layer Architecture, steps 1 and 4)
            x_a, sv["ln_a"] = layer_norm_fwd(x, W["ln_a_g"], W["ln_a_b"], lowp)
        else:
            x_a = x
        QKV = qkv_fwd(x_a, W["qkv"], lowp)
        A = attn_core_fwd(QKV, n_seqs, seq_len, spec.d_head, head_kv[l], kvw, lowp)
        x_mid = o_fwd(A, W["o"], alpha_a, lowp, residual=x)
        if "ln_f_g" in W:
            x_f, sv["ln_f"] = layer_norm_fwd(x_mid, W["ln_f_g"], W["ln_f_b"], lowp)
        else:
            x_f = x_mid
        x_out, ffn_saved = ffn_fwd(x_f, W["up"], W.get("gate"), W["down"], spec.ffn_kind, alpha_f, lowp,
                                   residual=x_mid)
        sv.update({"x_a": x_a, "QKV": QKV, "A": A, "x_mid": x_mid, "x_f": x_f, "ffn": ffn_saved})
        saved.append(sv)
        x = x_out
    return x, saved


def stack_bwd(spec, layers, head_kv, saved, dX, n_seqs, seq_len, lowp):
    """Gradients of every layer's slices for the loss gradient dX at the output; also returns
    the gradient with respect to the input.  The gradient of each residual sum flows both
    through the block and over the skip connection."""
    grads = [None] * len(layers)
    dx = dX
    for l in reversed(range(len(layers))):
        W, sv = layers[l], saved[l]
        alpha_f = act_scale(spec.d_ff, W["up"].shape[0])
        alpha_a = act_scale(spec.n_heads * spec.d_head, W["o"].shape[0])
        g = {}
        if "ln_f" in sv:     # the skip connection's gradient joins the normalised branch's at the normalisation's input
            d_f, dWu, dWg, dWd = ffn_bwd(dx, sv["x_f"], sv["ffn"], W["up"], W.get("gate"), W["down"],
                                         spec.ffn_kind, alpha_f, lowp)
            dx_mid, g["ln_f_g"], g["ln_f_b"] = layer_norm_bwd(d_f, sv["ln_f"], W["ln_f_g"], lowp, residual=dx)
        else:
            dx_mid, dWu, dWg, dWd = ffn_bwd(dx, sv["x_mid"], sv["ffn"], W["up"], W.get("gate"), W["down"],
                                            spec.ffn_kind, alpha_f, lowp, residual=dx)
        dA, dWo = o_bwd(dx_mid, sv["A"], W["o"], alpha_a, lowp)
        dQKV = attn_core_bwd(dA, sv["QKV"], n_seqs, seq_len, spec.d_head, head_kv[l], sv["kvw"], lowp)
        if "ln_a" in sv:
            d_a, dWq = qkv_bwd(dQKV, sv["x_a"], W["qkv"], lowp)
            dx, g["ln_a_g"], g["ln_a_b"] = layer_norm_bwd(d_a, sv["ln_a"], W["ln_a_g"], lowp, residual=dx_mid)
        else:
            dx, dWq = qkv_bwd(dQKV, sv["x"], W["qkv"], lowp, residual=dx_mid)
        g.update({"up": dWu, "gate": dWg, "down": dWd, "qkv": dWq, "o": dWo})
        grads[l] = g
    return grads, dx


def local_steps_stack(spec, slices, head_kv, get_batch, rnd, s, n_seqs, seq_len, lowp):
    """K local SGD steps of subnet s through the whole stack (masters `slices[l]`, float64,
    updated in place).  Batch kinds: 0 input X of width d, 1 target of width d.  Returns the losses."""
    losses = []
    opt = _Optimizer(spec)
    for k in range(spec.local_steps):
        opt.begin_step()
        X0 = get_batch(0, rnd, s, k, spec.d_model).astype(np.float64)
        Tgt = get_batch(1, rnd, s, k, spec.d_model).astype(np.float64)
        # compute copies: the partitioned matrices in stored precision; the normalisation's parameters stay wide
        layers = [{m: (v if m in LN_PARAMS else _q(v, lowp)) for m, v in sl.items()} for sl in slices]
        xL, saved = stack_fwd(spec, layers, head_kv, X0, n_seqs, seq_len, lowp)
        loss, dX = mse(xL, Tgt, lowp)
        grads, _ = stack_bwd(spec, layers, head_kv, saved, dX, n_seqs, seq_len, lowp)
        losses.append(loss)
        for l, (sl, g) in enumerate(zip(slices, grads)):
            for m in sl:
                sl[m] = opt.update((l, m), sl[m], g[m], lowp and m not in LN_PARAMS)
    return losses


def round_stack(spec, full, get_batch, rnd, n_seqs, seq_len, lowp):
    """One full round in STACK composition.  full[l] = dict of the layer's full matrices.
    Returns (new full weights per layer, blueprints per layer, losses per subnet)."""
    L = spec.n_layers
    bps = [layer_blueprints(spec, rnd, l) for l in range(L)]
    all_slices, losses = [], []
    for s in range(spec.n_subnets):
        slices = [{m: np.asarray(v, dtype=np.float64) for m, v in gather_layer(spec, full[l], bps[l], s).items()}
                  for l in range(L)]
        head_kv = [head_kv_positions(bps[l], spec, s) for l in range(L)]
        losses.append(local_steps_stack(spec, slices, head_kv, get_batch, rnd, s, n_seqs, seq_len, lowp))
        all_slices.append(slices)
    new = [aggregate_layer(spec, full[l], [all_slices[s][l] for s in range(spec.n_subnets)], bps[l]) for l in range(L)]
    return new, bps, losses


# ----------------------------------------------------------------------------------------
# Parameter-count model of App. C (used to pin the byte counts of gather / aggregate).
# ----------------------------------------------------------------------------------------

def n_attn_params(d_attn, d_model, bias=True):
    """N_attn = 4 d_attn d_model (+ 3 d_attn + d_model with biases)."""
    return 4 * d_attn * d_model + ((3 * d_attn + d_model) if bias else 0)


def n_ffn_params(d_ffn, d_model, bias=True):
    """N_ffn = 2 d_ffn d_model (+ d_ffn + d_model with biases)."""
    return 2 * d_ffn * d_model + ((d_ffn + d_model) if bias else 0)
