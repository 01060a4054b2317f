"""CPU oracle (fp64, numpy) for TarFlow forward, sequential inverse and Jacobi inverse.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the CUDA library must
compute; it shares no code with the CUDA path and the product never imports it.  Only the test
suite, the smoke check and the benchmark's CPU-baseline leg call it.

What follows the paper, and where:
  * block forward  v_1 = u_1, v_l = (u_l - g(u_<l)) * exp(s(u_<l))        -- Eq. 4 (the AR affine block)
  * block inverse  u_1 = v_1, u_l = v_l * exp(-s(u_<l)) + g(u_<l)         -- Eq. 5, strictly in order
  * Jacobi decoding of one block                                          -- Algorithm 1 / Eq. 8
  * selective policy (first block in generation order sequential, rest Jacobi) -- Sec. 3.5
  * token-order reversal between blocks                                   -- remark after Eq. 4
Notation here: mu = g, alpha = -s, so the inverse reads u_l = v_l * exp(alpha_l) + mu_l and the
log-determinant of x -> z is  -sum(alpha)  (Eq. 1 with Eq. 4).

The parameter network (a causal pre-LayerNorm transformer; the paper defers its details to the
TarFlow code, which is not available) is fixed by the readings listed in the design notes:
LayerNorm eps 1e-5, attention scale 1/sqrt(head_dim) with a causal mask that includes the
position itself, exact (erf) GELU, biases everywhere, a final LayerNorm before the output head,
head output split as [mu~ | alpha~], and the one-position shift  mu_l = mu~_{l-1}, alpha_l =
alpha~_{l-1}, mu_1 = alpha_1 = 0  that makes (mu_l, alpha_l) a function of u_<l only.

Pins (tests/test_oracle_pins.py): forward/inverse round trip, log|det J| by finite differences,
strict lower-triangularity of the dependence, Prop. 3.2 (first t tokens exact after t sweeps,
u^L = sequential, u^{L+1} = u^L), fixed point F(u*) = u*, cached == uncached sequential, the
zero-head identity flow, textbook special cases of softmax / LayerNorm / GELU, and brute-force
scalar loops on micro inputs.  Absolute agreement with the authors' trained system (iteration
counts 4-7, reconstruction MSE, timings) is "parity unpinned": those need weights that are not here.
"""
from __future__ import annotations

import math

import numpy as np
from scipy.special import erf

LN_EPS = 1e-5


# --------------------------------------------------------------------------------------------
# layout: image <-> token sequence, block permutation
# --------------------------------------------------------------------------------------------
def patchify(x, p):
    """[B,C,H,W] -> [B,L,D]; patches in raster order, inside a token the order is (c, py, px)."""
    B, C, H, W = x.shape
    t = x.reshape(B, C, H // p, p, W // p, p)          # b c gy py gx px
    t = t.transpose(0, 2, 4, 1, 3, 5)                   # b gy gx c py px
    return np.ascontiguousarray(t.reshape(B, (H // p) * (W // p), C * p * p))


def unpatchify(t, C, H, W, p):
    """Exact inverse of patchify."""
    B = t.shape[0]
    x = t.reshape(B, H // p, W // p, C, p, p).transpose(0, 3, 1, 4, 2, 5)
    return np.ascontiguousarray(x.reshape(B, C, H, W))


def permute(seq, g):
    """Block permutation P_g: identity for even g, token reversal for odd g (its own inverse).

    The paper reverses the sequence after each transformation (remark after Eq. 4); applying the
    reversal on entry to, and undoing it on exit from, every odd block is the same flow with all
    inter-block tensors kept in raster order.
    """
    return seq[:, ::-1, :] if (g % 2 == 1) else seq


# --------------------------------------------------------------------------------------------
# textbook pieces
# --------------------------------------------------------------------------------------------
def layer_norm(x, gamma, beta):
    mean = x.mean(axis=-1, keepdims=True)
    var = ((x - mean) ** 2).mean(axis=-1, keepdims=True)
    return (x - mean) / np.sqrt(var + LN_EPS) * gamma + beta


def gelu(x):
    return 0.5 * x * (1.0 + erf(x / math.sqrt(2.0)))


def softmax_lastdim(s):
    s = s - s.max(axis=-1, keepdims=True)
    e = np.exp(s)
    return e / e.sum(axis=-1, keepdims=True)


def linear(x, w, b):
    """y = x @ w.T + b with w stored [out, in]."""
    return x @ w.T + b


def causal_attention(q, k, v, n_heads):
    """Multi-head attention, position i attends to positions j <= i.  q,k,v: [B,L,d]."""
    B, L, d = q.shape
    hd = d // n_heads
    qh = q.reshape(B, L, n_heads, hd).transpose(0, 2, 1, 3)
    kh = k.reshape(B, L, n_heads, hd).transpose(0, 2, 1, 3)
    vh = v.reshape(B, L, n_heads, hd).transpose(0, 2, 1, 3)
    s = (qh @ kh.transpose(0, 1, 3, 2)) / math.sqrt(hd)          # [B,h,L,L]
    future = np.triu(np.ones((L, L), dtype=bool), k=1)
    s = np.where(future, -np.inf, s)
    o = softmax_lastdim(s) @ vh                                    # [B,h,L,hd]
    return o.transpose(0, 2, 1, 3).reshape(B, L, d)


# --------------------------------------------------------------------------------------------
# parameter network of one block
# --------------------------------------------------------------------------------------------
def _f64(blk):
    return {k: np.asarray(v, dtype=np.float64) for k, v in blk.items()}


def head_raw(blk, u, labels, cfg):
    """Un-shifted head output o[b,l] = (mu~_l, alpha~_l) from a full causal pass over u [B,L,D]."""
    w = _f64(blk)
    B, L, D = u.shape
    h = linear(u, w["w_in"], w["b_in"]) + w["pos"][None, :L, :]
    if cfg["n_classes"] > 0:
        h = h + w["cls"][np.asarray(labels)][:, None, :]
    d = cfg["width"]
    for i in range(cfg["n_layers"]):
        p = f"l{i}."
        qkv = linear(layer_norm(h, w[p + "ln1_g"], w[p + "ln1_b"]), w[p + "w_qkv"], w[p + "b_qkv"])
        a = causal_attention(qkv[..., :d], qkv[..., d:2 * d], qkv[..., 2 * d:], cfg["n_heads"])
        h = h + linear(a, w[p + "w_o"], w[p + "b_o"])
        m = gelu(linear(layer_norm(h, w[p + "ln2_g"], w[p + "ln2_b"]), w[p + "w_1"], w[p + "b_1"]))
        h = h + linear(m, w[p + "w_2"], w[p + "b_2"])
    return linear(layer_norm(h, w["lnf_g"], w["lnf_b"]), w["w_out"], w["b_out"])   # [B,L,2D]


def block_params(blk, u, labels, cfg):
    """(mu, alpha), each [B,L,D], with mu_l, alpha_l functions of u_<l only (Eq. 4's g, -s)."""
    D = u.shape[2]
    o = head_raw(blk, u, labels, cfg)
    mu = np.zeros_like(u)
    alpha = np.zeros_like(u)
    mu[:, 1:, :] = o[:, :-1, :D]
    alpha[:, 1:, :] = o[:, :-1, D:]
    return mu, alpha


# --------------------------------------------------------------------------------------------
# one block: forward (Eq. 4), sequential inverse (Eq. 5), Jacobi inverse (Algorithm 1)
# --------------------------------------------------------------------------------------------
def block_forward(blk, u, labels, cfg):
    """v = f(u) and this block's contribution to log|det d v / d u| per sample (= -sum alpha)."""
    mu, alpha = block_params(blk, u, labels, cfg)
    v = (u - mu) * np.exp(-alpha)
    return v, -alpha.sum(axis=(1, 2))


def block_inverse_sequential_uncached(blk, v, labels, cfg):
    """Eq. 5 taken literally: for l = 1..L recompute the network on what is known, set u_l."""
    B, L, D = v.shape
    u = np.zeros_like(v)
    for l in range(L):
        mu, alpha = block_params(blk, u, labels, cfg)    # only rows < l of u matter for row l
        u[:, l, :] = v[:, l, :] * np.exp(alpha[:, l, :]) + mu[:, l, :]
    return u


def block_inverse_sequential(blk, v, labels, cfg):
    """Eq. 5 with a key/value cache: L-1 single-token passes (Sec. 3.5, sequential decoding)."""
    w = _f64(blk)
    B, L, D = v.shape
    d, nh, N = cfg["width"], cfg["n_heads"], cfg["n_layers"]
    hd = d // nh
    kc = np.zeros((N, B, L, d))
    vc = np.zeros((N, B, L, d))
    u = np.zeros_like(v)
    u[:, 0, :] = v[:, 0, :]
    for t in range(L - 1):                               # token t is known; produce token t+1
        h = linear(u[:, t, :], w["w_in"], w["b_in"]) + w["pos"][t][None, :]
        if cfg["n_classes"] > 0:
            h = h + w["cls"][np.asarray(labels)]
        for i in range(N):
            p = f"l{i}."
            qkv = linear(layer_norm(h, w[p + "ln1_g"], w[p + "ln1_b"]), w[p + "w_qkv"], w[p + "b_qkv"])
            kc[i, :, t, :] = qkv[:, d:2 * d]
            vc[i, :, t, :] = qkv[:, 2 * d:]
            q = qkv[:, :d].reshape(B, nh, hd)
            kk = kc[i, :, :t + 1, :].reshape(B, t + 1, nh, hd)
            vv = vc[i, :, :t + 1, :].reshape(B, t + 1, nh, hd)
            s = np.einsum("bhc,bjhc->bhj", q, kk) / math.sqrt(hd)
            a = np.einsum("bhj,bjhc->bhc", softmax_lastdim(s), vv).reshape(B, d)
            h = h + linear(a, w[p + "w_o"], w[p + "b_o"])
            m = gelu(linear(layer_norm(h, w[p + "ln2_g"], w[p + "ln2_b"]), w[p + "w_1"], w[p + "b_1"]))
            h = h + linear(m, w[p + "w_2"], w[p + "b_2"])
        o = linear(layer_norm(h, w["lnf_g"], w["lnf_b"]), w["w_out"], w["b_out"])
        u[:, t + 1, :] = v[:, t + 1, :] * np.exp(o[:, D:]) + o[:, :D]
    return u


def jacobi_map(blk, u_prev, v, labels, cfg):
    """The iteration map F of Definition B.1: F(u)_1 = v_1, F(u)_l = v_l * exp(alpha_l(u)) + mu_l(u)."""
    mu, alpha = block_params(blk, u_prev, labels, cfg)
    u_new = v * np.exp(alpha) + mu          # row 0 has mu = alpha = 0, so u_new[:,0] = v[:,0]
    return u_new


def block_inverse_jacobi(blk, v, labels, cfg, tau, max_iters, u0=None, u_star=None, info=None):
    """Algorithm 1 applied to every sample of the batch independently.

    u^0 = 0 (or `u0`); sweep t: u^t = F(u^{t-1}); a sample stops after the first sweep whose
    max_{l,c} |u^t - u^{t-1}| <= tau  (tau < 0: never, run exactly max_iters sweeps); a sample
    that has stopped is not touched again.  Returns (u, iters[B], trace) where iters counts the
    sweeps a sample executed including the passing one, and trace[t-1][b] = ||u^t - u_star||_2
    when u_star is given (Fig. "Convergence dynamics").  If `info` is a dict it receives
    info["last_maxdiff"][b] = max|u^t - u^{t-1}| of the last sweep sample b executed.
    """
    B, L, D = v.shape
    u = np.zeros_like(v) if u0 is None else np.array(u0, dtype=np.float64)
    iters = np.zeros(B, dtype=np.int64)
    last_m = np.full(B, np.inf)
    active = np.arange(B)
    trace = []
    t = 0
    while active.size > 0 and t < max_iters:
        t += 1
        lab = None if labels is None else np.asarray(labels)[active]
        u_new = jacobi_map(blk, u[active], v[active], lab, cfg)
        m = np.abs(u_new - u[active]).reshape(active.size, -1).max(axis=1)
        u[active] = u_new
        iters[active] = t
        last_m[active] = m
        if u_star is not None:
            trace.append(np.sqrt(((u - u_star) ** 2).reshape(B, -1).sum(axis=1)))
        if tau >= 0:
            active = active[m > tau]
    if info is not None:
        info["last_maxdiff"] = last_m
    return u, iters, trace


# --------------------------------------------------------------------------------------------
# whole model
# --------------------------------------------------------------------------------------------
def model_forward(blocks, x, labels, cfg):
    """x -> z through blocks K-1 .. 0 (data side to noise side), logdet = -sum alpha over blocks."""
    seq = patchify(np.asarray(x, dtype=np.float64), cfg["patch"])
    logdet = np.zeros(seq.shape[0])
    for g in reversed(range(cfg["n_blocks"])):
        v, ld = block_forward(blocks[g], permute(seq, g), labels, cfg)
        seq = permute(v, g)
        logdet += ld
    return unpatchify(seq, cfg["C"], cfg["H"], cfg["W"], cfg["patch"]), logdet


def model_inverse(blocks, z, labels, cfg, policy, tau, max_iters, cached=True, init_mode=0, u0=None,
                  fallback_sweeps=0, return_states=False, ref_states=None):
    """z -> x through blocks 0 .. K-1 in generation order.

    policy[g] = 0: sequential (Eq. 5); 1: Jacobi (Algorithm 1).  Returns (x, iters[K,B]); a
    sequential block reports L-1 steps (as in Table "Average number of Jacobi iterations").

    Variants discussed around Algorithm 1 (Sec. 3.5, Sec. 4.4), all off by default:
      tau              a scalar, or one value per block;
      init_mode        0: u^0 = 0;  1: u^0 = v (the block's input);  2: u^0 = patchify(u0[g]) with
                       u0 [K,B,C,H,W] supplied by the caller (e.g. N(0, I) draws);
      fallback_sweeps  n > 0: a Jacobi block is cut after n sweeps and the samples that have not
                       passed the test by then are decoded sequentially (Eq. 5) from the block's
                       input; they report n + L - 1 iterations (ignored when tau < 0 or n >= max_iters);
      return_states    also return the image-shaped sequence after every block [K,B,C,H,W];
      ref_states       [K,B,C,H,W]: also return, per Jacobi block, the trace ||u^t - ref_g||_2 per
                       sweep and sample (Fig. "Convergence dynamics").
    With any of the last two the return value is (x, iters, extras) with extras a dict.
    """
    seq = patchify(np.asarray(z, dtype=np.float64), cfg["patch"])
    B, L, _ = seq.shape
    K = cfg["n_blocks"]
    taus = [float(tau)] * K if np.ndim(tau) == 0 else [float(t) for t in tau]
    iters = np.zeros((K, B), dtype=np.int64)
    states, traces = [], {}
    for g in range(K):
        v = np.ascontiguousarray(permute(seq, g))
        if policy[g] == 0:
            fn = block_inverse_sequential if cached else block_inverse_sequential_uncached
            u = fn(blocks[g], v, labels, cfg)
            iters[g, :] = L - 1
        else:
            if init_mode == 0:
                start = None
            elif init_mode == 1:
                start = v
            else:
                start = permute(patchify(np.asarray(u0[g], dtype=np.float64), cfg["patch"]), g)
            star = None
            if ref_states is not None:
                star = permute(patchify(np.asarray(ref_states[g], dtype=np.float64), cfg["patch"]), g)
            cut = taus[g] >= 0 and 0 < fallback_sweeps < max_iters
            info = {}
            u, it, tr = block_inverse_jacobi(blocks[g], v, labels, cfg, taus[g], fallback_sweeps if cut else max_iters,
                                             u0=start, u_star=star, info=info)
            if cut:
                # the samples whose last executed sweep did not pass the test fall back to Eq. 5
                left = np.nonzero(info["last_maxdiff"] > taus[g])[0]
                if left.size:
                    lab = None if labels is None else np.asarray(labels)[left]
                    u[left] = block_inverse_sequential(blocks[g], v[left], lab, cfg)
                    it[left] = fallback_sweeps + L - 1
            iters[g, :] = it
            if star is not None:
                traces[g] = np.array(tr)
        seq = np.ascontiguousarray(permute(u, g))
        if return_states:
            states.append(unpatchify(seq, cfg["C"], cfg["H"], cfg["W"], cfg["patch"]))
    x = unpatchify(seq, cfg["C"], cfg["H"], cfg["W"], cfg["patch"])
    if return_states or ref_states is not None:
        return x, iters, {"states": np.array(states) if return_states else None, "l2": traces}
    return x, iters


def model_inverse_sequential(blocks, z, labels, cfg):
    x, _ = model_inverse(blocks, z, labels, cfg, [0] * cfg["n_blocks"], 0.0, 0)
    return x
