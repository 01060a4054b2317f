"""CPU oracle (fp64, numpy) for Jacobi decoding of a masked autoregressive flow (MAF) built from MADE networks.

TEST INFRASTRUCTURE ONLY: the slow, plain statement of what the CUDA library's tf_maf_* calls must compute.  It shares
no code with the CUDA path and the product never imports it.

What follows the paper, and where: App. E.3 ("Experiments on Masked Autoregressive Flow") applies Algorithm 1 to every
layer of an MLP-based autoregressive flow, for which no key/value cache exists.  The flow itself is the affine
autoregressive block of Eq. 4 / Eq. 5 with one scalar per position (token dimension 1):
    forward   v_i = (u_i - mu_i(u_<i)) * exp(-alpha_i(u_<i))                  -- Eq. 4 with mu = g, alpha = -s
    inverse   u_i = v_i * exp(alpha_i(u_<i)) + mu_i(u_<i),  i = 1..D in order -- Eq. 5
    Jacobi    u^t = v * exp(alpha(u^{t-1})) + mu(u^{t-1}),  u^0 = 0            -- Algorithm 1 / Eq. 8
and the order of the D dimensions is reversed between layers (remark after Eq. 4).

The parameter network (the paper uses a library implementation that is not available here) is fixed by these readings:
a MADE network [Germain et al. 2015] with two hidden layers of H ReLU units.  Degrees: input i has degree i (1..D);
hidden unit j of either hidden layer has degree 1 + (j mod (D-1)); output i (both mu_i and alpha_i) has degree i.
A hidden unit sees the inputs / hidden units of degree <= its own, an output sees hidden units of degree < its own,
so (mu_i, alpha_i) is a function of u_<i only and (mu_1, alpha_1) is a constant (the output bias).  Weights are
dense tensors multiplied element-wise by these 0/1 masks; the output layer is stored [mu | alpha] (first D rows mu).

Pins (tests/test_maf_oracle_pins.py): connectivity of the masks by brute force over paths, strict lower-triangular
dependence by finite differences, forward o inverse = identity, log|det J| against the brute-force Jacobian
determinant, Prop. 3.2 (first t values exact after t sweeps, D sweeps = sequential decoding, one more sweep changes
nothing), fixed point, zero-output-layer identity flow.  Agreement with the authors' trained models is "parity
unpinned": no weights exist here.
"""
from __future__ import annotations

import numpy as np


def degrees(D, H):
    """(input degrees [D], hidden degrees [H], output degrees [D])."""
    d_in = np.arange(1, D + 1)
    d_hid = 1 + (np.arange(H) % max(D - 1, 1))
    return d_in, d_hid, d_in.copy()


def masks(D, H):
    """0/1 masks of the three linear layers, each [out, in]."""
    d_in, d_hid, d_out = degrees(D, H)
    m1 = (d_hid[:, None] >= d_in[None, :]).astype(np.float64)      # hidden 1 <- input
    m2 = (d_hid[:, None] >= d_hid[None, :]).astype(np.float64)     # hidden 2 <- hidden 1
    m3 = (d_out[:, None] > d_hid[None, :]).astype(np.float64)      # output   <- hidden 2 (strict)
    return m1, m2, np.concatenate([m3, m3], axis=0)                # [mu | alpha] rows share the mask


def made_params(blk, u):
    """(mu, alpha), each [B, D]; mu_i, alpha_i depend on u_<i only."""
    D = u.shape[1]
    H = blk["w1"].shape[0]
    m1, m2, m3 = masks(D, H)
    w = {k: np.asarray(v, dtype=np.float64) for k, v in blk.items()}
    h1 = np.maximum(u @ (w["w1"] * m1).T + w["b1"], 0.0)
    h2 = np.maximum(h1 @ (w["w2"] * m2).T + w["b2"], 0.0)
    o = h2 @ (w["w3"] * m3).T + w["b3"]
    return o[:, :D], o[:, D:]


def permute(x, g):
    """Layer permutation: identity for even g, reversal of the D dimensions for odd g (its own inverse)."""
    return x[:, ::-1] if (g % 2 == 1) else x


def block_forward(blk, u):
    mu, alpha = made_params(blk, u)
    return (u - mu) * np.exp(-alpha), -alpha.sum(axis=1)


def block_inverse_sequential(blk, v):
    """Eq. 5 literally: D passes of the network, dimension i fixed in pass i (there is no cache to reuse)."""
    B, D = v.shape
    u = np.zeros_like(v)
    for i in range(D):
        mu, alpha = made_params(blk, u)                  # only u_<i matters for column i
        u[:, i] = v[:, i] * np.exp(alpha[:, i]) + mu[:, i]
    return u


def jacobi_map(blk, u_prev, v):
    mu, alpha = made_params(blk, u_prev)
    return v * np.exp(alpha) + mu


def block_inverse_jacobi(blk, v, tau, max_iters):
    """Algorithm 1 per sample: u^0 = 0; a sample stops after the first sweep with max_i |u^t - u^{t-1}| <= tau
    (tau < 0: exactly max_iters sweeps).  Returns (u, iters[B])."""
    B, D = v.shape
    u = np.zeros_like(v)
    iters = np.zeros(B, dtype=np.int64)
    active = np.arange(B)
    t = 0
    while active.size > 0 and t < max_iters:
        t += 1
        new = jacobi_map(blk, u[active], v[active])
        m = np.abs(new - u[active]).max(axis=1)
        u[active] = new
        iters[active] = t
        if tau >= 0:
            active = active[m > tau]
    return u, iters


def model_forward(blocks, x):
    """x -> z through layers K-1 .. 0, logdet = -sum alpha."""
    s = np.asarray(x, dtype=np.float64)
    logdet = np.zeros(s.shape[0])
    for g in reversed(range(len(blocks))):
        v, ld = block_forward(blocks[g], np.ascontiguousarray(permute(s, g)))
        s = np.ascontiguousarray(permute(v, g))
        logdet += ld
    return s, logdet


def model_inverse(blocks, z, tau, max_iters, jacobi=True):
    """z -> x through layers 0 .. K-1.  jacobi: Algorithm 1 on every layer (App. E.3), else sequential decoding.
    Returns (x, iters[K, B]); a sequentially decoded layer reports D passes."""
    s = np.asarray(z, dtype=np.float64)
    B, D = s.shape
    iters = np.zeros((len(blocks), B), dtype=np.int64)
    for g in range(len(blocks)):
        v = np.ascontiguousarray(permute(s, g))
        if jacobi:
            u, it = block_inverse_jacobi(blocks[g], v, tau, max_iters)
            iters[g] = it
        else:
            u = block_inverse_sequential(blocks[g], v)
            iters[g] = D
        s = np.ascontiguousarray(permute(u, g))
    return s, iters
