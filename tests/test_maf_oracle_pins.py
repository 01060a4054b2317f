"""Pins for the MAF oracle: what the MADE construction, Eq. 4 / Eq. 5 and Prop. 3.2 fix, independent of its code."""
import itertools

import numpy as np

from oracle import maf_oracle as M
from paper_2505_24791_b200 import synth


def _model(D=7, hidden=10, n_blocks=3, out_scale=0.6, seed=5):
    cfg = synth.maf_config("maf_tiny", D=D, hidden=hidden, n_blocks=n_blocks)
    return cfg, synth.make_maf_weights(cfg, seed=seed, out_scale=out_scale)


def test_mask_connectivity_by_brute_force_over_paths():
    """Output i is connected to input j through some (hidden 1, hidden 2) path iff j < i; this enumerates every path."""
    for D, H in ((5, 6), (4, 9), (6, 5)):
        m1, m2, m3 = M.masks(D, H)
        assert m1.shape == (H, D) and m2.shape == (H, H) and m3.shape == (2 * D, H)
        for i, j in itertools.product(range(D), range(D)):
            connected = any(m3[i, b] and m2[b, a] and m1[a, j] for a in range(H) for b in range(H))
            if j >= i:
                assert not connected                       # never sees itself or later inputs
            elif H >= D - 1:
                assert connected                           # every earlier input is reachable when all degrees occur
        assert np.array_equal(m3[:D], m3[D:])               # mu_i and alpha_i have the same inputs
        assert not m3[0].any() and not m3[D].any()          # the first output is a constant


def test_dependence_is_strictly_lower_triangular():
    cfg, blocks = _model(hidden=48)
    rng = np.random.default_rng(1)
    u = rng.standard_normal((2, cfg["D"]))
    mu0, al0 = M.made_params(blocks[0], u)
    for j in range(cfg["D"]):
        up = u.copy()
        up[:, j] += 0.37
        mu1, al1 = M.made_params(blocks[0], up)
        assert np.array_equal(mu1[:, :j + 1], mu0[:, :j + 1]) and np.array_equal(al1[:, :j + 1], al0[:, :j + 1])
        if j < cfg["D"] - 1:
            assert np.abs(mu1[:, j + 1:] - mu0[:, j + 1:]).max() > 0 or np.abs(al1[:, j + 1:] - al0[:, j + 1:]).max() > 0
    # the first output is the bias of the output layer
    assert np.allclose(mu0[:, 0], blocks[0]["b3"][0]) and np.allclose(al0[:, 0], blocks[0]["b3"][cfg["D"]])


def test_forward_and_sequential_inverse_are_mutual_inverses_and_logdet_is_the_jacobian():
    cfg, blocks = _model(D=5, hidden=8, n_blocks=3)
    rng = np.random.default_rng(2)
    z = rng.standard_normal((3, cfg["D"]))
    x, it = M.model_inverse(blocks, z, 0.0, 0, jacobi=False)
    assert np.all(it == cfg["D"])
    zf, ld = M.model_forward(blocks, x)
    assert np.abs(zf - z).max() < 1e-12
    x2, _ = M.model_inverse(blocks, M.model_forward(blocks, x)[0], 0.0, 0, jacobi=False)
    assert np.abs(x2 - x).max() < 1e-12
    # log|det dz/dx| by central differences on the whole 3-layer flow
    eps = 1e-6
    for b in range(2):
        J = np.zeros((cfg["D"], cfg["D"]))
        for j in range(cfg["D"]):
            xp, xm = x[b:b + 1].copy(), x[b:b + 1].copy()
            xp[0, j] += eps
            xm[0, j] -= eps
            J[:, j] = (M.model_forward(blocks, xp)[0][0] - M.model_forward(blocks, xm)[0][0]) / (2 * eps)
        assert abs(np.log(abs(np.linalg.det(J))) - ld[b]) < 1e-6
    # and the closed form: -sum of alpha over layers
    s, tot = x.copy(), np.zeros(3)
    for g in reversed(range(3)):
        u = np.ascontiguousarray(M.permute(s, g))
        mu, al = M.made_params(blocks[g], u)
        tot -= al.sum(axis=1)
        s = np.ascontiguousarray(M.permute((u - mu) * np.exp(-al), g))
    assert np.abs(tot - ld).max() < 1e-12


def test_prop_3_2_prefix_exactness_finite_convergence_and_fixed_point():
    cfg, blocks = _model(D=9, hidden=12, n_blocks=1)
    D = cfg["D"]
    rng = np.random.default_rng(3)
    v = rng.standard_normal((3, D))
    u_star = M.block_inverse_sequential(blocks[0], v)
    u = np.zeros_like(v)
    for t in range(1, D + 2):
        u = M.jacobi_map(blocks[0], u, v)
        assert np.abs(u[:, :t] - u_star[:, :t]).max() < 1e-13          # first t values exact after t sweeps
        if t == 1:
            assert np.abs(u[:, 2:] - u_star[:, 2:]).max() > 1e-6       # and the rest is not there yet
    assert np.abs(M.jacobi_map(blocks[0], u_star, v) - u_star).max() < 1e-13   # fixed point
    uj, it = M.block_inverse_jacobi(blocks[0], v, -1.0, D)
    assert np.all(it == D) and np.abs(uj - u_star).max() < 1e-13
    ut, itt = M.block_inverse_jacobi(blocks[0], v, 1e-10, D + 1)
    assert np.all(itt >= 2) and np.all(itt <= D + 1) and np.abs(ut - u_star).max() < 1e-8


def test_reversal_between_layers_and_zero_output_identity():
    cfg, blocks = _model(D=6, hidden=7, n_blocks=2)
    rng = np.random.default_rng(4)
    z = rng.standard_normal((2, 6))
    # layer 1 works on the reversed order: its first (constant-parameter) dimension is the last raster dimension
    x, _ = M.model_inverse(blocks, z, 0.0, 0, jacobi=False)
    s0 = M.block_inverse_sequential(blocks[0], z)
    s1 = M.block_inverse_sequential(blocks[1], np.ascontiguousarray(s0[:, ::-1]))[:, ::-1]
    assert np.array_equal(x, s1)
    b3 = blocks[1]["b3"].astype(np.float64)
    assert np.allclose(x[:, -1], s0[:, -1] * np.exp(b3[6]) + b3[0])
    cfg0 = synth.maf_config("maf_tiny", D=6, hidden=7, n_blocks=2)
    ident = synth.make_maf_weights(cfg0, zero_out=True)
    xi, it = M.model_inverse(ident, z, 0.0, 10)
    assert np.array_equal(xi, z) and np.all(it == 2)


def test_per_sample_stopping_is_independent_of_batch_mates():
    cfg, blocks = _model(D=10, hidden=16, n_blocks=1, out_scale=0.8)
    rng = np.random.default_rng(6)
    v = rng.standard_normal((4, 10))
    v[2] *= 0.01
    u, it = M.block_inverse_jacobi(blocks[0], v, 1e-5, 11)
    for b in range(4):
        ub, itb = M.block_inverse_jacobi(blocks[0], v[b:b + 1], 1e-5, 11)
        assert itb[0] == it[b] and np.abs(ub[0] - u[b]).max() < 1e-13
