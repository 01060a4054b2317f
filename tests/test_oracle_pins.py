"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle's code.

Each test is chosen so that one plausible mistake (dropped term, wrong sign, off-by-one shift,
causality leak, transposed operand, wrong reduction axis) fails it.
"""
import math
import os

import numpy as np
import pytest

from oracle import tarflow_oracle as O
from paper_2505_24791_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _load(name):
    rows = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append([float(t) for t in line.split()])
    return rows


def _model(head_scale=0.6, seed=11, **kw):
    cfg = synth.micro_config(**kw)
    blocks = synth.make_weights(cfg, seed=seed, head_scale=head_scale)
    # larger residual-path weights so the network depends visibly on its input
    for blk in blocks:
        for k in blk:
            if k.split(".")[-1] in ("w_in", "w_qkv", "w_o", "w_1", "w_2"):
                blk[k] = blk[k] * np.float32(2.0)
    return cfg, blocks


# ---------------------------------------------------------------- layout
def test_patchify_matches_hand_worked_example():
    x = np.arange(16, dtype=np.float64).reshape(1, 1, 4, 4)
    want = np.array(_load("patchify_1x4x4_p2.txt"))
    got = O.patchify(x, 2)
    assert got.shape == (1, 4, 4)
    assert np.array_equal(got[0], want)
    assert np.array_equal(O.unpatchify(got, 1, 4, 4, 2), x)


def test_patchify_channel_major_inside_token_and_roundtrip():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((2, 3, 4, 6))
    t = O.patchify(x, 2)
    # token 4 = grid (1,1); element (c=2, py=1, px=0) sits at index 2*4 + 1*2 + 0
    assert t[1, 4, 2 * 4 + 2] == x[1, 2, 3, 2]
    assert np.array_equal(O.unpatchify(t, 3, 4, 6, 2), x)


def test_permutation_is_an_involution_and_identity_on_even_blocks():
    s = np.arange(24.0).reshape(2, 4, 3)
    assert np.array_equal(O.permute(s, 0), s)
    assert np.array_equal(O.permute(s, 1)[:, 0], s[:, 3])
    assert np.array_equal(O.permute(O.permute(s, 3), 3), s)


# ---------------------------------------------------------------- textbook pieces
def test_gelu_against_gaussian_cdf_table():
    for x, phi in _load("gaussian_cdf.txt"):
        assert O.gelu(np.array([x]))[0] == pytest.approx(x * phi, abs=1e-14)


def test_layer_norm_statistics_and_affine():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((5, 64)) * 3 + 2
    y = O.layer_norm(x, np.ones(64), np.zeros(64))
    assert np.allclose(y.mean(-1), 0, atol=1e-12)
    assert np.allclose((y ** 2).mean(-1), x.var(-1) / (x.var(-1) + 1e-5), rtol=1e-12)
    g, b = rng.standard_normal(64), rng.standard_normal(64)
    assert np.allclose(O.layer_norm(x, g, b), y * g + b)
    # invariant to shift and (up to eps) to scale of the input
    assert np.allclose(O.layer_norm(x + 7.0, g, b), O.layer_norm(x, g, b), atol=1e-9)


def test_attention_special_cases():
    rng = np.random.default_rng(2)
    B, L, d, nh = 2, 5, 8, 2
    q, k, v = (rng.standard_normal((B, L, d)) for _ in range(3))
    o = O.causal_attention(q, k, v, nh)
    # first position attends only to itself: softmax over one score is 1
    assert np.allclose(o[:, 0], v[:, 0])
    # identical keys -> uniform weights -> running mean of the values
    kc = np.broadcast_to(k[:, :1], k.shape)
    o2 = O.causal_attention(q, kc, v, nh)
    run_mean = np.cumsum(v, axis=1) / np.arange(1, L + 1)[None, :, None]
    assert np.allclose(o2, run_mean)


def test_attention_against_scalar_loops():
    rng = np.random.default_rng(3)
    B, L, d, nh = 1, 4, 6, 3
    hd = d // nh
    q, k, v = (rng.standard_normal((B, L, d)) for _ in range(3))
    o = O.causal_attention(q, k, v, nh)
    for h in range(nh):
        for i in range(L):
            sc = [sum(q[0, i, h * hd + c] * k[0, j, h * hd + c] for c in range(hd)) / math.sqrt(hd)
                  for j in range(i + 1)]
            mx = max(sc)
            e = [math.exp(s - mx) for s in sc]
            for c in range(hd):
                want = sum(e[j] * v[0, j, h * hd + c] for j in range(i + 1)) / sum(e)
                assert o[0, i, h * hd + c] == pytest.approx(want, abs=1e-13)


def test_linear_is_x_times_w_transposed():
    w = np.array([[1.0, 2.0, 3.0], [4.0, 5.0, 6.0]])      # [out=2, in=3]
    x = np.array([[1.0, 0.0, -1.0]])
    assert np.array_equal(O.linear(x, w, np.array([10.0, 20.0])), [[8.0, 18.0]])


# ---------------------------------------------------------------- structure of one block
def test_dependence_is_strictly_lower_triangular():
    """(mu_l, alpha_l) must not move when u_j, j >= l, moves (Eq. 4: functions of u_<l only)."""
    cfg, blocks = _model()
    L, D = synth.seq_len(cfg), synth.token_dim(cfg)
    rng = np.random.default_rng(4)
    u = rng.standard_normal((1, L, D))
    mu0, al0 = O.block_params(blocks[0], u, None, cfg)
    assert np.all(mu0[:, 0] == 0) and np.all(al0[:, 0] == 0)
    moved_below = False
    for j in range(L):
        up = u.copy()
        up[0, j, :] += 0.37
        mu1, al1 = O.block_params(blocks[0], up, None, cfg)
        assert np.array_equal(mu1[:, :j + 1], mu0[:, :j + 1])
        assert np.array_equal(al1[:, :j + 1], al0[:, :j + 1])
        if j + 1 < L:
            # ... and the very next position does depend on u_j (shift is by exactly one)
            moved_below |= bool(np.any(mu1[:, j + 1] != mu0[:, j + 1]))
            assert np.any(mu1[:, j + 1] != mu0[:, j + 1])
    assert moved_below


def test_forward_and_sequential_inverse_are_mutual_inverses():
    cfg, blocks = _model(H=2, W=6, patch=1, C=2, n_blocks=3)
    rng = np.random.default_rng(5)
    z = rng.standard_normal((2, cfg["C"], cfg["H"], cfg["W"]))
    x = O.model_inverse_sequential(blocks, z, None, cfg)
    assert np.abs(x - z).max() > 1e-2            # the flow is not the identity
    z2, _ = O.model_forward(blocks, x, None, cfg)
    assert np.abs(z2 - z).max() < 1e-10
    x2 = O.model_inverse_sequential(blocks, z2, None, cfg)
    assert np.abs(x2 - x).max() < 1e-10
    # and starting from the data side
    xd = rng.standard_normal(z.shape)
    zd, _ = O.model_forward(blocks, xd, None, cfg)
    assert np.abs(O.model_inverse_sequential(blocks, zd, None, cfg) - xd).max() < 1e-10


def test_logdet_equals_bruteforce_jacobian_determinant():
    """Eq. 1: logdet of x -> z; compared with log|det| of the central-difference Jacobian."""
    cfg, blocks = _model(H=2, W=2, patch=1, C=2, n_blocks=2, head_scale=0.8)
    rng = np.random.default_rng(6)
    x = rng.standard_normal((1, cfg["C"], cfg["H"], cfg["W"]))
    z, logdet = O.model_forward(blocks, x, None, cfg)
    n = x.size
    J = np.zeros((n, n))
    eps = 1e-6
    for i in range(n):
        dx = np.zeros(n)
        dx[i] = eps
        zp, _ = O.model_forward(blocks, x + dx.reshape(x.shape), None, cfg)
        zm, _ = O.model_forward(blocks, x - dx.reshape(x.shape), None, cfg)
        J[:, i] = (zp - zm).reshape(-1) / (2 * eps)
    sign, lad = np.linalg.slogdet(J)
    assert sign > 0
    assert abs(logdet[0]) > 0.05
    assert logdet[0] == pytest.approx(lad, abs=1e-6)


def test_logdet_is_minus_sum_alpha_per_sample():
    cfg, blocks = _model(n_blocks=1)
    rng = np.random.default_rng(7)
    u = rng.standard_normal((3, synth.seq_len(cfg), synth.token_dim(cfg)))
    _, alpha = O.block_params(blocks[0], u, None, cfg)
    _, ld = O.block_forward(blocks[0], u, None, cfg)
    for b in range(3):
        assert ld[b] == pytest.approx(-sum(alpha[b].reshape(-1)), abs=1e-12)


def test_cached_sequential_equals_uncached():
    cfg, blocks = _model(H=2, W=5, patch=1, C=2, n_layers=2)
    rng = np.random.default_rng(8)
    v = rng.standard_normal((2, synth.seq_len(cfg), synth.token_dim(cfg)))
    a = O.block_inverse_sequential(blocks[0], v, None, cfg)
    b = O.block_inverse_sequential_uncached(blocks[0], v, None, cfg)
    assert np.abs(a - b).max() < 1e-12


# ---------------------------------------------------------------- Jacobi iteration (Alg. 1, Prop. 3.2)
def test_prop_3_2_prefix_exactness_and_finite_convergence():
    cfg, blocks = _model(H=2, W=6, patch=1, C=2, head_scale=1.0)
    L = synth.seq_len(cfg)
    rng = np.random.default_rng(9)
    v = rng.standard_normal((2, L, synth.token_dim(cfg)))
    u_star = O.block_inverse_sequential(blocks[0], v, None, cfg)
    u = np.zeros_like(v)
    errs = []
    for t in range(1, L + 2):
        u = O.jacobi_map(blocks[0], u, v, None, cfg)
        assert np.abs(u[:, :t] - u_star[:, :t]).max() < 1e-12, f"first {t} tokens after {t} sweeps"
        errs.append(np.abs(u - u_star).max())
    assert errs[0] > 1e-3                       # not converged after one sweep: the test has teeth
    assert errs[L - 1] < 1e-12                  # u^L = u*
    assert errs[L] < 1e-12                      # stays there
    # fixed point: F(u*) = u*
    assert np.abs(O.jacobi_map(blocks[0], u_star, v, None, cfg) - u_star).max() < 1e-12


def test_jacobi_fixed_iterations_equals_sequential_and_counts():
    cfg, blocks = _model(H=2, W=4, patch=1, C=1)
    L = synth.seq_len(cfg)
    rng = np.random.default_rng(10)
    v = rng.standard_normal((3, L, synth.token_dim(cfg)))
    u_star = O.block_inverse_sequential(blocks[0], v, None, cfg)
    u, it, trace = O.block_inverse_jacobi(blocks[0], v, None, cfg, -1.0, L, u_star=u_star)
    assert np.all(it == L) and len(trace) == L
    assert np.abs(u - u_star).max() < 1e-12
    assert np.all(trace[-1] < 1e-12)
    # tau mode: stops within L+1 sweeps, at least 2, and the answer is within the method's own bound
    u2, it2, _ = O.block_inverse_jacobi(blocks[0], v, None, cfg, 1e-9, L + 1)
    assert np.all(it2 >= 2) and np.all(it2 <= L + 1)
    assert np.abs(u2 - u_star).max() < 1e-6


def test_per_sample_stopping_is_independent_of_batch_mates():
    cfg, blocks = _model(H=2, W=6, patch=1, C=2, head_scale=0.5)
    L = synth.seq_len(cfg)
    rng = np.random.default_rng(12)
    v = rng.standard_normal((4, L, synth.token_dim(cfg)))
    v[1] *= 0.01                                  # samples of different scale side by side
    u, it, _ = O.block_inverse_jacobi(blocks[0], v, None, cfg, 1e-4, L + 1)
    for b in range(4):
        ub, itb, _ = O.block_inverse_jacobi(blocks[0], v[b:b + 1], None, cfg, 1e-4, L + 1)
        assert itb[0] == it[b]
        assert np.array_equal(ub[0], u[b])
    assert len(set(it.tolist())) > 1              # the samples really stop at different sweeps


def test_zero_head_makes_every_block_the_identity_and_jacobi_stops_at_sweep_two():
    cfg = synth.micro_config(H=2, W=4, n_blocks=3)
    blocks = synth.make_weights(cfg, seed=3, zero_head=True)
    rng = np.random.default_rng(13)
    z = rng.standard_normal((2, cfg["C"], cfg["H"], cfg["W"]))
    x, it = O.model_inverse(blocks, z, None, cfg, [1, 1, 1], 0.0, 10)
    assert np.array_equal(x, z)
    assert np.all(it == 2)                        # sweep 1: 0 -> v (diff |v|), sweep 2: no change
    zf, ld = O.model_forward(blocks, z, None, cfg)
    assert np.array_equal(zf, z) and np.all(ld == 0)


def test_policy_variants_agree():
    cfg, blocks = _model(H=2, W=4, patch=1, C=2, n_blocks=3)
    L = synth.seq_len(cfg)
    rng = np.random.default_rng(14)
    z = rng.standard_normal((2, cfg["C"], cfg["H"], cfg["W"]))
    x_seq = O.model_inverse_sequential(blocks, z, None, cfg)
    x_all, it_all = O.model_inverse(blocks, z, None, cfg, [1, 1, 1], -1.0, L)
    x_sel, it_sel = O.model_inverse(blocks, z, None, cfg, [0, 1, 1], -1.0, L)
    assert np.abs(x_all - x_seq).max() < 1e-11
    assert np.abs(x_sel - x_seq).max() < 1e-11
    assert np.all(it_sel[0] == L - 1) and np.all(it_sel[1:] == L)
    # uncached sequential path through the whole model
    x_unc, _ = O.model_inverse(blocks, z, None, cfg, [0, 0, 0], 0.0, 0, cached=False)
    assert np.abs(x_unc - x_seq).max() < 1e-11


def test_reversal_lets_every_position_be_transformed():
    """With one block the first token passes through; with two (reversed) blocks none does."""
    cfg, blocks = _model(H=1, W=5, patch=1, C=1, n_blocks=2)
    rng = np.random.default_rng(15)
    z = rng.standard_normal((1, 1, 1, 5))
    cfg1 = dict(cfg, n_blocks=1)
    x1 = O.model_inverse_sequential(blocks[:1], z, None, cfg1)
    assert x1[0, 0, 0, 0] == z[0, 0, 0, 0]
    assert np.all(x1[0, 0, 0, 1:] != z[0, 0, 0, 1:])
    x2 = O.model_inverse_sequential(blocks, z, None, cfg)
    assert np.all(x2 != z)
    # block 1 works on the reversed sequence: its pass-through token is the last raster position
    assert x2[0, 0, 0, 4] == x1[0, 0, 0, 4]


def test_sequential_step_count_matches_paper_table():
    for L, steps in _load("paper_sequential_steps.txt"):
        assert steps == L - 1
    cfg, blocks = _model(H=2, W=4)
    z = np.zeros((1, cfg["C"], cfg["H"], cfg["W"]))
    _, it = O.model_inverse(blocks, z, None, cfg, [0, 1], 1e-3, 9)
    assert np.all(it[0] == synth.seq_len(cfg) - 1)


def test_class_conditioning_changes_output_only_through_label():
    cfg, blocks = _model(H=2, W=4, n_classes=5)
    rng = np.random.default_rng(16)
    z = rng.standard_normal((2, cfg["C"], cfg["H"], cfg["W"]))
    z[1] = z[0]
    x = O.model_inverse_sequential(blocks, z, np.array([1, 1]), cfg)
    assert np.array_equal(x[0], x[1])
    x = O.model_inverse_sequential(blocks, z, np.array([1, 3]), cfg)
    assert np.abs(x[0] - x[1]).max() > 1e-6
    zz, _ = O.model_forward(blocks, x, np.array([1, 3]), cfg)
    assert np.abs(zz - z).max() < 1e-10


def test_cfg1_selective_policy_close_to_sequential():
    """The tiny benchmark configuration: selective Jacobi at tau = 1e-5 lands on the sequential answer."""
    cfg = synth.config("cfg1")
    blocks = synth.make_weights(cfg)
    z = synth.make_latents(cfg, 2025)
    L = synth.seq_len(cfg)
    x_seq = O.model_inverse_sequential(blocks, z, None, cfg)
    x, it = O.model_inverse(blocks, z, None, cfg, [0, 1], cfg["tau"], L + 1)
    assert np.all(it[1] >= 2) and np.all(it[1] <= L + 1)
    assert np.abs(x - x_seq).max() < 1e-4
    z2, ld = O.model_forward(blocks, x_seq, None, cfg)
    assert np.abs(z2 - z).max() < 1e-9


# ---------------------------------------------------------------- variants around Algorithm 1
def test_any_initial_iterate_reaches_the_sequential_solution_in_L_sweeps():
    """Prop. 3.2's induction never uses u^0: from zeros, from the block input and from random draws, L sweeps
    give the sequential solution exactly and after t sweeps the first t tokens are already exact."""
    cfg, blocks = _model(H=2, W=5, patch=1, C=2, n_blocks=2)
    L = synth.seq_len(cfg)
    rng = np.random.default_rng(21)
    z = rng.standard_normal((3, cfg["C"], cfg["H"], cfg["W"]))
    u0 = rng.standard_normal((2, 3, cfg["C"], cfg["H"], cfg["W"]))
    x_seq = O.model_inverse_sequential(blocks, z, None, cfg)
    for mode in (0, 1, 2):
        x, it = O.model_inverse(blocks, z, None, cfg, [1, 1], -1.0, L, init_mode=mode, u0=u0)
        assert np.abs(x - x_seq).max() < 1e-12 and np.all(it == L)
    # the start really is used: after one sweep only token 1 is fixed (it copies v_1), the rest depends on u^0
    v = O.patchify(z, 1)
    outs = [O.block_inverse_jacobi(blocks[0], v, None, cfg, -1.0, 1, u0=s)[0]
            for s in (None, v, O.patchify(u0[0], 1))]
    assert np.array_equal(outs[0][:, :1], outs[1][:, :1]) and np.array_equal(outs[0][:, :1], outs[2][:, :1])
    assert np.abs(outs[0][:, 1:] - outs[1][:, 1:]).max() > 1e-3 and np.abs(outs[0][:, 1:] - outs[2][:, 1:]).max() > 1e-3


def test_per_block_tau_equals_uniform_tau_blockwise_and_states_chain():
    cfg, blocks = _model(H=2, W=4, patch=1, C=2, n_blocks=3, head_scale=0.3)
    L = synth.seq_len(cfg)
    rng = np.random.default_rng(22)
    z = rng.standard_normal((2, cfg["C"], cfg["H"], cfg["W"]))
    taus = [1e-2, 1e-6, 1e-4]
    x, it, ex = O.model_inverse(blocks, z, None, cfg, [1, 1, 1], taus, L + 1, return_states=True)
    # chaining single blocks by hand with each block's own tau gives the same states and counts
    seq = O.patchify(z, 1)
    for g in range(3):
        u, itg, _ = O.block_inverse_jacobi(blocks[g], np.ascontiguousarray(O.permute(seq, g)), None, cfg, taus[g], L + 1)
        seq = np.ascontiguousarray(O.permute(u, g))
        assert np.array_equal(O.unpatchify(seq, cfg["C"], cfg["H"], cfg["W"], 1), ex["states"][g])
        assert np.array_equal(itg, it[g])
    assert np.array_equal(ex["states"][-1], x)
    assert it[1].min() > it[0].max()            # the tighter threshold costs sweeps
    xu, itu = O.model_inverse(blocks, z, None, cfg, [1, 1, 1], 1e-6, L + 1)
    xl, itl = O.model_inverse(blocks, z, None, cfg, [1, 1, 1], [1e-6] * 3, L + 1)
    assert np.array_equal(xu, xl) and np.array_equal(itu, itl)


def test_fallback_decodes_exactly_the_stragglers_sequentially():
    cfg, blocks = _model(H=2, W=6, patch=1, C=2, n_blocks=1, head_scale=0.5)
    L = synth.seq_len(cfg)
    rng = np.random.default_rng(12)
    z = rng.standard_normal((4, cfg["C"], cfg["H"], cfg["W"]))
    x_plain, it_plain = O.model_inverse(blocks, z, None, cfg, [1], 1e-3, L + 1)
    x_seq = O.model_inverse_sequential(blocks, z, None, cfg)
    cut = int(it_plain[0].min()) + 1             # some samples are done by then, others are not
    assert it_plain[0].min() <= cut < it_plain[0].max()
    x_fb, it_fb = O.model_inverse(blocks, z, None, cfg, [1], 1e-3, L + 1, fallback_sweeps=cut)
    done = it_plain[0] <= cut
    assert done.any() and (~done).any()
    assert np.array_equal(x_fb[done], x_plain[done]) and np.array_equal(it_fb[0][done], it_plain[0][done])
    assert np.array_equal(x_fb[~done], x_seq[~done])            # bit-identical to Eq. 5 for the stragglers
    assert np.all(it_fb[0][~done] == cut + L - 1)
    # a cut that nobody reaches, a cut at or beyond max_iters, and fixed-iteration mode change nothing
    for kw in (dict(fallback_sweeps=int(it_plain.max())), dict(fallback_sweeps=L + 1)):
        x2, it2 = O.model_inverse(blocks, z, None, cfg, [1], 1e-3, L + 1, **kw)
        assert np.array_equal(x2, x_plain) and np.array_equal(it2, it_plain)
    x3, it3 = O.model_inverse(blocks, z, None, cfg, [1], -1.0, 5, fallback_sweeps=2)
    assert np.all(it3 == 5)


def test_distance_trace_matches_direct_norms_and_ends_at_zero():
    cfg, blocks = _model(H=2, W=4, patch=1, C=2, n_blocks=2)
    L = synth.seq_len(cfg)
    rng = np.random.default_rng(23)
    z = rng.standard_normal((2, cfg["C"], cfg["H"], cfg["W"]))
    _, _, ref = O.model_inverse(blocks, z, None, cfg, [0, 0], 0.0, 1, return_states=True)
    x, it, ex = O.model_inverse(blocks, z, None, cfg, [1, 1], -1.0, L, ref_states=ref["states"], return_states=True)
    for g in range(2):
        tr = ex["l2"][g]
        assert tr.shape == (L, 2)
        assert np.all(tr[-1] < 1e-12)                          # u^L = sequential solution (Prop. 3.2)
        assert np.all(tr[0] > 1e-3)
        d = np.sqrt(((ex["states"][g] - ref["states"][g]) ** 2).reshape(2, -1).sum(axis=1))
        assert np.allclose(tr[-1], d, atol=1e-12)
