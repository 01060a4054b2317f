"""GPU parity: the CUDA library, called through its C ABI, against the fp64 CPU oracle.

Tolerances (from the build contract): fp32 engine max|dx| <= 1e-4 in fixed-iteration mode; bf16
engine relative L2 error on x <= 2e-2 and sweep counts per block within +-1 of the oracle.
"""
import numpy as np
import pytest
import torch

from oracle import tarflow_oracle as O
from paper_2505_24791_b200 import binding, synth
from tests.gpu_util import Model, rel_l2

pytestmark = pytest.mark.gpu

FP32_TOL = 1e-4
BF16_REL_L2 = 2e-2
BF16_MAX_ABS = 5e-2   # element-wise companion of the norm: no entry may be off by more than this


def bf16_close(x, xo):
    """Relative L2 within the contract's tolerance and no single entry far off."""
    return bool(np.isfinite(x).all() and rel_l2(x, xo) <= BF16_REL_L2 and np.abs(x - xo).max() <= BF16_MAX_ABS)


# ---------------------------------------------------------------- single kernels
def test_jacobi_update_kernel_matches_oracle_map():
    """First kernel: Algorithm 1's update line + per-sample max-norm, fed the oracle's head output."""
    cfg = synth.config("cfg1")
    blocks = synth.make_weights(cfg, head_scale=0.5)
    L, D, B = synth.seq_len(cfg), synth.token_dim(cfg), 3
    rng = np.random.default_rng(0)
    v = rng.standard_normal((B, L, D))
    u_prev = rng.standard_normal((B, L, D))
    for g in (0, 1):
        o = O.head_raw(blocks[g], O.permute(u_prev, g), None, cfg)                 # [B,L,2D] in core order
        want = O.permute(O.jacobi_map(blocks[g], O.permute(u_prev, g), O.permute(v, g), None, cfg), g)
        want32_in = [torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda() for a in (o, v, u_prev)]
        md = torch.full((B,), -1.0, dtype=torch.float32, device="cuda")
        binding.tf_jacobi_update(want32_in[0], want32_in[1], want32_in[2], md, B, L, D, g % 2)
        torch.cuda.synchronize()
        got = want32_in[2].cpu().numpy().astype(np.float64)
        assert np.abs(got - want).max() < 5e-6
        want_md = np.abs(want - u_prev).reshape(B, -1).max(axis=1)
        assert np.abs(md.cpu().numpy() - want_md).max() < 5e-6


@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (256, 128, 128), (384, 512, 1024), (200, 96, 512), (1000, 24, 512),
                                   (16384 + 128, 1024, 1024), (333, 384, 192)])
def test_tensor_core_gemm_matches_fp64_matmul(M, N, K):
    rng = np.random.default_rng(M + N + K)
    a = synth.round_to_bf16(rng.standard_normal((M, K)).astype(np.float32))
    w = synth.round_to_bf16((rng.standard_normal((N, K)) / np.sqrt(K)).astype(np.float32))
    bias = rng.standard_normal(N).astype(np.float32)
    at = torch.from_numpy(a).cuda().to(torch.bfloat16)
    wt = torch.from_numpy(w).cuda().to(torch.bfloat16)
    bt = torch.from_numpy(bias).cuda()
    ct = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    binding.tf_gemm_bf16(at, wt, bt, ct, M, N, K)
    assert binding.tf_gemm_status() == 0
    want = O.linear(a.astype(np.float64), w.astype(np.float64), bias.astype(np.float64))
    got = ct.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    assert np.abs(got - want).max() < 2e-4 * max(1.0, np.sqrt(K) / 8)


# ---------------------------------------------------------------- fp32 engine, tiny configuration
@pytest.fixture(scope="module")
def cfg1_model():
    with Model(synth.config("cfg1"), max_batch=6) as m:
        yield m


def test_cfg1_fixed_iteration_parity(cfg1_model):
    m = cfg1_model
    z = synth.make_latents(m.cfg, 2025)
    x, ib, its, rc = m.inverse(z, None, [0, 1], -1.0, 7)
    xo, ito = O.model_inverse(m.blocks, z, None, m.cfg, [0, 1], -1.0, 7)
    assert rc == 0 and list(ib) == [m.L - 1, 7]
    assert np.abs(x - xo).max() <= FP32_TOL
    assert np.array_equal(its, ito)


def test_cfg1_selective_tau_mode_parity_and_counts(cfg1_model):
    m = cfg1_model
    z = synth.make_latents(m.cfg, 2026)
    x, ib, its, rc = m.inverse(z, None, [0, 1], m.cfg["tau"], m.L + 1)
    xo, ito = O.model_inverse(m.blocks, z, None, m.cfg, [0, 1], m.cfg["tau"], m.L + 1)
    assert rc == 0
    assert np.abs(x - xo).max() <= FP32_TOL
    assert np.abs(its - ito).max() <= 1
    assert ib[1] == its[1].max() and ib[0] == m.L - 1


def test_cfg1_sequential_and_prop_3_2_on_gpu(cfg1_model):
    """All-Jacobi with L fixed sweeps reproduces sequential decoding (Prop. 3.2), both vs the oracle."""
    m = cfg1_model
    z = synth.make_latents(m.cfg, 2027)
    xs = m.inverse_sequential(z, None)
    xo = O.model_inverse_sequential(m.blocks, z, None, m.cfg)
    assert np.abs(xs - xo).max() <= FP32_TOL
    xj, ib, _, rc = m.inverse(z, None, [1, 1], -1.0, m.L)
    assert rc == 0 and list(ib) == [m.L, m.L]
    assert np.abs(xj - xo).max() <= FP32_TOL
    xp, _, _, _ = m.inverse(z, None, [0, 0], 0.0, 1)
    assert np.array_equal(xp, xs)


def test_cfg1_forward_roundtrip_and_logdet(cfg1_model):
    m = cfg1_model
    z = synth.make_latents(m.cfg, 2028)
    xo = O.model_inverse_sequential(m.blocks, z, None, m.cfg)
    zg, ld = m.forward(xo, None)
    zo, ldo = O.model_forward(m.blocks, xo, None, m.cfg)
    assert np.abs(zg - zo).max() <= FP32_TOL
    assert np.abs(zg - z).max() <= 2 * FP32_TOL
    assert np.abs(ld - ldo).max() <= 1e-3 * max(1.0, np.abs(ldo).max())


def test_cfg1_batch_sizes_and_sample_independence(cfg1_model):
    m = cfg1_model
    z = synth.make_latents(m.cfg, 2029, B=6)
    x6, _, it6, _ = m.inverse(z, None, [0, 1], 1e-4, m.L + 1)
    x1, _, it1, _ = m.inverse(z[2:3], None, [0, 1], 1e-4, m.L + 1)
    assert np.abs(x6[2] - x1[0]).max() <= 1e-5
    assert abs(int(it6[1, 2]) - int(it1[1, 0])) <= 1


def test_cfg1_init_from_input_converges_to_same_answer(cfg1_model):
    m = cfg1_model
    z = synth.make_latents(m.cfg, 2030)
    xo = O.model_inverse_sequential(m.blocks, z, None, m.cfg)
    x, _, _, rc = m.inverse(z, None, [0, 1], 1e-6, m.L + 1, init_mode=1)
    assert rc == 0 and np.abs(x - xo).max() <= FP32_TOL


def test_zero_head_is_identity_and_two_sweeps():
    cfg = synth.config("cfg1")
    with Model(cfg, zero_head=True) as m:
        z = synth.make_latents(cfg, 5)
        x, ib, its, rc = m.inverse(z, None, [1, 1], 0.0, 10)
        assert rc == 0 and np.array_equal(x, z.astype(np.float64))
        assert list(ib) == [2, 2] and np.all(its == 2)


def test_max_iters_status_and_error_codes(cfg1_model):
    m = cfg1_model
    z = synth.make_latents(m.cfg, 2031)
    _, ib, _, rc = m.inverse(z, None, [0, 1], 1e-7, 2)
    assert rc == binding.TF_MAXITER and ib[1] == 2
    zt = torch.from_numpy(z).cuda()
    xt = torch.empty_like(zt)
    for kwargs in (dict(B=0), dict(B=7), dict(max_iters=0), dict(init_mode=5), dict(policy=[0, 2])):
        a = dict(B=4, policy=[0, 1], max_iters=3, init_mode=0)
        a.update(kwargs)
        with pytest.raises(binding.TarflowError) as e:
            binding.tf_inverse_jacobi(m.m, zt, None, a["B"], a["policy"], 1e-3, a["max_iters"], a["init_mode"], xt)
        assert e.value.code == binding.TF_EINVAL
    with pytest.raises(binding.TarflowError) as e:
        binding.tf_load(m.cfg, m.blob[:-4], 4)
    assert e.value.code == binding.TF_ESIZE
    bad = m.blob.copy()
    bad.view(np.int32)[8] += 1
    with pytest.raises(binding.TarflowError) as e:
        binding.tf_load(m.cfg, bad, 4)
    assert e.value.code == binding.TF_ESIZE


def test_nan_input_is_reported_not_crashed(cfg1_model):
    m = cfg1_model
    z = synth.make_latents(m.cfg, 2032)
    z[1, 0, 3, 3] = np.nan
    zt = torch.from_numpy(z).cuda()
    xt = torch.empty_like(zt)
    with pytest.raises(binding.TarflowError) as e:
        binding.tf_inverse_jacobi(m.m, zt, None, 4, [0, 1], 1e-3, 5, 0, xt)
    assert e.value.code == binding.TF_ENONFINITE
    # the model is still usable afterwards
    x, _, _, rc = m.inverse(synth.make_latents(m.cfg, 2033), None, [0, 1], -1.0, 3)
    assert rc == 0 and np.isfinite(x).all()


# ---------------------------------------------------------------- fp32 engine, ragged sizes
def test_fp32_ragged_sizes_with_classes():
    cfg = synth.config("cfg1", H=10, W=6, patch=2, n_classes=7, width=96, n_heads=3, n_blocks=3)   # L=15, D=12
    with Model(cfg, max_batch=3) as m:
        z = synth.make_latents(cfg, 77, B=3)
        lab = synth.make_labels(cfg, B=3)
        x, ib, its, rc = m.inverse(z, lab, [0, 1, 1], -1.0, 5)
        xo, ito = O.model_inverse(m.blocks, z, lab, cfg, [0, 1, 1], -1.0, 5)
        assert rc == 0 and np.abs(x - xo).max() <= FP32_TOL
        zg, ld = m.forward(xo, lab)
        zo, ldo = O.model_forward(m.blocks, xo, lab, cfg)
        assert np.abs(zg - zo).max() <= FP32_TOL and np.abs(ld - ldo).max() <= 1e-3


# ---------------------------------------------------------------- bf16 tensor-core engine
def _bf16_case(cfg, B, seed, policy, tau, labels=None):
    with Model(cfg, max_batch=B) as m:
        z = synth.make_latents(cfg, seed, B=B)
        x, ib, its, rc = m.inverse(z, labels, policy, tau, m.L + 1)
        xo, ito = O.model_inverse(m.blocks, z, labels, cfg, policy, tau, m.L + 1)
        return m, x, xo, its, ito, rc


def test_bf16_small_model_selective_parity():
    """cfg2's architecture at a batch the oracle finishes quickly; M = 4*256 spans 8 GEMM row tiles."""
    cfg = synth.config("cfg2")
    m, x, xo, its, ito, rc = _bf16_case(cfg, 4, 2024, [0, 1, 1, 1], cfg["tau"])
    assert rc == 0
    assert bf16_close(x, xo)
    assert np.abs(its - ito).max() <= 1


def test_bf16_cfg2_full_batch_sampled_against_oracle():
    """The benchmark's launch configuration (cfg2, batch 64, selective policy, tau 1e-3): three samples of the
    batch are checked against the oracle one by one (samples are independent: per-sample stopping test), the
    rest through properties that hold at any size."""
    cfg = synth.config("cfg2")
    B = cfg["B"]
    policy = [0] + [1] * (cfg["n_blocks"] - 1)
    with Model(cfg, max_batch=B) as m:
        z = synth.make_latents(cfg, 1000, B=B)
        x, ib, its, rc = m.inverse(z, None, policy, cfg["tau"], m.L + 1)
        assert rc == 0 and np.isfinite(x).all()
        assert (its[0] == m.L - 1).all()                       # the sequential block reports L - 1 steps
        assert (its[1:] >= 2).all() and (its[1:] <= m.L).all()  # Jacobi: at least two sweeps, at most L (Prop. 3.2)
        pick = [0, 37, B - 1]
        xo, ito = O.model_inverse(m.blocks, z[pick], None, cfg, policy, cfg["tau"], m.L + 1)
        assert bf16_close(x[pick], xo)
        assert np.abs(its[:, pick] - ito).max() <= 1
        x2, _, its2, rc2 = m.inverse(z, None, policy, cfg["tau"], m.L + 1)  # run-twice determinism
        assert rc2 == 0 and np.array_equal(x, x2) and np.array_equal(its, its2)


def test_bf16_cfg3_full_batch_sampled_against_oracle():
    """cfg3 at its full size (8 blocks x 8 layers, width 1024, 1000 classes, batch 64): one sample of the batch
    against the oracle (about 45 s of CPU), sweep-count properties for all."""
    cfg = synth.config("cfg3")
    B = cfg["B"]
    policy = [0] + [1] * (cfg["n_blocks"] - 1)
    lab = synth.make_labels(cfg, B=B)
    with Model(cfg, max_batch=B) as m:
        z = synth.make_latents(cfg, 1000, B=B)
        x, ib, its, rc = m.inverse(z, lab, policy, cfg["tau"], m.L + 1)
        assert rc == 0 and np.isfinite(x).all()
        assert (its[0] == m.L - 1).all() and (its[1:] >= 2).all() and (its[1:] <= m.L).all()
        pick = [41]
        xo, ito = O.model_inverse(m.blocks, z[pick], lab[pick], cfg, policy, cfg["tau"], m.L + 1)
        assert bf16_close(x[pick], xo)
        assert np.abs(its[:, pick] - ito).max() <= 1


def test_bf16_all_jacobi_and_all_sequential_agree_with_oracle():
    cfg = synth.config("cfg2", n_blocks=2, n_layers=2)
    with Model(cfg, max_batch=3) as m:
        z = synth.make_latents(cfg, 99, B=3)
        xo = O.model_inverse_sequential(m.blocks, z, None, cfg)
        xs = m.inverse_sequential(z, None)
        assert bf16_close(xs, xo)
        xj, ib, its, rc = m.inverse(z, None, [1, 1], 1e-3, m.L + 1)
        xjo, ito = O.model_inverse(m.blocks, z, None, cfg, [1, 1], 1e-3, m.L + 1)
        assert rc == 0 and bf16_close(xj, xjo) and np.abs(its - ito).max() <= 1
        zg, ld = m.forward(xo, None)
        zo, ldo = O.model_forward(m.blocks, xo, None, cfg)
        assert bf16_close(zg, zo)
        # logdet = -sum of L*D alphas, each carrying activation-rounding error of a few 1e-3 with random sign:
        # a bound relative to the root-sum-square scale of the sum, without absolute slack
        assert np.abs(ld - ldo).max() <= 2e-2 * max(np.abs(ldo).max(), np.sqrt(m.L * synth.token_dim(cfg)) * 0.1)


def test_bf16_ragged_sequence_length_and_classes():
    """L = 81 tokens (not a multiple of the 64-row attention tile or the 128-row GEMM tile), D = 48."""
    cfg = synth.config("cfg3", H=36, W=36, n_blocks=2, n_layers=2, width=256, n_heads=4, n_classes=10)
    lab = synth.make_labels(cfg, B=3)
    m, x, xo, its, ito, rc = _bf16_case(cfg, 3, 5, [0, 1], 1e-3, labels=lab)
    assert rc == 0 and bf16_close(x, xo) and np.abs(its - ito).max() <= 1


def test_bf16_ragged_rows_on_k_split_pair_tiles():
    """L = 81 tokens, 20 samples: 1620 rows = six 256-row pair tiles and a ragged seventh (84 rows, its second CTA
    empty), the residual projections cut into K slices whose partial tiles the next LayerNorm adds; as samples
    converge the row count passes through further ragged sizes down to the 128-row tiles.  All-Jacobi, tau 1e-3;
    three samples against the oracle, the forward direction on the same shapes."""
    cfg = synth.config("cfg3", H=36, W=36, n_blocks=2, n_layers=2, width=256, n_heads=4, n_classes=10)
    B = 20
    lab = synth.make_labels(cfg, B=B)
    with Model(cfg, max_batch=B) as m:
        z = synth.make_latents(cfg, 77, B=B)
        x, ib, its, rc = m.inverse(z, lab, [1, 1], 1e-3, m.L + 1)
        assert rc == 0 and np.isfinite(x).all() and np.array_equal(ib, its.max(axis=1))
        pick = [0, 9, B - 1]
        xo, ito = O.model_inverse(m.blocks, z[pick], lab[pick], cfg, [1, 1], 1e-3, m.L + 1)
        assert bf16_close(x[pick], xo) and np.abs(its[:, pick] - ito).max() <= 1
        zf, ld = m.forward(x, lab)
        zo, ldo = O.model_forward(m.blocks, x[pick], lab[pick], cfg)
        assert bf16_close(zf[pick], zo)
        assert np.abs(ld[pick] - ldo).max() <= 2e-2 * max(np.abs(ldo).max(), np.sqrt(m.L * synth.token_dim(cfg)) * 0.1)


def test_bf16_optional_kernel_paths_agree(monkeypatch):
    """The mma.sync attention and the one-CTA-per-tile GEMM give the same sweep as the default kernels."""
    cfg = synth.config("cfg2", n_blocks=1, n_layers=2)
    z = synth.make_latents(cfg, 17, B=3)
    outs = {}
    for name, env in (("default", {}), ("attn_mma", {"TARFLOW_ATTN_TC": "0"}), ("single_cta", {"TARFLOW_PAIR_GEMM": "0"})):
        for k in ("TARFLOW_ATTN_TC", "TARFLOW_PAIR_GEMM"):
            monkeypatch.delenv(k, raising=False)
        for k, v in env.items():
            monkeypatch.setenv(k, v)
        with Model(cfg, max_batch=3) as m:      # the switches are read when the model is loaded
            outs[name], _, _, rc = m.inverse(z, None, [1], -1.0, 3)
            assert rc == 0 and np.isfinite(outs[name]).all()
    xo, _ = O.model_inverse(synth.make_weights(cfg), z, None, cfg, [1], -1.0, 3)
    for name, x in outs.items():
        assert bf16_close(x, xo), name
    assert rel_l2(outs["attn_mma"], outs["default"]) <= 5e-3
    assert rel_l2(outs["single_cta"], outs["default"]) <= 1e-4


def test_bf16_two_term_attention_paths_agree(monkeypatch):
    """tau mode escalates to two-term operands: the tcgen05 two-term attention (default) and the mma.sync one converge
    to the same answer in the same number of sweeps (within one) and both match the oracle."""
    cfg = synth.config("cfg2", n_blocks=2, n_layers=2)
    z = synth.make_latents(cfg, 23, B=5)
    outs = {}
    for name, env in (("tcgen05", {}), ("mma_sync", {"TARFLOW_ATTN_TC_SPLIT": "0"})):
        monkeypatch.delenv("TARFLOW_ATTN_TC_SPLIT", raising=False)
        for k, v in env.items():
            monkeypatch.setenv(k, v)
        with Model(cfg, max_batch=5) as m:      # the switch is read when the model is loaded
            x, _, its, rc = m.inverse(z, None, [1, 1], 1e-3, m.L + 1)
            assert rc == 0 and np.isfinite(x).all()
            outs[name] = (x, its)
    xo, ito = O.model_inverse(synth.make_weights(cfg), z, None, cfg, [1, 1], 1e-3, synth.seq_len(cfg) + 1)
    for name, (x, its) in outs.items():
        assert bf16_close(x, xo), name
        assert np.abs(its - ito).max() <= 1, name
    assert rel_l2(outs["tcgen05"][0], outs["mma_sync"][0]) <= 5e-3


@pytest.mark.gpu
def test_bf16_optional_sequential_paths_agree(monkeypatch):
    """Sequential decoding: fused bias + GELU, the mma.sync step GEMM, the unfused step tail, the five-kernel layer chain and a
    single sample chain give the default path's result."""
    cfg = synth.config("cfg2", n_blocks=1, n_layers=2)
    z = synth.make_latents(cfg, 19, B=40)      # 40 samples: two chains of 20 by default
    outs = {}
    for name, env in (("default", {}), ("gelu_fused", {"TARFLOW_SEQ_FUSE_GELU": "1"}), ("mma_sync", {"TARFLOW_SEQ_MMA": "1"}),
                      ("tail_kernels", {"TARFLOW_SEQ_FUSE_TAIL": "0"}), ("fused_chain", {"TARFLOW_SEQ_FIN": "1"}),
                      ("fused_chain_unfused_tail", {"TARFLOW_SEQ_FIN": "1", "TARFLOW_SEQ_FUSE_TAIL": "0"}),
                      ("one_chain", {"TARFLOW_SEQ_CHAINS": "1"})):
        for k in ("TARFLOW_SEQ_FUSE_GELU", "TARFLOW_SEQ_MMA", "TARFLOW_SEQ_FUSE_TAIL", "TARFLOW_SEQ_FIN", "TARFLOW_SEQ_CHAINS"):
            monkeypatch.delenv(k, raising=False)
        for k, v in env.items():
            monkeypatch.setenv(k, v)
        with Model(cfg, max_batch=40) as m:     # the switches are read when the model is loaded
            outs[name], _, _, rc = m.inverse(z, None, [0], -1.0, 3)
            assert rc == 0 and np.isfinite(outs[name]).all()
    xo, _ = O.model_inverse(synth.make_weights(cfg), z, None, cfg, [0], -1.0, 3)
    for name, x in outs.items():
        assert bf16_close(x, xo), name
    assert rel_l2(outs["gelu_fused"], outs["default"]) <= 5e-3
    assert rel_l2(outs["mma_sync"], outs["default"]) <= 5e-3
    assert rel_l2(outs["tail_kernels"], outs["default"]) <= 5e-3
    assert rel_l2(outs["fused_chain"], outs["default"]) <= 5e-3
    assert rel_l2(outs["fused_chain_unfused_tail"], outs["default"]) <= 5e-3
    assert np.array_equal(outs["one_chain"], outs["default"])     # a sample's arithmetic does not depend on the chain split
