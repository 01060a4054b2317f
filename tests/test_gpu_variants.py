"""GPU parity of the variants around Algorithm 1 (tf_inverse_jacobi_ex) against the CPU oracle: caller-supplied
initial iterate, per-block thresholds, the sequential fall-back for stragglers, per-block states and the
distance-to-reference trace.  fp32 engine: max|dx| <= 1e-4; bf16 engine: relative L2 <= 2e-2, counts within +-1."""
import numpy as np
import pytest
import torch

from oracle import tarflow_oracle as O
from paper_2505_24791_b200 import binding, synth
from tests.gpu_util import Model, rel_l2

pytestmark = pytest.mark.gpu
FP32_TOL = 1e-4


def _ex(m, z, labels, policy, tau, max_iters, **kw):
    B, K = z.shape[0], m.K
    zt = torch.from_numpy(np.ascontiguousarray(z, dtype=np.float32)).cuda()
    xt = torch.full_like(zt, float("nan"))
    ib = np.full(K, -1, dtype=np.int32)
    its = torch.full((K, B), -1, dtype=torch.int32, device="cuda")
    for key in ("u0", "ref_states"):
        if kw.get(key) is not None:
            kw[key] = torch.from_numpy(np.ascontiguousarray(kw[key], dtype=np.float32)).cuda()
    states = None
    if kw.pop("want_states", False):
        states = torch.full((K,) + tuple(zt.shape), float("nan"), dtype=torch.float32, device="cuda")
        kw["states"] = states
    lab = None if labels is None else torch.from_numpy(np.asarray(labels, dtype=np.int32)).cuda()
    rc = binding.tf_inverse_jacobi_ex(m.m, zt, lab, B, policy, tau, max_iters, xt, ib, its, **kw)
    st = None if states is None else states.cpu().numpy().astype(np.float64)
    return xt.cpu().numpy().astype(np.float64), ib, its.cpu().numpy(), rc, st


@pytest.fixture(scope="module")
def small_fp32():
    with Model(synth.config("cfg1", n_blocks=3), max_batch=5) as m:
        yield m


def test_caller_supplied_start_and_prop_3_2(small_fp32):
    """u^0 = N(0, I) draws passed in by the caller: L sweeps still give sequential decoding (Prop. 3.2 does not use
    u^0), a few sweeps match the oracle started from the same draws, and tau mode converges to the same answer."""
    m = small_fp32
    cfg, B = m.cfg, 4
    z = synth.make_latents(cfg, 501, B=B)
    u0 = np.stack([synth.make_latents(cfg, 600 + g, B=B) for g in range(m.K)])
    x, ib, _, rc, _ = _ex(m, z, None, [1, 1, 1], -1.0, 5, init_mode=2, u0=u0)
    xo, _ = O.model_inverse(m.blocks, z, None, cfg, [1, 1, 1], -1.0, 5, init_mode=2, u0=u0)
    assert rc == 0 and list(ib) == [5, 5, 5] and np.abs(x - xo).max() <= FP32_TOL
    x0, _, _, _, _ = _ex(m, z, None, [1, 1, 1], -1.0, 5)                  # zeros start: a different 5-sweep iterate
    assert np.abs(x0 - x).max() > 1e-3
    xs = O.model_inverse_sequential(m.blocks, z, None, cfg)
    xL, _, _, rc, _ = _ex(m, z, None, [1, 1, 1], -1.0, m.L, init_mode=2, u0=u0)
    assert rc == 0 and np.abs(xL - xs).max() <= FP32_TOL
    xt_, ib, its, rc, _ = _ex(m, z, None, [0, 1, 1], 1e-5, m.L + 1, init_mode=2, u0=u0)
    xto, ito = O.model_inverse(m.blocks, z, None, cfg, [0, 1, 1], 1e-5, m.L + 1, init_mode=2, u0=u0)
    assert rc == 0 and np.abs(xt_ - xto).max() <= FP32_TOL and np.abs(its - ito).max() <= 1


def test_per_block_tau_and_states(small_fp32):
    m = small_fp32
    cfg, B = m.cfg, 3
    z = synth.make_latents(cfg, 502, B=B)
    taus = [1e-2, 1e-5, 1e-3]
    x, ib, its, rc, st = _ex(m, z, None, [1, 1, 1], 123.0, m.L + 1, tau_block=taus, want_states=True)
    xo, ito, ex = O.model_inverse(m.blocks, z, None, cfg, [1, 1, 1], taus, m.L + 1, return_states=True)
    assert rc == 0 and np.abs(its - ito).max() <= 1
    assert np.abs(st - ex["states"]).max() <= 2e-2            # block 0 stops at tau 1e-2: adjacent iterates differ by < tau
    assert np.array_equal(st[-1], x)
    assert its[1].min() > its[0].max()
    exact = np.array_equal(its, ito)
    if exact:
        assert np.abs(x - xo).max() <= 5e-3                   # same schedule: differences are rounding amplified by later blocks


def test_distance_trace_against_oracle(small_fp32):
    """||u^t - u_seq||_2 per sweep and sample (the paper's convergence figure): fixed L sweeps on a one-block view of
    the model, compared with the oracle's trace; it must reach zero at sweep L (Prop. 3.2)."""
    m = small_fp32
    cfg, B = m.cfg, 3
    z = synth.make_latents(cfg, 503, B=B)
    _, _, _, _, ref = _ex(m, z, None, [0, 0, 0], 0.0, 1, want_states=True)
    _, _, exo = O.model_inverse(m.blocks, z, None, cfg, [0, 0, 0], 0.0, 1, return_states=True)
    assert np.abs(ref - exo["states"]).max() <= FP32_TOL
    binding.tf_trace_enable(m.m, 1)
    try:
        x, ib, _, rc, _ = _ex(m, z, None, [1, 1, 1], -1.0, m.L, ref_states=ref)
        _, _, ext = O.model_inverse(m.blocks, z, None, cfg, [1, 1, 1], -1.0, m.L, ref_states=exo["states"])
        for g in range(m.K):
            tr = binding.tf_trace_read_l2(m.m, g, B).astype(np.float64)
            want = ext["l2"][g]
            assert tr.shape == want.shape == (m.L, B)
            assert np.abs(tr - want).max() <= 1e-3 * max(1.0, want.max())
            assert tr[-1].max() <= 1e-3 and tr[0].min() > 0.1
            assert (np.diff(tr[:, 0])[-10:] <= 1e-4).all()    # no growth at the end
    finally:
        binding.tf_trace_enable(m.m, 0)


def test_fallback_fp32_stragglers_equal_sequential_decoding(small_fp32):
    m = small_fp32
    cfg, B = m.cfg, 5
    z = synth.make_latents(cfg, 504, B=B)
    z[1] *= 0.05                                              # a small-scale sample: it needs about four sweeps more
    xp, _, itp, rc, _ = _ex(m, z, None, [1, 1, 1], 1e-5, m.L + 1)
    assert rc == 0
    cut = int(itp[0].min()) + 1
    assert cut + 1 < itp[0].max()
    x, ib, its, rc, _ = _ex(m, z, None, [1, 0, 0], 1e-5, m.L + 1, fallback_sweeps=cut)
    xo, ito = O.model_inverse(m.blocks, z, None, cfg, [1, 0, 0], 1e-5, m.L + 1, fallback_sweeps=cut)
    assert rc == 0 and np.abs(x - xo).max() <= FP32_TOL
    late = ito[0] == cut + m.L - 1
    assert late.any() and (~late).any()
    mismatch = (its[0] == cut + m.L - 1) != late
    assert (np.abs(itp[0][mismatch] - cut) <= 1).all()        # only a sample that converges right at the cut may differ
    assert ib[0] == its[0].max()
    # the stragglers carry the sequential answer of block 0: all-sequential decoding gives the same x for them
    xs = O.model_inverse_sequential(m.blocks, z, None, cfg)
    both = late & (its[0] == cut + m.L - 1)
    assert np.abs(x[both] - xs[both]).max() <= FP32_TOL


def test_fallback_bf16_engine_with_classes():
    """The tensor-core engine: stragglers of a class-conditional Jacobi block are decoded by the KV-cached step
    kernels on a gathered sub-batch and scattered back."""
    cfg = synth.config("cfg3", n_blocks=2, n_layers=2)
    B = 6
    with Model(cfg, max_batch=B) as m:
        z = synth.make_latents(cfg, 505, B=B)
        lab = synth.make_labels(cfg, B=B)
        xp, _, itp, rc, _ = _ex(m, z, lab, [1, 1], 1e-3, m.L + 1)
        assert rc == 0
        cut = int(itp[1].max()) - 1                           # one sweep short for the slowest samples of block 1
        x, ib, its, rc, _ = _ex(m, z, lab, [1, 1], 1e-3, m.L + 1, fallback_sweeps=cut)
        xo, ito = O.model_inverse(m.blocks, z, lab, cfg, [1, 1], 1e-3, m.L + 1, fallback_sweeps=cut)
        assert rc == 0 and np.isfinite(x).all()
        assert rel_l2(x, xo) <= 2e-2 and np.abs(x - xo).max() <= 5e-2
        fell = its >= m.L - 1
        assert fell.any()
        assert ((its[fell] == cut + m.L - 1)).all() and (its[~fell] <= cut).all()
        agree = (its >= m.L - 1) == (ito >= m.L - 1)
        assert agree.mean() >= 0.5                            # a sample right at the threshold may land on either side
        assert np.abs(its[agree & ~fell] - ito[agree & ~fell]).max(initial=0) <= 1
        # a second call with the same cut replays the cached graph of the gathered sub-batch
        x2, _, its2, rc2, _ = _ex(m, z, lab, [1, 1], 1e-3, m.L + 1, fallback_sweeps=cut)
        assert rc2 == 0 and np.array_equal(x, x2) and np.array_equal(its, its2)


def test_ex_argument_checks(small_fp32):
    m = small_fp32
    z = synth.make_latents(m.cfg, 506, B=2)
    for kw in (dict(init_mode=2), dict(init_mode=3), dict(fallback_sweeps=-1), dict(tau_block=[1e-3, float("nan"), 1e-3])):
        with pytest.raises(binding.TarflowError) as e:
            _ex(m, z, None, [1, 1, 1], 1e-3, 5, **kw)
        assert e.value.code == binding.TF_EINVAL
    t = binding.tf_block_times(m.m, m.K)
    x, _, _, rc, _ = _ex(m, z, None, [0, 1, 1], 1e-3, m.L + 1)
    t = binding.tf_block_times(m.m, m.K)
    assert rc == 0 and t.shape == (m.K,) and (t > 0).all()
