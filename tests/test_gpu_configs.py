"""GPU parity on the shapes of the long-sequence configuration and of the policy / batch / tau sweep.

Every case calls the CUDA library through its C ABI and compares with the fp64 CPU oracle on the same seeded
inputs.  The models keep the architecture of the named configuration (token count, token dimension, width,
heads, classes) at a reduced depth (2 flow blocks x 2 layers) so that the oracle decodes its samples in seconds;
samples are independent under the per-sample stopping test, so a few samples of a large GPU batch are checked
one by one and the rest through properties that hold for every sample.

Tolerances (bf16 engine): relative L2 error on x <= 2e-2 and sweep counts within +-1 of the oracle at the same
tau; beside the norm an element-wise bound max|dx| <= 5e-2 (the norm alone would let a handful of entries be
wrong by O(1)).
"""
import numpy as np
import pytest

from oracle import tarflow_oracle as O
from paper_2505_24791_b200 import binding, synth
from tests.gpu_util import Model, rel_l2

pytestmark = pytest.mark.gpu

BF16_REL_L2 = 2e-2
BF16_MAX_ABS = 5e-2


def _close(x, xo):
    assert np.isfinite(x).all()
    assert rel_l2(x, xo) <= BF16_REL_L2
    assert np.abs(x - xo).max() <= BF16_MAX_ABS


# ---------------------------------------------------------------- long sequences (L = 1024, D = 192)
@pytest.fixture(scope="module")
def long_model():
    cfg = synth.config("cfg4", n_blocks=2, n_layers=2)
    with Model(cfg, max_batch=cfg["B"]) as m:
        yield m


def test_long_sequence_selective_batch16_sampled_against_oracle(long_model):
    """1024 tokens of dimension 192, width 1024, 16 heads, batch 16, selective policy, tau 1e-3: eight query
    tiles per head and sixteen key tiles per query tile in the sweep attention, 1023 decoding steps in block 0."""
    m = long_model
    cfg, B = m.cfg, m.cfg["B"]
    z = synth.make_latents(cfg, 1000, B=B)
    x, ib, its, rc = m.inverse(z, None, [0, 1], cfg["tau"], m.L + 1)
    assert rc == 0 and np.isfinite(x).all()
    assert ib[0] == m.L - 1 and (its[0] == m.L - 1).all()
    assert (its[1] >= 2).all() and (its[1] <= m.L).all() and ib[1] == its[1].max()
    pick = [11]
    xo, ito = O.model_inverse(m.blocks, z[pick], None, cfg, [0, 1], cfg["tau"], m.L + 1)
    _close(x[pick], xo)
    assert np.abs(its[:, pick] - ito).max() <= 1
    # the same sample decoded alone gives the same answer (its schedule depends on that sample only)
    x1, _, it1, rc1 = m.inverse(z[pick], None, [0, 1], cfg["tau"], m.L + 1)
    assert rc1 == 0 and np.abs(x1 - x[pick]).max() <= 2e-3 and abs(int(it1[1, 0]) - int(its[1, pick[0]])) <= 1


def test_long_sequence_all_sequential_matches_oracle(long_model):
    """Both blocks decoded token by token (1023 steps each, the second on the reversed order), batch 16."""
    m = long_model
    cfg = m.cfg
    z = synth.make_latents(cfg, 1001, B=cfg["B"])
    xs = m.inverse_sequential(z, None)
    pick = [3]
    xo = O.model_inverse_sequential(m.blocks, z[pick], None, cfg)
    _close(xs[pick], xo)
    # sequential decoding is the limit of Jacobi decoding: the selective result lies within a few tau of it
    xj, _, _, rc = m.inverse(z, None, [0, 1], cfg["tau"], m.L + 1)
    assert rc == 0 and np.abs(xj - xs).max() <= 2e-2


# ---------------------------------------------------------------- policy / batch / tau sweep shapes
@pytest.fixture(scope="module")
def sweep_model():
    """The class-conditional architecture (256 tokens of dimension 48, width 1024, 16 heads, 1000 classes)."""
    cfg = synth.config("cfg3", n_blocks=2, n_layers=2)
    with Model(cfg, max_batch=256) as m:
        yield m


POLICIES = {"all_sequential": [0, 0], "all_jacobi": [1, 1], "selective": [0, 1]}


@pytest.mark.parametrize("B", [1, 8, 32, 256])
@pytest.mark.parametrize("policy", ["all_sequential", "all_jacobi", "selective"])
def test_sweep_shapes_batches_and_policies(sweep_model, B, policy):
    """Batches 1, 8, 32 (one 32-row step tile) and 256 (65 536 rows per sweep, four 64-row step tiles) under the
    three policies at tau = 1e-3; up to two samples of each batch against the oracle."""
    m = sweep_model
    cfg, pol = m.cfg, POLICIES[policy]
    z = synth.make_latents(cfg, 3000 + B, B=B)
    lab = synth.make_labels(cfg, B=B)
    x, ib, its, rc = m.inverse(z, lab, pol, 1e-3, m.L + 1)
    assert rc == 0 and np.isfinite(x).all()
    for g, p in enumerate(pol):
        if p == 0:
            assert ib[g] == m.L - 1 and (its[g] == m.L - 1).all()
        else:
            assert (its[g] >= 2).all() and (its[g] <= m.L).all() and ib[g] == its[g].max()
    pick = sorted({0, B - 1})
    xo, ito = O.model_inverse(m.blocks, z[pick], lab[pick], cfg, pol, 1e-3, m.L + 1)
    _close(x[pick], xo)
    assert np.abs(its[:, pick] - ito).max() <= 1


@pytest.mark.parametrize("tau", [1e-2, 1e-4])
@pytest.mark.parametrize("policy", ["all_jacobi", "selective"])
def test_sweep_shapes_thresholds(sweep_model, tau, policy):
    """tau = 1e-2 (single bf16 operands are enough, no escalation) and tau = 1e-4 (two-term operands; the
    stopping test has to pass below the rounding floor of single operands), batch 8, two samples checked."""
    m = sweep_model
    cfg, pol, B = m.cfg, POLICIES[policy], 8
    z = synth.make_latents(cfg, 3100, B=B)
    lab = synth.make_labels(cfg, B=B)
    x, ib, its, rc = m.inverse(z, lab, pol, tau, m.L + 1)
    assert rc == 0 and np.isfinite(x).all()
    pick = [2, 5]
    xo, ito = O.model_inverse(m.blocks, z[pick], lab[pick], cfg, pol, tau, m.L + 1)
    _close(x[pick], xo)
    assert np.abs(its[:, pick] - ito).max() <= 1


# ---------------------------------------------------------------- precision modes and the convergence trace
def test_precision_modes_and_trace(sweep_model):
    m = sweep_model
    cfg, B = m.cfg, 6
    z = synth.make_latents(cfg, 3200, B=B)
    lab = synth.make_labels(cfg, B=B)
    xo, ito = O.model_inverse(m.blocks, z, lab, cfg, [1, 1], 1e-3, m.L + 1)
    try:
        # mode 2: two-term operands from the first sweep; same answer, counts within one
        binding.tf_set_precision(m.m, 2)
        binding.tf_trace_enable(m.m, 1)
        x2, ib2, its2, rc2 = m.inverse(z, lab, [1, 1], 1e-3, m.L + 1)
        trace = binding.tf_trace_read(m.m)
        assert rc2 == 0
        _close(x2, xo)
        assert np.abs(its2 - ito).max() <= 1
        # the trace: one record per executed sweep; the active count of sweep t of block g is the number of
        # samples whose own sweep count is >= t (a sample leaves after the sweep that passes its test)
        assert len(trace) == int(ib2.sum())
        for g, t, active, md in trace:
            assert active == int((its2[g] >= t).sum())
            assert md >= 0.0
        for g in range(2):
            mds = [md for gg, t, a, md in trace if gg == g]
            assert mds[-1] <= 1e-3 < mds[0]              # the last sweep of a block passed the test, the first did not
        # the oracle's active counts agree wherever its per-sample counts do
        for g, t, active, _ in trace:
            assert abs(active - int((ito[g] >= t).sum())) <= int((its2[g] != ito[g]).sum())
        binding.tf_trace_enable(m.m, 0)
        # mode 1: single operands only.  At tau = 1e-2 that is what the default does too; at tau = 1e-3 the
        # rounding floor of single operands keeps the test from passing, which is reported as TF_MAXITER
        binding.tf_set_precision(m.m, 1)
        x1, _, its1, rc1 = m.inverse(z, lab, [1, 1], 1e-2, m.L + 1)
        xo1, ito1 = O.model_inverse(m.blocks, z, lab, cfg, [1, 1], 1e-2, m.L + 1)
        assert rc1 == 0
        _close(x1, xo1)
        assert np.abs(its1 - ito1).max() <= 1
        x1b, ib1b, _, rc1b = m.inverse(z, lab, [1, 1], 1e-3, 12)
        assert rc1b in (binding.TF_OK, binding.TF_MAXITER)
        _close(x1b, xo)                                   # the last iterate is still a good sample
    finally:
        binding.tf_set_precision(m.m, 0)
        binding.tf_trace_enable(m.m, 0)
    # mode 0 again (escalation per sample)
    x0, _, its0, rc0 = m.inverse(z, lab, [1, 1], 1e-3, m.L + 1)
    assert rc0 == 0
    _close(x0, xo)
    assert np.abs(its0 - ito).max() <= 1


# ---------------------------------------------------------------- error paths that must not fault
def test_out_of_range_label_is_refused(sweep_model):
    m = sweep_model
    cfg, B = m.cfg, 4
    z = synth.make_latents(cfg, 3300, B=B)
    lab = synth.make_labels(cfg, B=B)
    for bad in (cfg["n_classes"], -1, 2 ** 30):
        lab_bad = lab.copy()
        lab_bad[2] = bad
        with pytest.raises(binding.TarflowError) as e:
            m.inverse(z, lab_bad, [1, 1], 1e-2, 4)
        assert e.value.code == binding.TF_EINVAL and "label" in str(e.value)
        with pytest.raises(binding.TarflowError) as e:
            m.forward(z, lab_bad)
        assert e.value.code == binding.TF_EINVAL
    x, _, _, rc = m.inverse(z, lab, [1, 1], 1e-2, m.L + 1)    # the model is still usable
    assert rc == 0 and np.isfinite(x).all()


def test_bounded_wait_runs_out_is_reported_once_and_model_recovers(sweep_model):
    """A wait that nothing satisfies (1 ms limit) makes the kernel record a code and return; the host reports
    TF_ETIMEOUT once, clears the word, and the next call on the model gives the right answer."""
    m = sweep_model
    cfg, B = m.cfg, 2
    z = synth.make_latents(cfg, 3400, B=B)
    lab = synth.make_labels(cfg, B=B)
    x_before, _, _, rc = m.inverse(z, lab, [1, 1], -1.0, 3)
    assert rc == 0
    with pytest.raises(binding.TarflowError) as e:
        binding.tf_selftest_wait_timeout(m.m, 1000)
    assert e.value.code == binding.TF_ETIMEOUT and "code 9" in str(e.value)
    x_after, _, _, rc = m.inverse(z, lab, [1, 1], -1.0, 3)
    assert rc == 0 and np.array_equal(x_before, x_after)
    zf, ld = m.forward(x_after, lab)
    assert np.isfinite(zf).all() and np.isfinite(ld).all()


# ---------------------------------------------------------------- the long-sequence configuration at its full size
def test_long_sequence_full_size_properties():
    """cfg4 as the benchmark runs it (8 blocks x 8 layers, 1024 tokens, batch 16, selective policy, tau 1e-3).  The
    oracle needs six minutes per sample here, so the checks are properties that hold at any size: the forward
    direction applied to the sample returns the latent (Eq. 4 and Eq. 5 are mutual inverses, through all 64 layers),
    the all-sequential sample agrees with the selective one to a few tau, sweep counts lie in Prop. 3.2's range."""
    cfg = synth.config("cfg4")
    B = cfg["B"]
    policy = [0] + [1] * (cfg["n_blocks"] - 1)
    with Model(cfg, max_batch=B) as m:
        z = synth.make_latents(cfg, 1000, B=B)
        x, ib, its, rc = m.inverse(z, None, policy, cfg["tau"], m.L + 1)
        assert rc == 0 and np.isfinite(x).all()
        assert (its[0] == m.L - 1).all() and (its[1:] >= 2).all() and (its[1:] <= 12).all()
        zr, ld = m.forward(x, None)
        assert np.isfinite(ld).all()
        assert rel_l2(zr, z.astype(np.float64)) <= BF16_REL_L2 and np.abs(zr - z).max() <= 0.15
        xs = m.inverse_sequential(z[:4], None)
        assert rel_l2(x[:4], xs) <= 5e-3 and np.abs(x[:4] - xs).max() <= 5e-2


# ---------------------------------------------------------------- sweeps over few rows (K-split residual projections)
@pytest.mark.parametrize("name", ["cfg2", "cfg3"])
def test_few_row_sweeps_agree_with_the_one_shape_path_and_the_oracle(name, monkeypatch):
    """Sweeps of up to 1024 rows run on 128 x 128 tiles with the residual projections cut into K slices that the next
    LayerNorm adds; up to 4096 rows the pair tiles are cut.  Batches 1 (256 rows, 8 slices at width 1024 / 4 at 512),
    3 (768 rows), 5 (1280 rows: pair tiles, 3 to 6 slices) and 8 (2048 rows) against the oracle, and against
    the same library with both paths switched off (every sweep on one tile shape, reduce-add epilogue).  The forward
    direction takes the same path."""
    cfg = synth.config(name, n_blocks=2, n_layers=2)
    L = synth.seq_len(cfg)
    lab_of = (lambda B: synth.make_labels(cfg, B=B)) if cfg.get("n_classes", 0) else (lambda B: None)
    with Model(cfg, max_batch=8) as m:
        monkeypatch.setenv("TARFLOW_SMALL_M_ROWS", "0")
        monkeypatch.setenv("TARFLOW_SPLIT_M_ROWS", "0")
        with Model(cfg, max_batch=8) as ref:
            for B in (1, 3, 5, 8):
                z = synth.make_latents(cfg, 5200 + B, B=B)
                lab = lab_of(B)
                x, ib, its, rc = m.inverse(z, lab, [1, 1], 1e-3, L + 1)
                xr, ibr, itsr, rcr = ref.inverse(z, lab, [1, 1], 1e-3, L + 1)
                assert rc == 0 and rcr == 0 and np.isfinite(x).all()
                assert np.abs(x - xr).max() <= 2e-3 and np.abs(its - itsr).max() <= 1
                x2, _, its2, _ = m.inverse(z, lab, [1, 1], 1e-3, L + 1)          # fixed summation order: run-to-run identical
                assert np.array_equal(x, x2) and np.array_equal(its, its2)
                pick = [B - 1]
                xo, ito = O.model_inverse(m.blocks, z[pick], None if lab is None else lab[pick], cfg, [1, 1], 1e-3, L + 1)
                _close(x[pick], xo)
                assert np.abs(its[:, pick] - ito).max() <= 1
                zf, ld = m.forward(xo, None if lab is None else lab[pick])
                zo, ldo = O.model_forward(m.blocks, xo, None if lab is None else lab[pick], cfg)
                assert rel_l2(zf, zo) <= 2e-2 and np.abs(ld - ldo).max() <= 2e-2 * max(1.0, np.abs(ldo).max())
