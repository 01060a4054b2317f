"""GPU parity of the second workload (Jacobi decoding of an MLP-based masked autoregressive flow, App. E.3) against
the fp64 CPU oracle, through the C ABI.  fp32 engine: max|dx| <= 1e-4 in fixed-iteration mode; bf16 engine: relative
L2 <= 2e-2 (and max|dx| <= 5e-2), sweep counts within +-1 of the oracle at the same tau."""
import numpy as np
import pytest
import torch

from oracle import maf_oracle as MO
from paper_2505_24791_b200 import binding, synth

pytestmark = pytest.mark.gpu
FP32_TOL = 1e-4


class Maf:
    def __init__(self, cfg, max_batch, **wkw):
        self.cfg = cfg
        self.blocks = synth.make_maf_weights(cfg, **wkw)
        self.m = binding.tf_maf_load(cfg, synth.pack_maf_blob(cfg, self.blocks), max_batch)
        self.K, self.D = cfg["n_blocks"], cfg["D"]

    def __enter__(self):
        return self

    def __exit__(self, *a):
        try:
            damaged = binding.tf_debug_check_guards(self.m)
        finally:
            binding.tf_free(self.m)
        assert damaged == 0, f"{damaged} guard words around the model's device buffers were overwritten"

    def jacobi(self, z, tau, max_iters, init_mode=0):
        B = z.shape[0]
        zt = torch.from_numpy(np.ascontiguousarray(z, dtype=np.float32)).cuda()
        xt = torch.full_like(zt, float("nan"))
        ib = np.full(self.K, -1, dtype=np.int32)
        its = torch.full((self.K, B), -1, dtype=torch.int32, device="cuda")
        rc = binding.tf_maf_inverse_jacobi(self.m, zt, B, tau, max_iters, init_mode, xt, ib, its)
        return xt.cpu().numpy().astype(np.float64), ib, its.cpu().numpy(), rc

    def sequential(self, z):
        zt = torch.from_numpy(np.ascontiguousarray(z, dtype=np.float32)).cuda()
        xt = torch.full_like(zt, float("nan"))
        binding.tf_maf_inverse_sequential(self.m, zt, z.shape[0], xt)
        return xt.cpu().numpy().astype(np.float64)

    def forward(self, x):
        xt = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()
        zt = torch.full_like(xt, float("nan"))
        ld = torch.full((x.shape[0],), float("nan"), dtype=torch.float32, device="cuda")
        binding.tf_maf_forward(self.m, xt, x.shape[0], zt, ld)
        return zt.cpu().numpy().astype(np.float64), ld.cpu().numpy().astype(np.float64)


def rel_l2(a, b):
    return float(np.sqrt(((a - b) ** 2).sum()) / np.sqrt((b ** 2).sum()))


# ---------------------------------------------------------------- fp32 engine
@pytest.fixture(scope="module")
def tiny():
    with Maf(synth.maf_config("maf_tiny"), 7, out_scale=0.5) as m:
        yield m


def test_fp32_fixed_sweeps_sequential_and_prop_3_2(tiny):
    m = tiny
    z = synth.make_maf_latents(m.cfg, 11, B=5)
    x, ib, its, rc = m.jacobi(z, -1.0, 4)
    xo, ito = MO.model_inverse(m.blocks, z, -1.0, 4)
    assert rc == 0 and list(ib) == [4] * m.K and np.abs(x - xo).max() <= FP32_TOL and np.array_equal(its, ito)
    xs = m.sequential(z)
    xso, _ = MO.model_inverse(m.blocks, z, 0.0, 0, jacobi=False)
    assert np.abs(xs - xso).max() <= FP32_TOL
    xL, _, _, rc = m.jacobi(z, -1.0, m.D)                      # D sweeps = sequential decoding (Prop. 3.2)
    assert rc == 0 and np.abs(xL - xso).max() <= FP32_TOL


def test_fp32_tau_mode_counts_forward_and_logdet(tiny):
    m = tiny
    z = synth.make_maf_latents(m.cfg, 12, B=7)
    x, ib, its, rc = m.jacobi(z, 1e-6, m.D + 1)
    xo, ito = MO.model_inverse(m.blocks, z, 1e-6, m.D + 1)
    assert rc == 0 and np.abs(x - xo).max() <= FP32_TOL and np.abs(its - ito).max() <= 1
    assert np.array_equal(ib, its.max(axis=1))
    zg, ld = m.forward(xo)
    zo, ldo = MO.model_forward(m.blocks, xo)
    assert np.abs(zg - zo).max() <= FP32_TOL and np.abs(zg - z).max() <= 2 * FP32_TOL
    assert np.abs(ld - ldo).max() <= 1e-4 * max(1.0, np.abs(ldo).max())
    x1, _, it1, _ = m.jacobi(z[3:4], 1e-6, m.D + 1)             # a sample's schedule depends on that sample alone
    assert np.abs(x1[0] - x[3]).max() <= 1e-5 and abs(int(it1[0, 0]) - int(its[0, 3])) <= 1
    xi, _, _, rc = m.jacobi(z, 1e-6, m.D + 1, init_mode=1)       # start from the layer input: same fixed point
    assert rc == 0 and np.abs(xi - xo).max() <= FP32_TOL


def test_zero_output_layer_is_identity_and_error_codes(tiny):
    with Maf(synth.maf_config("maf_tiny"), 4, zero_out=True) as m0:
        z = synth.make_maf_latents(m0.cfg, 13, B=4)
        x, ib, its, rc = m0.jacobi(z, 0.0, 9)
        assert rc == 0 and np.array_equal(x, z.astype(np.float64)) and np.all(its == 2)
    m = tiny
    z = synth.make_maf_latents(m.cfg, 14, B=3)
    _, ib, _, rc = m.jacobi(z, 1e-9, 2)
    assert rc == binding.TF_MAXITER and list(ib) == [2] * m.K
    zt = torch.from_numpy(z).cuda()
    xt = torch.empty_like(zt)
    for B, iters, mode in ((0, 3, 0), (8, 3, 0), (3, 0, 0), (3, 3, 2)):
        with pytest.raises(binding.TarflowError) as e:
            binding.tf_maf_inverse_jacobi(m.m, zt, B, 1e-3, iters, mode, xt)
        assert e.value.code == binding.TF_EINVAL
    with pytest.raises(binding.TarflowError) as e:               # a flow of this kind is not a TarFlow model
        binding.tf_inverse_sequential(m.m, zt, None, 3, xt)
    assert e.value.code == binding.TF_EINVAL
    with pytest.raises(binding.TarflowError) as e:
        binding.tf_maf_load(m.cfg, synth.pack_maf_blob(m.cfg, m.blocks)[:-4], 4)
    assert e.value.code == binding.TF_ESIZE


# ---------------------------------------------------------------- bf16 tensor-core engine
def test_bf16_ising_shape_sampled_against_oracle():
    """256 dimensions, hidden width 1024, 8 layers, a batch of 2000 rows (pair tiles with a ragged last one): a few
    samples against the oracle, properties for all; run twice for determinism."""
    cfg = synth.maf_config("maf_ising")
    B = 2000
    with Maf(cfg, B) as m:
        z = synth.make_maf_latents(cfg, 21, B=B)
        x, ib, its, rc = m.jacobi(z, cfg["tau"], m.D + 1)
        assert rc == 0 and np.isfinite(x).all()
        assert (its >= 2).all() and (its <= m.D).all() and np.array_equal(ib, its.max(axis=1))
        pick = [0, 777, B - 1]
        xo, ito = MO.model_inverse(m.blocks, z[pick], cfg["tau"], m.D + 1)
        assert rel_l2(x[pick], xo) <= 2e-2 and np.abs(x[pick] - xo).max() <= 5e-2
        assert np.abs(its[:, pick] - ito).max() <= 1
        x2, _, its2, rc2 = m.jacobi(z, cfg["tau"], m.D + 1)
        assert rc2 == 0 and np.array_equal(x, x2) and np.array_equal(its, its2)
        # the first 900 samples alone (one-CTA sweep control instead of the count / scan / scatter kernels, other row
        # tiles): a sample's result and schedule do not depend on its batch mates
        x3, _, its3, rc3 = m.jacobi(z[:900], cfg["tau"], m.D + 1)
        assert rc3 == 0 and np.array_equal(x3, x[:900]) and np.array_equal(its3, its[:, :900])


def test_bf16_ragged_dimension_sequential_forward_and_thresholds():
    """D = 72 (one full and one partial 64-wide k slab in the first layer, 144 output columns), hidden 192, 3 layers."""
    cfg = synth.maf_config("maf_ising", D=72, hidden=192, n_blocks=3)
    B = 37
    with Maf(cfg, B) as m:
        z = synth.make_maf_latents(cfg, 22, B=B)
        xso, _ = MO.model_inverse(m.blocks, z, 0.0, 0, jacobi=False)
        xs = m.sequential(z)
        assert rel_l2(xs, xso) <= 2e-2 and np.abs(xs - xso).max() <= 5e-2
        for tau in (1e-2, 1e-3, 1e-4):
            x, ib, its, rc = m.jacobi(z, tau, m.D + 1)
            xo, ito = MO.model_inverse(m.blocks, z, tau, m.D + 1)
            assert rc == 0 and rel_l2(x, xo) <= 2e-2 and np.abs(x - xo).max() <= 5e-2
            assert np.abs(its - ito).max() <= 1
        zg, ld = m.forward(xso)
        zo, ldo = MO.model_forward(m.blocks, xso)
        assert rel_l2(zg, zo) <= 2e-2 and np.abs(zg - zo).max() <= 5e-2
        assert np.abs(ld - ldo).max() <= 2e-2 * max(np.abs(ldo).max(), np.sqrt(m.D * m.K) * 0.1)


def test_bf16_mnist_shape_ragged_k_and_head_width():
    """784 dimensions (12.25 k slabs in the first layer: the last one is zero-filled by the tensor map; 1568 head
    columns, not a multiple of the 256-column pair tile), hidden width 1024, 2 layers, 100 samples."""
    cfg = synth.maf_config("maf_mnist", n_blocks=2)
    B = cfg["B"]
    with Maf(cfg, B) as m:
        z = synth.make_maf_latents(cfg, 23, B=B)
        x, ib, its, rc = m.jacobi(z, cfg["tau"], m.D + 1)
        assert rc == 0 and np.isfinite(x).all() and (its >= 2).all()
        pick = [0, 1, 57, B - 1]
        xo, ito = MO.model_inverse(m.blocks, z[pick], cfg["tau"], m.D + 1)
        assert rel_l2(x[pick], xo) <= 2e-2 and np.abs(x[pick] - xo).max() <= 5e-2
        assert np.abs(its[:, pick] - ito).max() <= 1
        xf, _, itf, rc = m.jacobi(z[:3], -1.0, 5)                   # fixed sweeps: the same iterate as the oracle's
        xfo, _ = MO.model_inverse(m.blocks, z[:3], -1.0, 5)
        assert rc == 0 and rel_l2(xf, xfo) <= 2e-2 and np.abs(xf - xfo).max() <= 5e-2
