"""The allocation-free GEMM entry point against the library's ordinary GEMM entry point.

tf_skinny_gemm_noalloc exists for callers that cannot let the library call cudaMalloc (all device memory
already owned by their own pool, or a loop that cannot afford the device-wide synchronisation an
allocation implies): its split-K partial tiles live in a static device array that is shared by all
calls and keeps the previous call's contents.  The test therefore runs different problems back to
back through the C ABI and compares each with tf_gemm_bf16 on the same operands and with the fp64 product
of the CPU oracle, so stale scratch from the first call would show up in the second.  It is collected last
on purpose.
"""
import numpy as np
import pytest
import torch

from oracle import tarflow_oracle as O
from paper_2505_24791_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _case(M, N, K, seed, with_bias):
    rng = np.random.default_rng(seed)
    a = synth.round_to_bf16(rng.standard_normal((M, K)).astype(np.float32))
    w = synth.round_to_bf16((rng.standard_normal((N, K)) / np.sqrt(K)).astype(np.float32))
    at = torch.from_numpy(a).cuda().to(torch.bfloat16)
    wt = torch.from_numpy(w).cuda().to(torch.bfloat16)
    bias = rng.standard_normal(N).astype(np.float32) if with_bias else np.zeros(N, dtype=np.float32)
    bt = torch.from_numpy(bias).cuda() if with_bias else None
    want = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    got = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    binding.tf_gemm_bf16(at, wt, bt, want, M, N, K)
    assert binding.tf_gemm_status() == 0
    binding.tf_skinny_gemm_noalloc(at, wt, bt, got, M, N, K)
    torch.cuda.synchronize()
    got, want = got.cpu().numpy().astype(np.float64), want.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    # both accumulate bf16 products in fp32, in different orders: the tolerance of the GEMM parity test
    assert np.abs(got - want).max() < 2e-4 * max(1.0, np.sqrt(K) / 8)
    # and against the plain fp64 product (the operands are exactly representable, so only accumulation differs)
    ref = O.linear(a.astype(np.float64), w.astype(np.float64), bias.astype(np.float64))
    assert np.abs(got - ref).max() < 2e-4 * max(1.0, np.sqrt(K) / 8)


def test_no_alloc_gemm_matches_gemm_entry_point_on_two_calls_in_a_row():
    _case(200, 512, 2048, 1, True)     # 8 K slices, 4 row tiles with a ragged last one
    _case(37, 96, 512, 2, False)       # smaller problem second: leftovers of the first call lie beyond its tiles
    _case(200, 512, 2048, 3, True)     # and the large one again over the second call's leftovers


def test_no_alloc_gemm_rejects_what_does_not_fit():
    t = torch.zeros(8, dtype=torch.bfloat16, device="cuda")
    c = torch.zeros(8, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.TarflowError) as e:   # 16 * 1024 * 1024 * 4 bytes of tiles > 8 MiB
        binding.tf_skinny_gemm_noalloc(t, t, None, c, 1024, 1024, 4096)
    assert e.value.code == binding.TF_EINVAL and "static scratch" in str(e.value)
    with pytest.raises(binding.TarflowError) as e:
        binding.tf_skinny_gemm_noalloc(t, t, None, c, 4, 8, 100)
    assert e.value.code == binding.TF_EINVAL
    # operands that are not 16-byte aligned (a bf16 view starting at an odd element) are refused before any launch
    big = torch.zeros(8 * 256 + 8, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(4 * 8 + 4, dtype=torch.float32, device="cuda")
    for a_, w_ in ((big[1:], big), (big, big[3:])):
        with pytest.raises(binding.TarflowError) as e:
            binding.tf_skinny_gemm_noalloc(a_, w_, None, out, 4, 8, 256)
        assert e.value.code == binding.TF_EINVAL and "aligned" in str(e.value)
    binding.tf_skinny_gemm_noalloc(big, big, None, out, 4, 8, 256)     # aligned: accepted
    torch.cuda.synchronize()
