"""Helpers shared by the GPU parity tests (the CUDA path is reached only through the C-ABI binding)."""
import numpy as np
import torch

from paper_2505_24791_b200 import binding, synth


class Model:
    def __init__(self, cfg, max_batch=None, seed=synth.WEIGHT_SEED, **wkw):
        self.cfg = cfg
        self.blocks = synth.make_weights(cfg, seed=seed, **wkw)
        self.blob = synth.pack_blob(cfg, self.blocks, seed=seed)
        self.max_batch = max_batch or cfg["B"]
        self.m = binding.tf_load(cfg, self.blob, self.max_batch)
        self.L = synth.seq_len(cfg)
        self.K = cfg["n_blocks"]

    def close(self):
        if self.m is not None:
            try:    # no kernel of any call on this model wrote outside its buffer
                damaged = binding.tf_debug_check_guards(self.m)
            finally:
                binding.tf_free(self.m)
                self.m = None
            assert damaged == 0, f"{damaged} guard words around the model's device buffers were overwritten"

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    def _lab(self, labels):
        return None if labels is None else torch.from_numpy(np.asarray(labels, dtype=np.int32)).cuda()

    def inverse(self, z, labels, policy, tau, max_iters, init_mode=0):
        B = z.shape[0]
        zt = torch.from_numpy(np.ascontiguousarray(z, dtype=np.float32)).cuda()
        xt = torch.full_like(zt, float("nan"))
        ib = np.full(self.K, -1, dtype=np.int32)
        its = torch.full((self.K, B), -1, dtype=torch.int32, device="cuda")
        rc = binding.tf_inverse_jacobi(self.m, zt, self._lab(labels), B, policy, tau, max_iters, init_mode, xt, ib, its)
        return xt.cpu().numpy().astype(np.float64), ib, its.cpu().numpy(), rc

    def inverse_sequential(self, z, labels):
        B = z.shape[0]
        zt = torch.from_numpy(np.ascontiguousarray(z, dtype=np.float32)).cuda()
        xt = torch.full_like(zt, float("nan"))
        binding.tf_inverse_sequential(self.m, zt, self._lab(labels), B, xt)
        torch.cuda.synchronize()
        return xt.cpu().numpy().astype(np.float64)

    def forward(self, x, labels):
        B = x.shape[0]
        xt = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()
        zt = torch.full_like(xt, float("nan"))
        ld = torch.full((B,), float("nan"), dtype=torch.float32, device="cuda")
        binding.tf_forward(self.m, xt, self._lab(labels), B, zt, ld)
        torch.cuda.synchronize()
        return zt.cpu().numpy().astype(np.float64), ld.cpu().numpy().astype(np.float64)


def rel_l2(a, b):
    return float(np.sqrt(((a - b) ** 2).sum()) / np.sqrt((b ** 2).sum()))
