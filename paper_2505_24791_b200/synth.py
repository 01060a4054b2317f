"""Seeded synthetic inputs for the TarFlow selective-Jacobi hot path.

This module only *draws numbers and packs bytes*: configurations, weight
tensors, latents, labels and the flat weight blob that ``tf_load`` parses.
It contains none of the method's arithmetic (no flow maps, no transformer),
so both the CPU oracle's tests and the CUDA binding may use it without the
two sharing any computation.

Workloads stand in for the paper's CIFAR-10/100 and AFHQ models (Table
"Experimental configuration for each dataset": resolution, patch size,
sequence length, blocks, layers per block, hidden width) with seeded random
weights, because no trained checkpoint or dataset is available.
"""
from __future__ import annotations

import numpy as np

MAGIC = 0x31574654  # "TFW1" little endian
VERSION = 1
HEADER_INTS = 16

# name -> configuration.  dtype: 0 = fp32 engine, 1 = bf16 operands / fp32 accumulate.
CONFIGS = {
    # tiny fp32 model the CPU oracle finishes in seconds
    "cfg1": dict(C=3, H=16, W=16, patch=2, n_blocks=2, n_layers=2, width=128, n_heads=4,
                 mlp_ratio=4, n_classes=0, dtype=0, B=4, tau=1e-5, z_scale=1.0),
    # CIFAR-shaped model (32x32, patch 2, L=256)
    "cfg2": dict(C=3, H=32, W=32, patch=2, n_blocks=4, n_layers=4, width=512, n_heads=8,
                 mlp_ratio=4, n_classes=0, dtype=1, B=64, tau=1e-3, z_scale=0.9),
    # class-conditional 64x64 model
    "cfg3": dict(C=3, H=64, W=64, patch=4, n_blocks=8, n_layers=8, width=1024, n_heads=16,
                 mlp_ratio=4, n_classes=1000, dtype=1, B=64, tau=1e-3, z_scale=1.0),
    # AFHQ-shaped long-sequence model (256x256, patch 8, L=1024)
    "cfg4": dict(C=3, H=256, W=256, patch=8, n_blocks=8, n_layers=8, width=1024, n_heads=16,
                 mlp_ratio=4, n_classes=0, dtype=1, B=16, tau=1e-3, z_scale=1.0),
}

WEIGHT_SEED = 1234
LABEL_SEED = 7


def config(name: str, **overrides) -> dict:
    cfg = dict(CONFIGS[name])
    cfg.update(overrides)
    return cfg


def micro_config(**kw) -> dict:
    """A very small model for brute-force checks (sizes chosen by the caller)."""
    cfg = dict(C=1, H=2, W=4, patch=1, n_blocks=2, n_layers=1, width=8, n_heads=2, mlp_ratio=2,
               n_classes=0, dtype=0, B=2, tau=1e-6, z_scale=1.0)
    cfg.update(kw)
    return cfg


def seq_len(cfg) -> int:
    return (cfg["H"] // cfg["patch"]) * (cfg["W"] // cfg["patch"])


def token_dim(cfg) -> int:
    return cfg["C"] * cfg["patch"] * cfg["patch"]


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16-representable value (ties to even), kept as fp32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32).astype(np.uint64)
    bias = ((bits >> 16) & 1) + 0x7FFF
    out = (((bits + bias) >> 16) << 16).astype(np.uint32)
    return out.view(np.float32).reshape(a.shape)


def block_tensor_specs(cfg):
    """(name, shape) of every tensor of one flow block, in blob order.

    Linear layers are stored [out_features, in_features]; y = x @ W.T + b.
    """
    d, D, L = cfg["width"], token_dim(cfg), seq_len(cfg)
    hid = cfg["mlp_ratio"] * d
    specs = [("w_in", (d, D)), ("b_in", (d,)), ("pos", (L, d))]
    if cfg["n_classes"] > 0:
        specs.append(("cls", (cfg["n_classes"], d)))
    for i in range(cfg["n_layers"]):
        p = f"l{i}."
        specs += [(p + "ln1_g", (d,)), (p + "ln1_b", (d,)),
                  (p + "w_qkv", (3 * d, d)), (p + "b_qkv", (3 * d,)),
                  (p + "w_o", (d, d)), (p + "b_o", (d,)),
                  (p + "ln2_g", (d,)), (p + "ln2_b", (d,)),
                  (p + "w_1", (hid, d)), (p + "b_1", (hid,)),
                  (p + "w_2", (d, hid)), (p + "b_2", (d,))]
    specs += [("lnf_g", (d,)), ("lnf_b", (d,)), ("w_out", (2 * D, d)), ("b_out", (2 * D,))]
    return specs


def _rng(seed, *key):
    return np.random.Generator(np.random.Philox(key=[(seed << 20) ^ _mix(key), 0x5EED]))


def _mix(key):
    h = 1469598103934665603
    for k in key:
        h = ((h ^ (int(k) & 0xFFFFFFFF)) * 1099511628211) & 0xFFFFFFFFFFFFFFFF
    return h >> 4


def make_weights(cfg, seed: int = WEIGHT_SEED, head_scale: float = 0.1, zero_head: bool = False):
    """Seeded weights: a list (one dict per block, generation order) of fp32 arrays.

    Matrices: Xavier-normal std = sqrt(2/(fan_in+fan_out)).  Head matrix w_out: std =
    head_scale/sqrt(width) so mu~ and alpha~ have standard deviation about head_scale.
    pos / cls embeddings: std 0.02.  Biases: std 0.02, LayerNorm gain 1 + 0.02 n, shift 0.02 n
    (small but non-zero so that every term is exercised by the parity tests).
    For dtype == 1 every matrix operand is rounded to a bf16-representable value, so the fp32
    blob, the bf16 copy the engine makes of it and the fp64 copy the oracle makes are equal.
    """
    d = cfg["width"]
    blocks = []
    for g in range(cfg["n_blocks"]):
        blk = {}
        for ti, (name, shape) in enumerate(block_tensor_specs(cfg)):
            r = _rng(seed, g, ti)
            n = r.standard_normal(shape, dtype=np.float32)
            base = name.split(".")[-1]
            if base in ("w_in", "w_qkv", "w_o", "w_1", "w_2"):
                t = n * np.float32(np.sqrt(2.0 / (shape[0] + shape[1])))
            elif base == "w_out":
                t = n * np.float32(0.0 if zero_head else head_scale / np.sqrt(d))
            elif base in ("pos", "cls"):
                t = n * np.float32(0.02)
            elif base in ("ln1_g", "ln2_g", "lnf_g"):
                t = np.float32(1.0) + n * np.float32(0.02)
            elif base == "b_out":
                t = n * np.float32(0.0 if zero_head else 0.02)
            else:  # biases, LayerNorm shifts
                t = n * np.float32(0.02)
            if cfg["dtype"] == 1 and base.startswith("w_"):
                t = round_to_bf16(t)
            blk[name] = np.ascontiguousarray(t, dtype=np.float32)
        blocks.append(blk)
    return blocks


def pack_blob(cfg, blocks, seed: int = WEIGHT_SEED) -> np.ndarray:
    """Flat little-endian blob: 16 int32 header, then every tensor (fp32) in blob order."""
    hdr = np.zeros(HEADER_INTS, dtype=np.int32)
    hdr[:14] = [MAGIC, VERSION, cfg["C"], cfg["H"], cfg["W"], cfg["patch"], cfg["n_blocks"],
                cfg["n_layers"], cfg["width"], cfg["n_heads"], cfg["mlp_ratio"], cfg["n_classes"],
                cfg["dtype"], seed]
    parts = [hdr.view(np.uint8)]
    for blk in blocks:
        for name, shape in block_tensor_specs(cfg):
            a = blk[name]
            assert a.shape == tuple(shape) and a.dtype == np.float32, name
            parts.append(a.reshape(-1).view(np.uint8))
    return np.concatenate(parts)


def blob_nbytes(cfg) -> int:
    n = sum(int(np.prod(s)) for _, s in block_tensor_specs(cfg))
    return HEADER_INTS * 4 + 4 * n * cfg["n_blocks"]


def make_latents(cfg, seed: int, B: int | None = None) -> np.ndarray:
    """z ~ N(0,1) * z_scale, image shaped [B,C,H,W], fp32.  Row b depends only on (seed, b)."""
    B = cfg["B"] if B is None else B
    z = np.empty((B, cfg["C"], cfg["H"], cfg["W"]), dtype=np.float32)
    for b in range(B):
        z[b] = _rng(seed, 0xA11CE, b).standard_normal(z.shape[1:], dtype=np.float32)
    return z * np.float32(cfg["z_scale"])


def make_labels(cfg, B: int | None = None, seed: int = LABEL_SEED):
    """Uniform class labels [B] int32, or None for an unconditional model."""
    if cfg["n_classes"] <= 0:
        return None
    B = cfg["B"] if B is None else B
    out = np.empty(B, dtype=np.int32)
    for b in range(B):
        out[b] = _rng(seed, 0x1ABE1, b).integers(0, cfg["n_classes"])
    return out


def shard_batch(B: int, rank: int, world: int):
    """Contiguous [start, stop) slice of a batch of B samples owned by `rank` of `world`.

    Samples are independent under the per-sample stopping test, so a multi-GPU run is a plain
    batch split with replicated weights and no exchange on the data path.
    """
    base, rem = divmod(B, world)
    start = rank * base + min(rank, rem)
    return start, start + base + (1 if rank < rem else 0)


# ------------------------------------------------------------------------------------------------
# second workload: masked autoregressive flow (MLP-based, Jacobi decoding on every layer)
# ------------------------------------------------------------------------------------------------
MAF_MAGIC = 0x3146414D  # "MAF1" little endian

# The paper's two MAF experiments are an 8-layer flow on a 2-D Ising lattice (100 000 samples) and an 8-layer flow
# on binary MNIST (100 images); lattice size and hidden width are not stated, so these stand-ins fix them.
MAF_CONFIGS = {
    "maf_tiny": dict(D=12, hidden=32, n_blocks=3, dtype=0, B=5, tau=1e-6, z_scale=1.0),
    "maf_ising": dict(D=256, hidden=1024, n_blocks=8, dtype=1, B=100000, tau=1e-3, z_scale=1.0),
    "maf_mnist": dict(D=784, hidden=1024, n_blocks=8, dtype=1, B=100, tau=1e-3, z_scale=1.0),
}


def maf_config(name: str, **overrides) -> dict:
    cfg = dict(MAF_CONFIGS[name])
    cfg.update(overrides)
    return cfg


def maf_tensor_specs(cfg):
    D, H = cfg["D"], cfg["hidden"]
    return [("w1", (H, D)), ("b1", (H,)), ("w2", (H, H)), ("b2", (H,)), ("w3", (2 * D, H)), ("b3", (2 * D,))]


def make_maf_weights(cfg, seed: int = WEIGHT_SEED, out_scale: float = 0.1, zero_out: bool = False):
    """Seeded dense weights of every layer (no masks applied: masking is the method's, done by each side itself).

    Hidden matrices: normal with std sqrt(2 / fan_in) scaled by sqrt(2) (about half of a row is masked away);
    output matrix std = out_scale / sqrt(hidden / 2) so that mu and alpha have standard deviation of the order of
    out_scale; biases std 0.02.  For dtype == 1 the matrices are rounded to bf16-representable values.
    """
    blocks = []
    for g in range(cfg["n_blocks"]):
        blk = {}
        for ti, (name, shape) in enumerate(maf_tensor_specs(cfg)):
            n = _rng(seed, 0x3AF, g, ti).standard_normal(shape, dtype=np.float32)
            if name in ("w1", "w2"):
                t = n * np.float32(2.0 / np.sqrt(shape[1]))
            elif name == "w3":
                t = n * np.float32(0.0 if zero_out else out_scale / np.sqrt(shape[1] / 2.0))
            elif name == "b3":
                t = n * np.float32(0.0 if zero_out else 0.02)
            else:
                t = n * np.float32(0.02)
            if cfg["dtype"] == 1 and name.startswith("w"):
                t = round_to_bf16(t)
            blk[name] = np.ascontiguousarray(t, dtype=np.float32)
        blocks.append(blk)
    return blocks


def pack_maf_blob(cfg, blocks, seed: int = WEIGHT_SEED) -> np.ndarray:
    """16 int32 header {magic, version, D, hidden, n_blocks, dtype, seed, 0...} then the fp32 tensors of every layer."""
    hdr = np.zeros(HEADER_INTS, dtype=np.int32)
    hdr[:7] = [MAF_MAGIC, VERSION, cfg["D"], cfg["hidden"], cfg["n_blocks"], cfg["dtype"], seed]
    parts = [hdr.view(np.uint8)]
    for blk in blocks:
        for name, shape in maf_tensor_specs(cfg):
            a = blk[name]
            assert a.shape == tuple(shape) and a.dtype == np.float32, name
            parts.append(a.reshape(-1).view(np.uint8))
    return np.concatenate(parts)


def make_maf_latents(cfg, seed: int, B: int | None = None) -> np.ndarray:
    """z ~ N(0,1) * z_scale, [B, D] fp32; row b depends only on (seed, b)."""
    B = cfg["B"] if B is None else B
    z = np.empty((B, cfg["D"]), dtype=np.float32)
    blk = 4096
    for b0 in range(0, B, blk):   # a generator per group of rows keeps large batches quick to draw
        n = min(blk, B - b0)
        z[b0:b0 + n] = _rng(seed, 0x3A11CE, b0).standard_normal((n, cfg["D"]), dtype=np.float32)
    return z * np.float32(cfg["z_scale"])
