#!/usr/bin/env python
"""Benchmark of selective-Jacobi TarFlow sampling on B200 (one process per GPU).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3] [--impl ours|reference]
    python bench.py --sweep cfg5            policy x batch x tau table on the class-conditional architecture

A "step" is one whole sampling call (patchify, block 0 decoded sequentially with the KV cache, the
other blocks by Jacobi sweeps with the per-sample stopping test, unpatchify) over one batch of seeded
synthetic latents.  The line printed by rank 0 carries:
  value     samples/s with the latents already resident in device memory (CUDA events, max over ranks),
  e2e       the same through the host-buffer entry point (pinned host z in, x out, copies timed),
  roofline  the kernel class with the largest share of the step; roofline_tensor the tensor-bound class with the
            largest share; roofline_seq_block the sequentially decoded block as a whole (bytes it must stream / its
            time).  Class times come from CUDA events the library records on the launching stream in a second pass
            over the same steps, in which the sequential block runs exactly as in the timed pass,
  blocks    device time per block (events recorded in the timed pass itself), sweeps and active samples per sweep,
  gpu_sequential / gpu_all_jacobi   the same batch decoded with the other policies,
  other_workloads   short legs on the other bf16 configurations (selective / sequential / all-Jacobi),
  second_workload_maf   Jacobi against sequential decoding of an MLP-based autoregressive flow (paper App. E.3),
  cpu_baseline   the fp64 CPU oracle timed on this machine's host cores on a bounded sub-batch.
`--impl reference` times only the CPU oracle (there is no other implementation of the paper).
With N > 1 every rank decodes its own batch (weak scaling, no data-path collective); `--gpus N` without a
torchrun environment starts the N ranks itself.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "TarFlow sampling imgs/s (selective Jacobi vs KV-cached sequential), % TC peak"
UNIT = "samples/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
L2_BYTES = 126e6

# dram bytes per launch (read + write) of a kernel class from the committed ncu capture of that class
# (profiles/gemm_tc2_kernel_cfg3_sweep.md: one single-term launch over the full batch of 16 384 rows; the live class
# also holds two-term launches and launches over fewer rows); None = no capture of the current kernel.
# {workload: {class: bytes}}
NCU_TRAFFIC: dict = {"cfg3": {"gemm_qkv": 89.9e6, "gemm_out": 111.9e6, "gemm_mlp_up": 124.5e6, "gemm_mlp_down": 253.9e6}}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------------------------------------
# algorithmic work per kernel class (what the method itself must compute or move)
# ------------------------------------------------------------------------------------------------
def seq_block_bytes(cfg, L, D, B):
    """Bytes one sequentially decoded block has to stream from device memory (Eq. 5 with a KV cache).

    Weights: every step multiplies by every matrix of the block, n_layers * 12 d^2 + 2 D d values of 2 bytes; they
    are counted once per step when a block's weights exceed the L2 cache and once per block when they stay
    resident.  Cache: step t reads t + 1 rows of K and of V per layer and sample, 2 d L (L - 1) bytes per layer and
    sample over the block, and appends 4 d bytes per step.
    """
    d, hid, nl = cfg["width"], cfg["width"] * cfg["mlp_ratio"], cfg["n_layers"]
    esz = 2 if cfg["dtype"] == 1 else 4
    w_blk = (nl * (4 * d * d + 2 * hid * d) + 2 * D * d) * esz
    w_total = w_blk * (L - 1) if w_blk > L2_BYTES / 2 else w_blk
    kv = nl * B * (esz * d * L * (L - 1) + 2 * esz * d * (L - 1))
    return float(w_total + kv), float(w_blk)


def sweep_flops_per_row(cfg, L, D):
    """FLOPs of one Jacobi sweep per token row: projections 24 d^2 per layer, causal attention 2 d L per layer,
    embedding 2 D d, head 4 D d."""
    d, nl = cfg["width"], cfg["n_layers"]
    return nl * (24.0 * d * d + 2.0 * d * L) + 2.0 * D * d + 4.0 * D * d


def class_work(cfg, L, D, B):
    """-> {class: (bound, per_row, per_launch)}: FLOPs (bound 'tensor') or bytes (bound 'hbm').

    per_row multiplies the activation rows a launch processed, per_launch is added once per launch.
    GEMM [rows, K] x [N, K]^T: 2*N*K FLOPs per row.  Causal attention: QK^T and PV are d*L^2 FLOPs
    each per sample and layer, i.e. 2*d*L per row.  Bandwidth-bound classes: the bytes of every
    operand read once and every result written once (esz = operand size, residual stream fp32).
    """
    d, hid, nl = cfg["width"], cfg["width"] * cfg["mlp_ratio"], cfg["n_layers"]
    esz = 2 if cfg["dtype"] == 1 else 4
    bound = "tensor" if cfg["dtype"] == 1 else "alu"
    w_layer = 3 * d * d + d * d + 2 * hid * d
    head_gemm = not (cfg["dtype"] == 1 and 2 * D * d * esz <= 64 * 1024)
    seq_launches = nl * 4 + (1 if head_gemm else 0)
    seq_w_bytes = (nl * w_layer + (2 * D * d if head_gemm else 0)) * esz / seq_launches
    blk_bytes, _ = seq_block_bytes(cfg, L, D, B)
    return {
        "gemm_qkv": (bound, 2.0 * 3 * d * d, 0.0),
        "gemm_out": (bound, 2.0 * d * d, 0.0),
        "gemm_mlp_up": (bound, 2.0 * hid * d, 0.0),
        "gemm_mlp_down": (bound, 2.0 * hid * d, 0.0),
        "gemm_head_update": (bound, 2.0 * 2 * D * d, 0.0),
        "gemm_head": (bound, 2.0 * 2 * D * d, 0.0),
        "attention": (bound, 2.0 * d * L, 0.0),
        "layernorm": ("hbm", d * (4.0 + esz), 0.0),
        "embed": ("hbm", D * 4.0 + d * (4.0 + esz), 0.0),
        "forward_affine": ("hbm", D * (2 * 4.0 + 2 * 4.0), 0.0),
        "layout": ("hbm", 0.0, 0.0),
        "sweep_control": ("hbm", 0.0, 0.0),
        "seq_gemm": ("hbm", 0.0, seq_w_bytes),
        "seq_attention": ("hbm", (L / 2.0) * 2 * d * esz, 0.0),
        "seq_layernorm": ("hbm", d * (4.0 + esz), 0.0),
        "seq_embed": ("hbm", D * 4.0 + d * 4.0, 0.0),
        "seq_update": ("hbm", D * 4.0 * 4, 0.0),
        "seq_block": ("hbm", 0.0, blk_bytes),
    }


def roofline_report(prof, cfg, L, D, B, pk, pk_kind, workload, step_ms, prof_step_ms):
    """Per-class table and the three roofline objects of the JSON line."""
    work = class_work(cfg, L, D, B)
    total_ms = sum(v[0] for v in prof.values()) or 1.0
    rows = []
    for name, (ms, n, nrows) in prof.items():
        if n == 0:
            continue
        bound, per_row, per_launch = work.get(name, ("hbm", 0.0, 0.0))
        amount = per_row * nrows + per_launch * n
        avg_s = ms * 1e-3 / n
        if bound == "hbm":
            achieved, peak, unit = amount / n / avg_s / 1e9, pk["hbm_gbs"], "GB/s"
        else:
            achieved, peak, unit = amount / n / avg_s / 1e12, pk["bf16_tflops_sustained"], "TFLOP/s"
        rows.append({"kernel": name, "launches": int(n), "total_ms": round(ms, 4), "share": round(ms / total_ms, 4),
                     "avg_us": round(avg_s * 1e6, 3), "bound": bound, "achieved": round(achieved, 2), "peak": peak,
                     "unit": unit, "frac": round(achieved / peak, 4)})
    rows.sort(key=lambda r: -r["total_ms"])

    def obj(r):
        return {"kernel": r["kernel"], "bound": r["bound"], "achieved": r["achieved"], "peak": r["peak"], "unit": r["unit"],
                "frac": r["frac"], "traffic": NCU_TRAFFIC.get(workload, {}).get(r["kernel"]),
                "peak_source": f"of {pk_kind}" + (" (sustained bf16)" if r["bound"] == "tensor" else ""),
                "share_of_device_time": r["share"], "avg_launch_us": r["avg_us"], "launches_per_step": None}

    # the class with the largest share that has algorithmic work attached (control kernels have none)
    top = next((r for r in rows if r["achieved"] > 0), rows[0])
    tens = next((r for r in rows if r["bound"] in ("tensor", "alu") and r["achieved"] > 0), None)
    seqb = next((r for r in rows if r["kernel"] == "seq_block"), None)
    roof = obj(top)
    roof["profiled_ms_per_step"] = round(prof_step_ms, 3)
    roof["timed_ms_per_step"] = round(step_ms, 3)
    out = {"roofline": roof}
    if tens is not None:
        out["roofline_tensor"] = obj(tens)
        # all tensor-bound classes together: the sweeps as a whole against the sustained bf16 rate
        fl = sum(work[r["kernel"]][1] * prof[r["kernel"]][2] for r in rows if r["bound"] in ("tensor", "alu"))
        ms = sum(r["total_ms"] for r in rows if r["bound"] in ("tensor", "alu"))
        out["roofline_tensor"]["all_tensor_classes"] = {
            "achieved": round(fl / (ms * 1e-3) / 1e12, 2), "unit": "TFLOP/s", "peak": pk["bf16_tflops_sustained"],
            "frac": round(fl / (ms * 1e-3) / 1e12 / pk["bf16_tflops_sustained"], 4), "share_of_device_time": round(ms / total_ms, 4)}
    if seqb is not None:
        out["roofline_seq_block"] = obj(seqb)
    return out, rows


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.lines, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7 or not (t0 <= ts <= t1 + 0.2):
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for nm, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# CPU oracle leg
# ------------------------------------------------------------------------------------------------
def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return 1


def oracle_run(cfg, blocks, z, labels, policy, tau, L):
    from oracle import tarflow_oracle as O
    t0 = time.perf_counter()
    O.model_inverse(blocks, z, labels, cfg, policy, tau, L + 1)
    return time.perf_counter() - t0


def cpu_sample_size(workload):
    return {"cfg1": 4, "cfg2": 2, "cfg3": 1, "cfg4": 1}.get(workload, 1)


def run_reference(args, cfg, L, rank):
    """The oracle as it stands, timed on the host cores: each step decodes a bounded sub-batch."""
    if rank != 0:
        return
    from paper_2505_24791_b200 import synth
    blocks = synth.make_weights(cfg)
    bs = cpu_sample_size(args.workload)
    policy = [0] + [1] * (cfg["n_blocks"] - 1)
    times = []
    args.warmup = min(args.warmup, 1)   # a CPU run needs no more than one untimed step; every step costs tens of seconds
    for i in range(args.warmup + args.steps):
        z = synth.make_latents(cfg, 4000 + i, B=bs)
        lab = synth.make_labels(cfg, B=bs)
        dt = oracle_run(cfg, blocks, z, lab, policy, cfg["tau"], L)
        if i >= args.warmup:
            times.append(dt)
    tot = sum(times)
    val = bs * len(times) / tot
    cores = oracle_threads()
    sample = f"{bs} of {cfg['B']} samples of the batch per step, selective policy, tau={cfg['tau']}"
    out = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": 1e3 * tot / len(times), "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": workload_config(args.workload, cfg, L, bs),
           "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
           "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


def workload_config(name, cfg, L, B):
    return {"workload": f"{name}: {cfg['C']}x{cfg['H']}x{cfg['W']} patch {cfg['patch']} -> {L} tokens, "
                        f"{cfg['n_blocks']} blocks x {cfg['n_layers']} layers, width {cfg['width']}, "
                        f"{cfg['n_heads']} heads, batch {B}",
            "policy": "selective (block 0 sequential with KV cache, others Jacobi)", "tau": cfg["tau"],
            "max_iters": L + 1, "batch_per_gpu": B, "l2": "flushed between timed steps (256 MiB write)"}


# ------------------------------------------------------------------------------------------------
# one workload on this rank's GPU
# ------------------------------------------------------------------------------------------------
class Runner:
    """A loaded model plus device / pinned-host inputs for `n_in` steps."""

    def __init__(self, name, cfg, B, n_in, rank, make_host=True):
        import torch
        from paper_2505_24791_b200 import binding, synth
        self.torch, self.binding, self.synth = torch, binding, synth
        self.name, self.cfg, self.B = name, cfg, B
        self.L, self.D = synth.seq_len(cfg), synth.token_dim(cfg)
        self.blocks = synth.make_weights(cfg)
        self.model = binding.tf_load(cfg, synth.pack_blob(cfg, self.blocks), B)
        self.K = cfg["n_blocks"]
        self.selective = [0] + [1] * (self.K - 1)
        self.tau, self.max_iters = cfg["tau"], self.L + 1
        self.stream = torch.cuda.current_stream()
        self.rank = rank
        lab_np = synth.make_labels(cfg, B=B, seed=synth.LABEL_SEED + rank)
        self.lab_np = lab_np
        self.z_np = [synth.make_latents(cfg, 1000 * (rank + 1) + i, B=B) for i in range(n_in)]
        self.z_dev = [torch.from_numpy(z).cuda() for z in self.z_np]
        self.lab_dev = None if lab_np is None else torch.from_numpy(lab_np).cuda()
        self.x_dev = torch.empty_like(self.z_dev[0])
        self.iters = np.zeros(self.K, dtype=np.int32)
        self.its_dev = torch.zeros((self.K, B), dtype=torch.int32, device="cuda")
        if make_host:
            self.z_host = [torch.from_numpy(z).pin_memory() for z in self.z_np]
            self.lab_host = None if lab_np is None else torch.from_numpy(lab_np).pin_memory()
            self.x_host = torch.empty_like(self.z_host[0]).pin_memory()

    def step_dev(self, i, pol=None, tau=None):
        return self.binding.tf_inverse_jacobi(self.model, self.z_dev[i], self.lab_dev, self.B, pol or self.selective,
                                              self.tau if tau is None else tau, self.max_iters, 0, self.x_dev, self.iters,
                                              self.its_dev, self.stream)

    def step_host(self, i):
        return self.binding.tf_inverse_jacobi_host(self.model, self.z_host[i], self.lab_host, self.B, self.selective,
                                                   self.tau, self.max_iters, 0, self.x_host, self.iters, None, self.stream)

    def close(self):
        self.binding.tf_free(self.model)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3", choices=["cfg1", "cfg2", "cfg3", "cfg4"])
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size")
    ap.add_argument("--tau", type=float, default=None)
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle leg")
    ap.add_argument("--no-policies", action="store_true", help="skip the all-sequential / all-Jacobi legs")
    ap.add_argument("--no-legs", action="store_true", help="skip the short legs on the other bf16 configurations")
    ap.add_argument("--kernels", action="store_true", help="add the per-kernel-class table to the JSON line")
    ap.add_argument("--maf", default=None, choices=["maf_ising", "maf_mnist"],
                    help="only the second workload (MLP-based flow, Jacobi on every layer): one JSON line, not the bench line")
    ap.add_argument("--sweep", default=None, choices=["cfg5"],
                    help="policy x batch x tau table on the class-conditional architecture (one JSON line, not the bench line)")
    ap.add_argument("--probe", default=None, choices=["sweep", "seq"],
                    help="small single-block run for ncu captures: 'sweep' = --sweeps fixed Jacobi sweeps of one block, "
                         "'seq' = one sequentially decoded block; run twice, the second call timed; not a bench value")
    ap.add_argument("--sweeps", type=int, default=2)
    ap.add_argument("--launch-list", action="store_true",
                    help="for an ncu launch-list capture: one warm-up (none with --warmup 0) and one step of the timed leg only; the line it "
                         "prints is marked as a profiling run and is not a bench value")
    args = ap.parse_args()
    if args.launch_list:
        args.warmup, args.steps, args.no_cpu, args.no_policies, args.no_legs = min(args.warmup, 1), 1, True, True, True
    elif args.warmup < 3 and args.impl == "ours":
        args.warmup = 3

    # `--gpus N` outside a torchrun environment: start the N ranks (one process per GPU) and relay their output
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not (args.probe or args.sweep or args.maf or args.launch_list):
        port = 29500 + (os.getpid() % 2000)
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.run(cmd).returncode)

    from paper_2505_24791_b200 import synth
    cfg = synth.config(args.workload)
    if args.tau is not None:
        cfg["tau"] = args.tau
    B = args.batch or cfg["B"]
    L, D = synth.seq_len(cfg), synth.token_dim(cfg)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, cfg, L, rank)
        return

    import torch
    import torch.distributed as dist
    import __graft_entry__ as entry
    entry.build()
    from paper_2505_24791_b200 import binding

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def timed(fn, idx, after=None):
        """Calls of fn(i), each bracketed by CUDA events on the launching stream; L2 flushed between."""
        barrier()
        t_wall0 = time.time()
        total = 0.0
        for i in idx:
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            fn(i)
            e1.record(stream)
            e1.synchronize()
            total += e0.elapsed_time(e1)
            if after is not None:
                after(i)
        barrier()
        t = torch.tensor([total], dtype=torch.float64, device="cuda")
        if world > 1:
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item()), t_wall0, time.time()

    if args.probe:
        run_probe(args, B, binding, synth, torch)
        return
    if args.sweep:
        run_cfg5_sweep(args, binding, synth, torch, timed)
        return
    if args.maf:
        print(json.dumps({"second_workload_maf": run_maf_leg(args.maf, binding, synth, torch, timed, peaks()[0])}), flush=True)
        return

    n_in = args.warmup + args.steps
    R = Runner(args.workload, cfg, B, n_in, rank)
    model, K = R.model, R.K
    warm, run = list(range(args.warmup)), list(range(args.warmup, n_in))
    for i in warm:
        R.step_dev(i)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    l0 = binding.tf_launch_count(model)
    block_ms = np.zeros(K)
    its_sum = np.zeros(K)
    its_max = np.zeros(K, dtype=np.int64)

    def after(_i):
        nonlocal block_ms, its_sum, its_max
        block_ms += binding.tf_block_times(model, K)
        its = R.its_dev.cpu().numpy()
        its_sum += its.mean(axis=1)
        its_max = np.maximum(its_max, its.max(axis=1))

    ms_total, w0, w1 = timed(R.step_dev, run, after)
    launches = binding.tf_launch_count(model) - l0
    clocks = sampler.stop(w0, w1) if rank == 0 else None
    value = world * B * args.steps / (ms_total * 1e-3)
    step_ms = ms_total / args.steps
    if args.launch_list:
        if rank == 0:
            print(json.dumps({"profiling_run": True, "note": "not a bench value", "ms_per_step": step_ms,
                              "gpu_launches": int(launches), "iters_per_block_max": [int(v) for v in its_max]}), flush=True)
        R.close()
        if world > 1:
            dist.destroy_process_group()
        return

    # end to end: pinned host latents in, host images out, copies inside the timed region
    for i in warm[:2]:
        R.step_host(i)
    ms_e2e, _, _ = timed(R.step_host, run)
    e2e_val = world * B * args.steps / (ms_e2e * 1e-3)
    nbytes = R.z_host[0].numel() * 4
    h2d = nbytes + (0 if R.lab_host is None else R.lab_host.numel() * 4)

    # per-kernel-class device time: the same steps again with the library's events on (the sweep kernels one by
    # one, the sequential block as it runs in the timed pass, as one unit)
    binding.tf_profile_enable(model, 2)
    ms_prof, _, _ = timed(R.step_dev, run)
    prof = binding.tf_profile_read(model)
    binding.tf_profile_enable(model, 0)
    pk, pk_kind = peaks()
    roofs, rows = roofline_report(prof, cfg, L, D, B, pk, pk_kind, args.workload, step_ms, ms_prof / args.steps)
    for r in roofs.values():
        r["launches_per_step"] = round(next(x["launches"] for x in rows if x["kernel"] == r["kernel"]) / args.steps, 1)

    # active samples per sweep of one step (the stopping test already reads the device every sweep, so the trace is free)
    binding.tf_trace_enable(model, 1)
    R.step_dev(run[0])
    trace = binding.tf_trace_read(model)
    binding.tf_trace_enable(model, 0)
    active = [[a for g, t, a, md in trace if g == gg] for gg in range(K)]

    seq_bytes, w_blk = seq_block_bytes(cfg, L, D, B)
    blocks_out = {"ms_per_block": [round(float(v), 3) for v in block_ms / args.steps],
                  "share_of_step": [round(float(v), 4) for v in block_ms / args.steps / step_ms],
                  "policy": R.selective, "sweeps_max": [int(v) for v in its_max],
                  "sweeps_mean": [round(float(v), 2) for v in its_sum / args.steps],
                  "active_samples_per_sweep": active}
    # the sequential block from the timed pass itself: bytes it must stream / its time
    if block_ms[0] > 0:
        gbs = seq_bytes / (block_ms[0] / args.steps * 1e-3) / 1e9
        blocks_out["seq_block_timed"] = {"ms": round(float(block_ms[0] / args.steps), 3), "algorithmic_bytes": seq_bytes,
                                         "achieved_gbs": round(gbs, 1), "frac_of_hbm_peak": round(gbs / pk["hbm_gbs"], 4),
                                         "weights_per_block_bytes": w_blk}

    extra = {}
    if not args.no_policies:
        for name, pol, n in (("gpu_sequential", [0] * K, 2), ("gpu_all_jacobi", [1] * K, 3)):
            R.step_dev(0, pol)
            ms, _, _ = timed(lambda i, pol=pol: R.step_dev(i, pol), run[:n])
            k = len(run[:n])
            extra[name] = {"value": world * B * k / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms / k, "steps": k,
                           "iters_per_block": [int(v) for v in R.iters]}
        extra["selective_over_sequential"] = round(value / extra["gpu_sequential"]["value"], 3)

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
           "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "bf16" if cfg["dtype"] == 1 else "f32", "data": "synthetic",
           "config": workload_config(args.workload, cfg, L, B),
           "iters_per_block_max": [int(v) for v in its_max],
           "iters_per_block_mean": [round(float(v), 2) for v in its_sum / args.steps],
           "clocks": clocks,
           "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": nbytes,
                   "ms_per_step": ms_e2e / args.steps},
           "gpu_launches": int(launches), "device_bytes": int(binding.tf_device_bytes(model)), "blocks": blocks_out}
    out.update(roofs)
    out.update(extra)
    if args.kernels:
        out["kernels"] = rows

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        bs = min(cpu_sample_size(args.workload), B)
        z, lab = R.z_np[args.warmup], R.lab_np
        dt = oracle_run(cfg, R.blocks, z[:bs], None if lab is None else lab[:bs], R.selective, R.tau, L)
        cpu = {"value": bs / dt, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
               "sample": f"first {bs} of the {B} samples of one step, selective policy, tau={R.tau}, {dt:.1f} s",
               "host_cpus": os.cpu_count()}
        out["cpu_baseline"] = cpu
    R.close()
    del R

    # short legs on the other bf16 configurations: the target is stated for all of them
    if world == 1 and not args.no_legs and args.workload in ("cfg2", "cfg3", "cfg4") and not args.batch:
        legs = {}
        for name in ("cfg2", "cfg3", "cfg4"):
            if name == args.workload:
                continue
            c2 = synth.config(name)
            R2 = Runner(name, c2, c2["B"], 4, rank, make_host=False)
            leg = {"config": workload_config(name, c2, R2.L, c2["B"])["workload"]}
            for pname, pol in (("selective", R2.selective), ("sequential", [0] * R2.K), ("all_jacobi", [1] * R2.K)):
                R2.step_dev(0, pol)
                n = 2 if pname == "sequential" else 3
                ms, _, _ = timed(lambda i, pol=pol: R2.step_dev(i, pol), [1, 2, 3][:n])
                leg[pname] = {"value": R2.B * n / (ms * 1e-3), "unit": UNIT, "ms_per_step": round(ms / n, 3), "steps": n,
                              "iters_per_block": [int(v) for v in R2.iters]}
                if pname == "selective":
                    leg["ms_per_block_selective"] = [round(float(v), 3) for v in binding.tf_block_times(R2.model, R2.K)]
            leg["selective_over_sequential"] = round(leg["selective"]["value"] / leg["sequential"]["value"], 3)
            legs[name] = leg
            R2.close()
            del R2
        out["other_workloads"] = legs
        out["second_workload_maf"] = run_maf_leg("maf_ising", binding, synth, torch, timed, pk)

    if rank == 0:
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_maf_leg(name, binding, synth, torch, timed, pk, steps=3):
    """Second workload (paper App. E.3): Jacobi decoding on every layer of an MLP-based autoregressive flow against
    sequential decoding (D whole passes per layer, no cache exists).  -> dict for the JSON line."""
    cfg = synth.maf_config(name)
    B, D, H, K = cfg["B"], cfg["D"], cfg["hidden"], cfg["n_blocks"]
    blocks = synth.make_maf_weights(cfg)
    model = binding.tf_maf_load(cfg, synth.pack_maf_blob(cfg, blocks), B)
    stream = torch.cuda.current_stream()
    zs = [torch.from_numpy(synth.make_maf_latents(cfg, 9000 + i, B=B)).cuda() for i in range(steps + 1)]
    x = torch.empty_like(zs[0])
    iters = np.zeros(K, dtype=np.int32)
    its = torch.zeros((K, B), dtype=torch.int32, device="cuda")

    def jac(i):
        return binding.tf_maf_inverse_jacobi(model, zs[i], B, cfg["tau"], D + 1, 0, x, iters, its, stream)

    jac(0)
    ms, _, _ = timed(jac, list(range(1, steps + 1)))
    ms /= steps
    itn = its.cpu().numpy()
    flops_row = 2.0 * (D * H + H * H + 2 * D * H)                     # one pass of one sample through one layer
    rows = float(itn.sum())                                            # sample-sweeps of the last step
    out = {"config": f"{name}: {D} dimensions, {K} layers, hidden {H}, batch {B}, tau {cfg['tau']}",
           "jacobi": {"value": B / (ms * 1e-3), "unit": UNIT, "ms_per_step": round(ms, 3), "steps": steps,
                      "sweeps_max": [int(v) for v in itn.max(axis=1)], "sweeps_mean": [round(float(v), 2) for v in itn.mean(axis=1)],
                      "ms_per_block": [round(float(v), 3) for v in binding.tf_block_times(model, K)],
                      "tensor_frac": round(rows * flops_row / (ms * 1e-3) / 1e12 / pk["bf16_tflops_sustained"], 4)}}
    Bs = min(B, 16384)                                                 # sequential decoding: a bounded sub-batch
    binding.tf_maf_inverse_sequential(model, zs[0][:Bs].contiguous(), Bs, x[:Bs], stream)
    zsub = [z[:Bs].contiguous() for z in zs]
    ms_s, _, _ = timed(lambda i: binding.tf_maf_inverse_sequential(model, zsub[i], Bs, x[:Bs], stream), [1])
    out["sequential"] = {"value": Bs / (ms_s * 1e-3), "unit": UNIT, "ms_per_step": round(ms_s, 3), "steps": 1, "batch": Bs,
                         "passes_per_layer": D,
                         "tensor_frac": round(Bs * K * D * flops_row / (ms_s * 1e-3) / 1e12 / pk["bf16_tflops_sustained"], 4)}
    out["jacobi_over_sequential"] = round(out["jacobi"]["value"] / out["sequential"]["value"], 2)
    binding.tf_free(model)
    return out


def run_probe(args, B, binding, synth, torch):
    cfg1 = synth.config(args.workload, n_blocks=1)
    m1 = binding.tf_load(cfg1, synth.pack_blob(cfg1, synth.make_weights(cfg1)), B)
    z = torch.from_numpy(synth.make_latents(cfg1, 1, B=B)).cuda()
    lab = synth.make_labels(cfg1, B=B)
    lab = None if lab is None else torch.from_numpy(lab).cuda()
    x = torch.empty_like(z)
    it = np.zeros(1, dtype=np.int32)
    ms = 0.0
    for _ in range(2):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        if args.probe == "sweep":
            binding.tf_inverse_jacobi(m1, z, lab, B, [1], -1.0, args.sweeps, 0, x, it)
        else:
            binding.tf_inverse_jacobi(m1, z, lab, B, [0], 0.0, 1, 0, x, it)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
    per = ms / args.sweeps if args.probe == "sweep" else ms
    print(json.dumps({"profiling_run": True, "note": "not a bench value", "probe": args.probe, "workload": args.workload,
                      "batch": B, "ms_per_sweep" if args.probe == "sweep" else "ms_per_sequential_block": per,
                      "finite": bool(torch.isfinite(x).all())}), flush=True)
    binding.tf_free(m1)


def run_cfg5_sweep(args, binding, synth, torch, timed):
    """Policy x batch x tau on the class-conditional architecture: sweeps per block, samples/s, and for each cell the
    roofline fraction that bounds it -- device-memory bytes for sequential decoding and for small-batch sweeps (which
    stream the weights once per sweep), tensor FLOPs for large-batch sweeps."""
    cfg = synth.config("cfg3")
    L, D, K = synth.seq_len(cfg), synth.token_dim(cfg), cfg["n_blocks"]
    pk, pk_kind = peaks()
    blocks = synth.make_weights(cfg)
    model = binding.tf_load(cfg, synth.pack_blob(cfg, blocks), 256)
    stream = torch.cuda.current_stream()
    frow = sweep_flops_per_row(cfg, L, D)
    _, w_blk = seq_block_bytes(cfg, L, D, 1)
    cells = []
    for B in ((args.batch,) if args.batch else (1, 8, 64, 256)):
        zs = [torch.from_numpy(synth.make_latents(cfg, 7000 + i, B=B)).cuda() for i in range(3)]
        lab = torch.from_numpy(synth.make_labels(cfg, B=B)).cuda()
        x = torch.empty_like(zs[0])
        iters = np.zeros(K, dtype=np.int32)
        its = torch.zeros((K, B), dtype=torch.int32, device="cuda")
        for pname, pol in (("all_sequential", [0] * K), ("all_jacobi", [1] * K), ("selective", [0] + [1] * (K - 1))):
            for tau in ((1e-3,) if pname == "all_sequential" else (1e-2, 1e-3, 1e-4)):
                def step(i, pol=pol, tau=tau):
                    return binding.tf_inverse_jacobi(model, zs[i], lab, B, pol, tau, L + 1, 0, x, iters, its, stream)
                rc = step(0)
                n = 2
                ms, _, _ = timed(step, [1, 2])
                ms /= n
                itn = its.cpu().numpy()
                nseq = sum(1 for p in pol if p == 0)
                jac_rows = float(sum(itn[g].sum() for g in range(K) if pol[g] == 1)) * L     # rows of the last step
                seq_bytes = nseq * seq_block_bytes(cfg, L, D, B)[0]
                sweeps_total = float(sum(itn[g].max() for g in range(K) if pol[g] == 1))
                jac_bytes = sweeps_total * w_blk                                             # weights once per sweep
                cell = {"batch": B, "policy": pname, "tau": None if pname == "all_sequential" else tau, "status": int(rc),
                        "samples_per_s": round(B / (ms * 1e-3), 2), "ms_per_step": round(ms, 3),
                        "sweeps_max": [int(v) for v in itn.max(axis=1)],
                        "sweeps_mean": [round(float(v), 2) for v in itn.mean(axis=1)],
                        "ms_per_block": [round(float(v), 3) for v in binding.tf_block_times(model, K)],
                        "tensor_frac": round(jac_rows * frow / (ms * 1e-3) / 1e12 / pk["bf16_tflops_sustained"], 4),
                        "hbm_frac": round((seq_bytes + jac_bytes) / (ms * 1e-3) / 1e9 / pk["hbm_gbs"], 4)}
                cell["bound"] = "tensor" if cell["tensor_frac"] >= cell["hbm_frac"] else "hbm"
                cells.append(cell)
    binding.tf_free(model)
    print(json.dumps({"sweep": "cfg5", "note": "policy x batch x tau on the class-conditional architecture; whole-step "
                      "fractions: tensor = sweep FLOPs / time / sustained bf16 peak, hbm = (sequential-block bytes + weights "
                      "once per sweep) / time / copy bandwidth", "peaks": f"of {pk_kind}", "workload":
                      workload_config("cfg5", cfg, L, "1|8|64|256")["workload"], "cells": cells}), flush=True)


if __name__ == "__main__":
    main()
