#!/usr/bin/env python
"""Benchmark of selective-Jacobi TarFlow sampling on B200 (one process per GPU).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl ours|reference]

A "step" is one whole sampling call (patchify, block 0 decoded sequentially with the KV cache, the
other blocks by Jacobi sweeps with the per-sample stopping test, unpatchify) over one batch of seeded
synthetic latents.  The line printed by rank 0 carries:
  value     samples/s with the latents already resident in device memory (CUDA events, max over ranks),
  e2e       the same through the host-buffer entry point (pinned host z in, x out, copies timed),
  roofline  the kernel class with the largest share of device time, from per-launch CUDA events
            recorded by the library on the launching stream in a second pass over the same steps,
  gpu_sequential / gpu_all_jacobi   the same batch decoded with the other policies,
  cpu_baseline   the fp64 CPU oracle timed on this machine's host cores on a bounded sub-batch.
`--impl reference` times only the CPU oracle (there is no other implementation of the paper).
With N > 1 (torchrun) every rank decodes its own batch (weak scaling, no data-path collective).
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

# dram bytes per launch (read + write) of a kernel class from the committed ncu capture of that class;
# None = no capture of the current kernel.  {workload: {class: bytes}}
# cfg2 / seq_gemm: mean over the 16 layer GEMMs of one decoding step (27.33 MB read, 0 written) in the ncu summary of
# that kernel under profiles/, captured with L2 flushed between replays; the algorithmic figure is 1.57 MB.
NCU_TRAFFIC: dict = {"cfg2": {"seq_gemm": 27.33e6 / 16}}


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
def class_work(cfg, L, D):
    """-> {class: (bound, per_row, per_launch)}: FLOPs (bound 'tensor') or bytes (bound 'hbm').

    per_row multiplies the activation rows a launch processed, per_launch is added once per launch.
    GEMM [rows, K] x [N, K]^T: 2*N*K FLOPs per row.  Causal attention: QK^T and PV are d*L^2 FLOPs
    each per sample and layer, i.e. 2*d*L per row.  Bandwidth-bound classes: the bytes of every
    operand read once and every result written once (esz = operand size, residual stream fp32).
    A sequential step streams each weight matrix once per launch whatever the batch.
    """
    d, hid, nl = cfg["width"], cfg["width"] * cfg["mlp_ratio"], cfg["n_layers"]
    esz = 2 if cfg["dtype"] == 1 else 4
    bound = "tensor" if cfg["dtype"] == 1 else "alu"
    w_layer = 3 * d * d + d * d + 2 * hid * d
    # a small head (<= 64 KB) is part of the one-kernel step tail, not a GEMM launch of its own
    head_gemm = not (cfg["dtype"] == 1 and 2 * D * d * esz <= 64 * 1024)
    seq_launches = nl * 4 + (1 if head_gemm else 0)
    seq_w_bytes = (nl * w_layer + (2 * D * d if head_gemm else 0)) * esz / seq_launches  # mean per launch of the class
    return {
        "gemm_qkv": (bound, 2.0 * 3 * d * d, 0.0),
        "gemm_out": (bound, 2.0 * d * d, 0.0),
        "gemm_mlp_up": (bound, 2.0 * hid * d, 0.0),
        "gemm_mlp_down": (bound, 2.0 * hid * d, 0.0),
        "gemm_head_update": (bound, 2.0 * 2 * D * d, 0.0),
        "gemm_head": (bound, 2.0 * 2 * D * d, 0.0),
        "attention": (bound, 2.0 * d * L, 0.0),
        "layernorm": ("hbm", d * (4.0 + esz), 0.0),
        "embed": ("hbm", D * 4.0 + d * (4.0 + esz), 0.0),  # token in, residual row and first LayerNorm's row out
        "forward_affine": ("hbm", D * (2 * 4.0 + 2 * 4.0), 0.0),
        "layout": ("hbm", 0.0, 0.0),
        "sweep_control": ("hbm", 0.0, 0.0),
        "seq_gemm": ("hbm", 0.0, seq_w_bytes),
        "seq_attention": ("hbm", (L / 2.0) * 2 * d * esz, 0.0),  # mean cache rows read per step: K and V
        "seq_layernorm": ("hbm", d * (4.0 + esz), 0.0),
        "seq_embed": ("hbm", D * 4.0 + d * 4.0, 0.0),
        "seq_update": ("hbm", D * 4.0 * 4 + (0.0 if head_gemm else 2 * d * (4.0 + esz) + 2 * D * d * esz), 0.0),
        "seq_step": ("hbm", (L / 2.0) * 2 * d * esz * nl, (nl * w_layer + 2 * D * d) * esz),
    }


def roofline_report(prof, cfg, L, D, pk, pk_kind, workload):
    work = class_work(cfg, L, D)
    total_ms = sum(v[0] for v in prof.values()) or 1.0
    rows = []
    for name, (ms, n, nrows) in prof.items():
        if n == 0:
            continue
        bound, per_row, per_launch = work.get(name, ("hbm", 0.0, 0.0))
        amount = per_row * nrows + per_launch * n  # FLOPs or bytes over all launches
        avg_s = ms * 1e-3 / n
        if bound == "hbm":
            achieved, peak, unit = amount / n / avg_s / 1e9, pk["hbm_gbs"], "GB/s"
        else:
            achieved, peak, unit = amount / n / avg_s / 1e12, pk["bf16_tflops_sustained"], "TFLOP/s"
        rows.append({"kernel": name, "launches": int(n), "total_ms": round(ms, 4), "share": round(ms / total_ms, 4),
                     "avg_us": round(avg_s * 1e6, 3), "bound": bound, "achieved": round(achieved, 2), "peak": peak,
                     "unit": unit, "frac": round(achieved / peak, 4)})
    rows.sort(key=lambda r: -r["total_ms"])
    top = rows[0]
    roof = {"kernel": top["kernel"], "bound": top["bound"], "achieved": top["achieved"], "peak": top["peak"],
            "unit": top["unit"], "frac": top["frac"], "traffic": NCU_TRAFFIC.get(workload, {}).get(top["kernel"]),
            "peak_source": f"of {pk_kind}" + (" (sustained bf16)" if top["bound"] == "tensor" else ""),
            "share_of_device_time": top["share"], "avg_launch_us": top["avg_us"]}
    return roof, rows


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
# main
# ------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg1", "cfg2", "cfg3", "cfg4"])
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size")
    ap.add_argument("--tau", type=float, default=None)
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle leg")
    ap.add_argument("--no-policies", action="store_true", help="skip the all-sequential / all-Jacobi legs")
    ap.add_argument("--kernels", action="store_true", help="add the per-kernel-class table to the JSON line")
    ap.add_argument("--probe", default=None, choices=["sweep", "seq"],
                    help="small single-block run for ncu captures: 'sweep' = --sweeps fixed Jacobi sweeps of one block, "
                         "'seq' = one sequentially decoded block; run twice, the second call timed; not a bench value")
    ap.add_argument("--sweeps", type=int, default=2)
    ap.add_argument("--launch-list", action="store_true",
                    help="for an ncu launch-list capture: one warm-up and one step of the timed leg only; the line it "
                         "prints is marked as a profiling run and is not a bench value")
    args = ap.parse_args()
    if args.launch_list:
        args.warmup, args.steps, args.no_cpu, args.no_policies = 1, 1, True, True
    elif args.warmup < 3 and args.impl == "ours":
        args.warmup = 3

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

    if args.probe:
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
        return

    blocks = synth.make_weights(cfg)
    blob = synth.pack_blob(cfg, blocks)
    model = binding.tf_load(cfg, blob, B)
    policy = [0] + [1] * (cfg["n_blocks"] - 1)
    tau, max_iters = cfg["tau"], L + 1
    stream = torch.cuda.current_stream()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def latents(i):
        z = synth.make_latents(cfg, 1000 * (rank + 1) + i, B=B)
        lab = synth.make_labels(cfg, B=B, seed=synth.LABEL_SEED + rank)
        return z, lab

    n_in = args.warmup + args.steps
    z_host = [torch.from_numpy(latents(i)[0]).pin_memory() for i in range(n_in)]
    lab_np = latents(0)[1]
    lab_host = None if lab_np is None else torch.from_numpy(lab_np).pin_memory()
    lab_dev = None if lab_np is None else lab_host.cuda()
    z_dev = [z.cuda() for z in z_host]
    x_dev = torch.empty_like(z_dev[0])
    x_host = torch.empty_like(z_host[0]).pin_memory()
    iters = np.zeros(cfg["n_blocks"], dtype=np.int32)
    its_dev = torch.zeros((cfg["n_blocks"], B), dtype=torch.int32, device="cuda")

    def timed(fn, idx):
        """K calls of fn(i), each bracketed by CUDA events on the launching stream; L2 flushed between."""
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
        barrier()
        t = torch.tensor([total], dtype=torch.float64, device="cuda")
        if world > 1:
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item()), t_wall0, time.time()

    def step_dev(i, pol=policy):
        return binding.tf_inverse_jacobi(model, z_dev[i], lab_dev, B, pol, tau, max_iters, 0, x_dev, iters, its_dev,
                                         stream)

    def step_host(i):
        return binding.tf_inverse_jacobi_host(model, z_host[i], lab_host, B, policy, tau, max_iters, 0, x_host, iters,
                                              None, stream)

    warm, run = list(range(args.warmup)), list(range(args.warmup, n_in))
    for i in warm:
        step_dev(i)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    l0 = binding.tf_launch_count(model)
    ms_total, w0, w1 = timed(step_dev, run)
    launches = binding.tf_launch_count(model) - l0
    clocks = sampler.stop(w0, w1) if rank == 0 else None
    iters_sel = iters.copy()
    its_mean = its_dev.float().mean(dim=1).cpu().numpy()
    value = world * B * args.steps / (ms_total * 1e-3)
    if args.launch_list:
        if rank == 0:
            print(json.dumps({"profiling_run": True, "note": "not a bench value", "ms_per_step": ms_total / args.steps,
                              "gpu_launches": int(launches), "iters_per_block_max": [int(v) for v in iters_sel]}), flush=True)
        binding.tf_free(model)
        if world > 1:
            dist.destroy_process_group()
        return

    # end to end: pinned host latents in, host images out, copies inside the timed region
    for i in warm[:2]:
        step_host(i)
    ms_e2e, _, _ = timed(step_host, run)
    e2e_val = world * B * args.steps / (ms_e2e * 1e-3)
    nbytes = z_host[0].numel() * 4
    h2d = nbytes + (0 if lab_host is None else lab_host.numel() * 4)

    # per-kernel-class device time: same steps again with the library's per-launch events on
    binding.tf_profile_enable(model, 1)
    ms_prof, _, _ = timed(step_dev, run)
    prof = binding.tf_profile_read(model)
    binding.tf_profile_enable(model, 0)
    pk, pk_kind = peaks()
    roof, rows = roofline_report(prof, cfg, L, D, pk, pk_kind, args.workload)
    roof["profiled_ms_per_step"] = round(ms_prof / args.steps, 3)

    extra = {}
    if not args.no_policies:
        for name, pol, n in (("gpu_sequential", [0] * cfg["n_blocks"], 2), ("gpu_all_jacobi", [1] * cfg["n_blocks"], 3)):
            step_dev(0, pol)
            ms, _, _ = timed(lambda i, pol=pol: step_dev(i, pol), run[:n])
            k = len(run[:n])
            extra[name] = {"value": world * B * k / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms / k, "steps": k,
                           "iters_per_block": [int(v) for v in iters]}

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
           "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "bf16" if cfg["dtype"] == 1 else "f32", "data": "synthetic",
           "config": workload_config(args.workload, cfg, L, B),
           "iters_per_block_max": [int(v) for v in iters_sel], "iters_per_block_mean": [round(float(v), 2) for v in its_mean],
           "clocks": clocks,
           "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": nbytes,
                   "ms_per_step": ms_e2e / args.steps},
           "gpu_launches": int(launches), "roofline": roof, "device_bytes": int(binding.tf_device_bytes(model))}
    out.update(extra)
    if args.kernels:
        out["kernels"] = rows

    if rank == 0 and world == 1 and not args.no_cpu:
        bs = min(cpu_sample_size(args.workload), B)
        z, lab = latents(args.warmup)
        dt = oracle_run(cfg, blocks, z[:bs], None if lab is None else lab[:bs], policy, tau, L)
        out["cpu_baseline"] = {"value": bs / dt, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                               "sample": f"first {bs} of the {B} samples of one step, selective policy, tau={tau}, "
                                         f"{dt:.1f} s", "host_cpus": os.cpu_count()}
    binding.tf_free(model)
    if rank == 0:
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
