#!/usr/bin/env python
"""Benchmark of the TSVD linear map y = U(diag(S)(V x)) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config cfg2]

One step = one full forward (V-stage, S scale, U-stage) over one batch of B synthetic
tokens.  Prints ONE JSON line: tokens/s with inputs resident in HBM (`value`), the same
through the host-buffer entry point with copies inside the timed region (`e2e`), the
roofline figures of the dominant kernel, and the CPU checker timed on the host cores.
With N > 1 (torchrun) every rank runs its own replica on its own tokens (weak scaling,
no data-path collective); the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import gen  # noqa: E402

METRIC = "tsvd_linear_tokens_per_s"
UNIT = "tokens/s"
L2_FLUSH_BYTES = 256 << 20
# measured on this machine's B200s (copy bandwidth, cuBLAS bf16 burst / sustained); used when
# MEASURED_PEAKS.json is not next to this file
PEAKS_COPY = {"hbm_gbs": 6524.9, "bf16_tflops": 1681.0, "bf16_tflops_sustained": 1398.7}
INT8_OVER_BF16 = 2.0  # nominal dense tensor ratio (4.5 / 2.25 PFLOP/s)


def max_over_ranks(dist, value, device):
    """Max of a per-rank scalar over all ranks (the time every N-GPU number is taken on)."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tokens_per_s(world, tokens_per_rank, ms_per_step_max):
    """Whole-job throughput of `world` replicas that each process their own tokens per step."""
    return world * tokens_per_rank / (ms_per_step_max * 1e-3)


def rank_spec(spec, rank):
    """Rank r works on its own tokens of the same layer (weak scaling: same B per rank)."""
    return gen.scaled(spec, seed=spec.seed + 1000 * rank) if rank else spec


def kernel_source_sha1(names):
    import hashlib
    h = hashlib.sha1()
    for name in names:
        with open(os.path.join(ROOT, "paper_2308_07641_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def recorded_traffic(workload, stage):
    """DRAM bytes per launch from the committed ncu capture, or None when the sources of the kernels
    that workload runs have changed since that capture was taken (profiles/dram_traffic.txt holds
    JSON: per workload the source files hashed, their hash, and the bytes per launch of each stage)."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.txt")) as f:
            d = json.load(f)["workloads"][workload]
        if d["sha1"] != kernel_source_sha1(d["sources"]):
            return None
        return d["bytes_per_launch"][stage]
    except Exception:
        return None


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in PEAKS_COPY}, "MEASURED_PEAKS.json"
    except Exception:
        return dict(PEAKS_COPY), "copy of MEASURED_PEAKS.json values recorded in bench.py"


class ClockSampler:
    """nvidia-smi clock / throttle-reason sampler running during the timed region."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1])); mx.append(float(parts[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                    "sw_power_cap"), parts[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
        finally:
            try:
                os.unlink(self.path)
            except OSError:
                pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


def cpu_baseline(spec, U, S, V, x_np, target_s=8.0, y_gpu=None):
    """Time the CPU checker, as it stands, on a bounded sample of the workload's tokens."""
    import oracle
    cores = oracle.threads()
    n0 = min(spec.B, max(cores, 8))
    xs = gen.widen_x(x_np[:n0], spec.x_dtype)
    oracle.forward(U, S, V, xs[:1])                      # warm-up (page in, thread pool)
    t0 = time.perf_counter(); oracle.forward(U, S, V, xs); t1 = time.perf_counter()
    per_tok = (t1 - t0) / n0
    n = int(min(spec.B, max(n0, target_s / max(per_tok, 1e-9))))
    n = max(cores, n - n % cores) if n >= cores else n
    xs = gen.widen_x(x_np[:n], spec.x_dtype)
    t0 = time.perf_counter(); ref = oracle.forward(U, S, V, xs); t1 = time.perf_counter()
    out = {"value": n / (t1 - t0), "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": f"first {n} of {spec.B} tokens of {spec.name}, one call, {t1 - t0:.2f} s wall"}
    parity = None
    if y_gpu is not None:
        err = np.abs(y_gpu[:n] - ref.y)
        if spec.x_dtype == "bf16":
            tol = 1e-2 * np.abs(ref.y) + 1e-3
            parity = {"tokens": n, "violations": int((err > tol).sum()), "worst_err_over_tol": float((err / tol).max())}
        else:
            parity = {"tokens": n, "max_err_over_max_ref": float(err.max() / np.abs(ref.y).max())}
    return out, parity


def run_reference(args, spec):
    """--impl reference: the CPU checker on the host cores, same workload and metric."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    U, V, S = gen.make_weights(spec)
    cores = oracle.threads()
    # size the per-step sample so that warmup+steps stay within about two minutes
    x_probe = gen.make_x(spec, 0, min(spec.B, cores))
    xp = gen.widen_x(x_probe, spec.x_dtype)
    oracle.forward(U, S, V, xp[:1])
    t0 = time.perf_counter(); oracle.forward(U, S, V, xp); per_tok = (time.perf_counter() - t0) / len(xp)
    budget = 100.0 / max(1, args.steps + args.warmup)
    n = int(min(spec.B, max(cores, budget / max(per_tok, 1e-9))))
    n = max(1, n - n % cores) if n >= cores else n
    x = gen.widen_x(gen.make_x(spec, 0, n), spec.x_dtype)
    for _ in range(args.warmup):
        oracle.forward(U, S, V, x)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.forward(U, S, V, x)
    dt = (time.perf_counter() - t0) / args.steps
    val = n / dt
    sample = f"{n} of {spec.B} tokens of {spec.name} per step"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(spec, "host cores; no GPU"),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def workload_config(spec, l2_note):
    return {"workload": spec.name, "M": spec.M, "N": spec.N, "K": spec.K, "B": spec.B,
            "density": spec.density, "x_dtype": spec.x_dtype, "s_dist": spec.s_dist, "seed": spec.seed,
            "l2": l2_note}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="cfg2", choices=sorted(gen.CONFIGS))
    ap.add_argument("--path", default="auto", choices=["auto", "simple", "decode", "tensor", "index"],
                    help="index = the index-list form (one to four tokens; meant for nonzero rates below 1/8)")
    ap.add_argument("--density", type=float, default=None,
                    help="override the workload's nonzero rate of U and V (the sparse sweep of the index-list form)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--eager", action="store_true", help="time eager launches with an L2 flush per step")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    spec = gen.CONFIGS[args.config]
    if args.density is not None:
        spec = gen.scaled(spec, name=f"{spec.name}_density{args.density:g}", density=args.density)

    if args.impl == "reference":
        run_reference(args, spec)
        return

    import torch
    from paper_2308_07641_b200 import TSVDLinear, binding, build as lib_build
    from paper_2308_07641_b200 import TSVD_FLAG_PATH_DECODE, TSVD_FLAG_PATH_SIMPLE, TSVD_FLAG_PATH_TENSOR

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the TSVD library has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        lib_build.build()
    if dist:
        dist.barrier()

    flags = {"auto": 0, "simple": TSVD_FLAG_PATH_SIMPLE, "decode": TSVD_FLAG_PATH_DECODE,
             "tensor": TSVD_FLAG_PATH_TENSOR, "index": binding.TSVD_FLAG_PATH_INDEX}[args.path]
    pack_flags = binding.TSVD_PACK_INDEX_LISTS if args.path == "index" else 0
    U, V, S = gen.make_weights(spec)
    x_np = gen.make_x(rank_spec(spec, rank))
    layer = TSVDLinear(U, S, V, pack_flags)
    info = layer.info
    from paper_2308_07641_b200 import device_activations
    x = device_activations(x_np, spec.x_dtype)
    y = layer.forward(x, flags=flags)
    torch.cuda.synchronize()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    # Rotating input/output buffers: together larger than twice the L2, so that every step
    # streams its activations from HBM and writes its results there.
    l2_bytes = int(torch.cuda.get_device_properties(local_rank).L2_cache_size)
    pair_bytes = x.numel() * x.element_size() + y.numel() * y.element_size()
    n_sets = int(min(64, max(2, -(-2 * l2_bytes // pair_bytes))))
    xs = [x] + [torch.roll(x, i, dims=0).contiguous() for i in range(1, n_sets)]
    ys = [y] + [torch.empty_like(y) for _ in range(1, n_sets)]
    # When the packed weights outweigh the activations (small batches) the weights are what must
    # come from HBM: pack the same layer several times and rotate over the copies as well.
    n_layers = 1
    if info["packed_bytes"] > pair_bytes:
        n_layers = int(min(64, max(2, -(-2 * l2_bytes // info["packed_bytes"]))))
    layers = [layer] + [TSVDLinear(U, S, V, pack_flags) for _ in range(1, n_layers)]
    for i, extra in enumerate(layers[1:]):       # size their scratch outside any timed region
        extra.forward(xs[0], out=ys[0], flags=flags)

    for i in range(args.warmup):
        flush.zero_()
        layer.forward(xs[i % n_sets], out=ys[i % n_sets], flags=flags)
    barrier()

    def timed_pass(steps):
        """`steps` eager forwards, L2 flushed before each, one CUDA-event pair per step."""
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        barrier()
        for a, b in ev:
            flush.zero_()                 # evict inputs, outputs and weights from L2 between steps
            a.record()
            layer.forward(x, out=y, flags=flags)
            b.record()
        barrier()
        return [a.elapsed_time(b) for a, b in ev]

    def graph_pass(steps):
        """`steps` forwards captured in one CUDA graph (no host launch latency between kernels),
        replayed once between two events; returns (total ms, launches in the graph)."""
        side = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        n0 = binding.tsvd_launch_count()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for i in range(steps):
                    layers[i % n_layers].forward(xs[i % n_sets], out=ys[i % n_sets], flags=flags)
        n_launch = binding.tsvd_launch_count() - n0
        g.replay()                         # one untimed replay (graph upload)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        a.record()
        g.replay()
        b.record()
        barrier()
        return a.elapsed_time(b), n_launch

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    # pass 1: the timed region proper (no per-kernel events: they cost ~5 us per kernel)
    if args.eager:
        launches0 = binding.tsvd_launch_count()
        step_ms = timed_pass(args.steps)
        launches = binding.tsvd_launch_count() - launches0
        total_ms = float(sum(step_ms))
        l2_note = "flushed between steps (256 MiB memset); eager launches"
    else:
        total_ms, launches = graph_pass(args.steps)
        l2_note = (f"inputs larger than L2: {n_sets} rotating x/y buffer pairs ({n_sets * pair_bytes / 1e6:.0f} MB) and "
                   f"{n_layers} packed copies of the layer ({n_layers * info['packed_bytes'] / 1e6:.0f} MB) against "
                   f"{l2_bytes / 1e6:.0f} MB of L2; the {args.steps} steps are one CUDA graph")
    # pass 2: the same steps again with an event pair around every kernel, for the roofline
    binding.tsvd_profile_enable(layer.handle, True)
    prof_step_ms = timed_pass(args.steps)
    stage_ms, stage_n = binding.tsvd_profile_read(layer.handle)
    binding.tsvd_profile_enable(layer.handle, False)
    clocks = sampler.stop() if rank == 0 else None
    total_ms = max_over_ranks(dist, total_ms, "cuda")
    ms_per_step = total_ms / args.steps
    value = aggregate_tokens_per_s(world, spec.B, ms_per_step)

    # end to end: host buffers, copies inside the timed region
    x_host = torch.from_numpy(x_np.view(np.int16) if spec.x_dtype == "bf16" else x_np).pin_memory()
    y_bf16 = y.dtype == torch.bfloat16
    y_host = torch.empty((spec.B, spec.M), dtype=torch.int16 if y_bf16 else torch.float32).pin_memory()
    dt_code = binding.DTYPES[spec.x_dtype]
    e2e_steps = max(3, min(args.steps, 20))
    for _ in range(2):
        binding.tsvd_forward_host(layer.handle, x_host.data_ptr(), y_host.data_ptr(), spec.B, dt_code, flags)
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        binding.tsvd_forward_host(layer.handle, x_host.data_ptr(), y_host.data_ptr(), spec.B, dt_code, flags)
    torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / e2e_steps
    e2e_s = max_over_ranks(dist, e2e_s, "cuda")
    e2e = {"value": aggregate_tokens_per_s(world, spec.B, e2e_s * 1e3), "unit": UNIT,
           "h2d_bytes_per_step": int(x_host.numel() * x_host.element_size()),
           "d2h_bytes_per_step": int(y_host.numel() * y_host.element_size()), "steps": e2e_steps}

    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    # roofline of the dominant kernel
    peaks, peaks_src = load_peaks()
    plan = binding.tsvd_plan(layer.handle, spec.B, binding.DTYPES[spec.x_dtype], flags)
    dom = int(np.argmax(stage_ms))
    dom_ms = stage_ms[dom] / max(1, stage_n[dom])
    pad = lambda v: (v + 127) // 128 * 128
    if dom in (1, 3) and plan["path"] == "index":
        # an index-list stage streams its row pointers and 16-bit entries once
        v_bytes, u_bytes = binding.tsvd_index_bytes(layer.handle)
        byts = float(v_bytes if dom == 1 else u_bytes)
        achieved = byts / (dom_ms * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": binding.STAGE_NAMES[dom] + "_index", "achieved": achieved,
                    "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                    "traffic": None, "peak_source": f"{peaks_src} (of measured)", "bytes_per_launch": byts,
                    "step_hbm_gbs": (v_bytes + u_bytes) / (ms_per_step * 1e-3) / 1e9}
        roofline["step_hbm_frac"] = roofline["step_hbm_gbs"] / peaks["hbm_gbs"]
    elif dom in (1, 3) and plan["path"] == "decode":
        # a decode stage streams its packed matrix once: 2 bits per entry of the padded matrix
        rows, contr = ((pad(spec.K), pad(spec.N)) if dom == 1 else (pad(spec.M), pad(spec.K)))
        byts = rows * contr / 4.0
        achieved = byts / (dom_ms * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": binding.STAGE_NAMES[dom], "achieved": achieved,
                    "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                    "traffic": recorded_traffic(spec.name, binding.STAGE_NAMES[dom]),
                    "peak_source": f"{peaks_src} (of measured)", "bytes_per_launch": byts}
    elif dom in (1, 3):
        rows, contr = ((pad(spec.K), pad(spec.N)) if dom == 1 else (pad(spec.M), pad(spec.K)))
        digits = max(1, plan["digits_x"] if dom == 1 else plan["digits_t"])
        # executed dense operations of that launch: 2 * rows * contraction * tokens * digits
        ops = 2.0 * rows * contr * spec.B * digits
        if plan["path"] == "tensor":
            peak, peak_note = peaks["bf16_tflops"] * INT8_OVER_BF16, "int8 = measured bf16 burst x 2 (nominal ratio)"
        else:
            peak, peak_note = peaks["bf16_tflops"], "measured bf16 burst"
        achieved = ops / (dom_ms * 1e-3) / 1e12
        roofline = {"bound": "tensor", "kernel": binding.STAGE_NAMES[dom], "achieved": achieved, "peak": peak,
                    "unit": "TFLOP/s", "frac": achieved / peak,
                    "traffic": recorded_traffic(spec.name, binding.STAGE_NAMES[dom]),
                    "peak_source": f"{peak_note}; {peaks_src} (of measured)", "ops_per_launch": ops,
                    "digits": digits}
    else:
        # a digit-conversion pass dominates: it is bound by HBM traffic (read values, write digits)
        elems = spec.B * (pad(spec.N) if dom == 0 else pad(spec.K))
        in_bytes = {"f32": 4, "bf16": 2, "i8": 1}[spec.x_dtype] if dom == 0 else 4
        nd = plan["digits_x"] if dom == 0 else plan["digits_t"]
        byts = float(elems) * (in_bytes + nd)
        achieved = byts / (dom_ms * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": binding.STAGE_NAMES[dom], "achieved": achieved,
                    "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                    "traffic": None, "peak_source": f"{peaks_src} (of measured)", "bytes_per_launch": byts}
    roofline["ms_per_launch"] = dom_ms
    roofline["stage_ms_per_step"] = {n: m / args.steps for n, m in zip(binding.STAGE_NAMES, stage_ms)}
    roofline["timing"] = ("second pass of the same steps with a CUDA-event pair around each kernel on its stream; "
                          "a pair includes the launch latency, so achieved is a lower bound; ms_per_step of that pass: "
                          f"{sum(prof_step_ms) / args.steps:.4f}")
    roofline["plan"] = plan
    # whole-step tensor figure: all executed tensor operations over the whole step time
    if plan["path"] == "decode":
        # whole-step figure: all packed bytes over the graph-timed step (both launches, no event pairs)
        roofline["step_hbm_gbs"] = info["packed_bytes"] / (ms_per_step * 1e-3) / 1e9
        roofline["step_hbm_frac"] = roofline["step_hbm_gbs"] / peaks["hbm_gbs"]
    if plan["path"] == "tensor":
        all_ops = 2.0 * spec.B * (pad(spec.K) * pad(spec.N) * plan["digits_x"] + pad(spec.M) * pad(spec.K) * plan["digits_t"])
        roofline["step_tensor_frac"] = all_ops / (ms_per_step * 1e-3) / 1e12 / (peaks["bf16_tflops"] * INT8_OVER_BF16)

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "int64" if plan["path"] == "index" else "int32" if plan["path"] in ("tensor", "decode") else {"f32": "f32", "bf16": "f32", "i8": "int32"}[spec.x_dtype],
            "data": "synthetic",
            "config": workload_config(spec, l2_note),
            "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "clocks": clocks,
            "packed_bytes": info["packed_bytes"],
            "algorithmic_adds_per_token": info["density_u"] * spec.M * spec.K + info["density_v"] * spec.K * spec.N,
            "path": args.path}
    if world == 1 and not args.no_cpu_baseline:
        y_gpu = y.float().double().cpu().numpy()
        cb, parity = cpu_baseline(spec, U, S, V, x_np, y_gpu=y_gpu)
        line["cpu_baseline"] = cb
        line["parity_on_cpu_sample"] = parity
    print(json.dumps(line), flush=True)
    for extra in layers:
        extra.close()
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
