#!/usr/bin/env python
"""Benchmark of the TSVD linear map y = U(diag(S)(V x)) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config cfg4]

One step = one full forward (V-stage, S scale, U-stage) over one batch of B synthetic tokens.
Prints ONE JSON line.  `value` is tokens/s with inputs resident in HBM: the K steps are captured
in one CUDA graph, the graph is replayed `--repeats` times between CUDA events, and the median
replay is reported (with the fastest and slowest).  `e2e` is the same through the host-buffer
entry point with the copies inside the timed region.  `roofline` describes the dominant kernel,
whose duration is taken inside the graph from time stamps the kernels write themselves.
`sustained` repeats the replays back to back for more than a second with the SM clock sampled.
`per_config` carries the same figures, and a parity check against the CPU checker on a bounded
token sample, for every workload of gen.CONFIGS.  `cpu_baseline` is the CPU checker timed on
the host cores.  With N > 1 (torchrun) every rank runs its own replica on its own tokens (weak
scaling, no data-path collective); the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import datetime
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
# measured on this machine's B200s (copy bandwidth, cuBLAS bf16 burst / sustained); used when
# MEASURED_PEAKS.json is not next to this file
PEAKS_COPY = {"hbm_gbs": 6471.4, "bf16_tflops": 1711.9, "bf16_tflops_sustained": 1428.0}
INT8_OVER_BF16 = 2.0          # nominal dense tensor ratio (4.5 / 2.25 PFLOP/s)
INT8_MAC_PER_CLK_PER_SM = 8192  # tcgen05 kind::i8: the hardware rate the clock-derived peak uses
HEADLINE = "cfg4"             # the largest single-GPU workload
ALL_CONFIGS = ("cfg1", "cfg2", "cfg3_b1", "cfg3_b4", "cfg3_b16", "cfg4", "cfg5_d05", "cfg5_d20", "cfg5_d50")
SUSTAINED = ("cfg2", "cfg4")
# A layer with the structure the paper's converted layers have, for which the container holds no
# trained weights: a Laplace matrix of the shape of the 192 -> 768 linear layer of the supplement's
# architecture listing (rank 763 there), taken through Algorithm 2 at theta = 0.576 to rank 768.  Rows
# of V and columns of U are ternarised singular vectors, S comes from Eq. 4's pseudo-inverse.
PAPER_LAYER = {"M": 768, "N": 192, "K": 768, "q": 32, "theta": 0.576, "seed": 6}


def paper_shaped_layer():
    """(U, V, S, info) by the library's own direct transition on the device."""
    import torch
    from paper_2308_07641_b200 import transition
    W = gen.laplace_matrix(PAPER_LAYER["seed"], PAPER_LAYER["M"], PAPER_LAYER["N"])
    t0 = time.perf_counter()
    out = transition.direct_transition(torch.from_numpy(W).cuda(), PAPER_LAYER["theta"], q=PAPER_LAYER["q"],
                                       max_rank=PAPER_LAYER["K"])
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    U, V, S = out.U.cpu().numpy(), out.V.cpu().numpy(), out.S.cpu().numpy()
    row_nnz_v = np.count_nonzero(V, axis=1) / V.shape[1]
    info = {"source": "Laplace [768,192] through Algorithm 2 (theta 0.576, q 32) on the device", "seconds": dt,
            "nonzero_rate": out.nonzero_rate, "rel_residual_fro": out.residual_fro[-1] / out.residual_fro[0],
            "v_row_nonzero_rate_min_max": [float(row_nnz_v.min()), float(row_nnz_v.max())],
            "s_negative_share": float((S < 0).mean())}
    return U, V, S, info


def time_calls(fn, iters=20, warm=3):
    """Median of `iters` CUDA-event timings of fn() on the current stream, in microseconds."""
    import torch
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    ts = []
    for _ in range(iters):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        ts.append(1e3 * e0.elapsed_time(e1))
    return float(np.median(ts))


def measure_ternarize(n_vec=4096, length=4096, theta=0.576):
    """Algorithm 1 on the device (one call ternarises n_vec vectors), checked on a few vectors."""
    import torch
    from paper_2308_07641_b200 import binding
    from oracle import transition as otr
    x = gen.rng.normal(4242, 1, n_vec * length).reshape(n_vec, length).astype(np.float32)
    xd = torch.from_numpy(x).cuda()
    t = torch.empty((n_vec, length), dtype=torch.int8, device="cuda")
    nnz = torch.empty((n_vec,), dtype=torch.int32, device="cuda")
    call = lambda: binding.tsvd_ternarize(xd.data_ptr(), n_vec, length, length, theta, t.data_ptr(), length, nnz.data_ptr())
    us = time_calls(call)
    th = t.cpu().numpy()
    bad = 0
    for v in (0, n_vec // 2, n_vec - 1):
        bad += int(not np.array_equal(th[v], otr.ternarize(x[v].astype(np.float64), theta)))
    return {"us_per_call": us, "vectors_per_s": n_vec / (us * 1e-6), "n_vec": n_vec, "length": length, "theta": theta,
            "nonzero_rate": float(np.count_nonzero(th)) / th.size,
            "timing": "median of 20 calls, CUDA events on the launching stream",
            "parity": {"vectors": 3, "mismatching_vectors": bad, "rule": "entry for entry equal to the checker"}}


def measure_conv(n_img=8, H=56, W=56, C=128, K=256, form=0):
    """A 3x3 convolution layer in TSVD form (Eq. 5, form 0: V(.) a [3,3] convolution, U(.) a [1,1] one) on
    bf16 NHWC images; parity on the first image against the checker."""
    import torch
    from paper_2308_07641_b200.conv import TSVDConv2d
    from oracle import conv as oconv
    g = np.random.default_rng(77)
    U = (g.random((C, K)) < 0.28).astype(np.int8) * g.choice(np.array([-1, 1], np.int8), (C, K))
    V = (g.random((K, C * 9)) < 0.28).astype(np.int8) * g.choice(np.array([-1, 1], np.int8), (K, C * 9))
    S = np.exp(0.5 * g.standard_normal(K)).astype(np.float32) / 50.0
    x = g.standard_normal((n_img, H, W, C)).astype(np.float32)
    xd = torch.from_numpy(x).cuda().to(torch.bfloat16).contiguous()
    layer = TSVDConv2d(U, S, V, form, C, C, 3, 3, stride=(1, 1), padding=(1, 1))
    try:
        for _ in range(3):
            layer.forward(xd)
        torch.cuda.synchronize()
        graph, side, reps = torch.cuda.CUDAGraph(), torch.cuda.Stream(), 5
        with torch.cuda.stream(side):
            layer.forward(xd)
            torch.cuda.synchronize()
            with torch.cuda.graph(graph, stream=side):
                for _ in range(reps):
                    layer.forward(xd)
        us = time_calls(graph.replay, iters=10) / reps
        y = layer.forward(xd[:1].contiguous()).double().cpu().numpy()
        ref = oconv.conv2d_tsvd(xd[:1].float().double().cpu().numpy(), U, S, V, form, C, C, 3, 3, (1, 1), (1, 1), (1, 1))
        err = np.abs(y - ref)
        status = layer.status()
    finally:
        layer.close()
    pixels = n_img * H * W
    return {"us_per_forward": us, "pixels_per_s": pixels / (us * 1e-6), "images": n_img, "H": H, "W": W,
            "C_in": C, "C_out": C, "kernel": [3, 3], "form": form, "rank": K, "x_dtype": "bf16",
            "timing": "median of 10 replays of a CUDA graph of 5 forwards (patch gather, V-stage, U-stage), CUDA events",
            "parity": {"pixels": H * W, "max_err_over_max_ref": float(err.max() / np.abs(ref).max()),
                       "rule": "max|y-ref| <= 1e-5 max|ref| (float32 outputs)"},
            "status_word": status}


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
    """nvidia-smi clock / throttle-reason sampler; `window(t0, t1)` summarises the samples whose
    own time stamp lies inside a wall-clock interval (the timed region)."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None
        self.rows = []

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.gpu)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        try:
            for line in open(self.path):
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    row = (ts, float(parts[1]), float(parts[2]), float(parts[3]),
                           [n for n, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                               "sw_power_cap"), parts[5:9]) if v.lower().startswith("active")])
                except ValueError:
                    continue
                self.rows.append(row)
        finally:
            try:
                os.unlink(self.path)
            except OSError:
                pass
        self.proc = None

    def window(self, t0, t1):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "power_w_max": None}
        rows = [r for r in self.rows if t0 <= r[0] <= t1]
        if not rows and self.rows:      # a region shorter than the sampling period: the nearest sample
            rows = sorted(self.rows, key=lambda r: abs(r[0] - 0.5 * (t0 + t1)))[:1]
            out["note"] = "no sample fell inside the region; nearest sample reported"
        if rows:
            out.update(sm_mhz=statistics.median(r[1] for r in rows), sm_max_mhz=max(r[2] for r in rows),
                       samples=len(rows), power_w_max=max(r[3] for r in rows),
                       reasons=sorted({n for r in rows for n in r[4]}))
        return out


def parity_against_checker(spec, U, S, V, x_np, y_gpu64, tokens):
    """The GPU output of the listed tokens against the CPU checker, at the stated tolerances."""
    import oracle
    idx = np.asarray(tokens)
    ref = oracle.forward(U, S, V, gen.widen_x(x_np[idx], spec.x_dtype))
    err = np.abs(y_gpu64[idx] - ref.y)
    if spec.x_dtype == "bf16":
        tol = 1e-2 * np.abs(ref.y) + 1e-3
        return {"tokens": int(idx.size), "violations": int((err > tol).sum()),
                "worst_err_over_tol": float((err / tol).max()), "rule": "|y-ref| <= 1e-2|ref| + 1e-3 per element"}
    scale = float(np.abs(ref.y).max())
    return {"tokens": int(idx.size), "max_err_over_max_ref": float(err.max() / scale) if scale else float(err.max()),
            "violations": int(err.max() > 1e-5 * scale), "rule": "max|y-ref| <= 1e-5 max|ref|"}


def sample_tokens(B):
    """All tokens of a small batch; else the first and last ones and the tile edges at 48 and 64."""
    if B <= 16:
        return list(range(B))
    return sorted({0, 1, B // 2, B - 2, B - 1, 47, 48, 63, 64} & set(range(B)))


def cpu_baseline(spec, U, S, V, x_np, target_s=15.0):
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
    t0 = time.perf_counter(); oracle.forward(U, S, V, xs); t1 = time.perf_counter()
    return {"value": n / (t1 - t0), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {n} of {spec.B} tokens of {spec.name}, one call, {t1 - t0:.2f} s wall"}


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
            "data": "synthetic", "config": workload_config(spec),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def workload_config(spec):
    return {"workload": spec.name, "M": spec.M, "N": spec.N, "K": spec.K, "B": spec.B,
            "density": spec.density, "x_dtype": spec.x_dtype, "s_dist": spec.s_dist, "seed": spec.seed}


def pad128(v):
    return (v + 127) // 128 * 128


class Workload:
    """One packed layer (plus rotating copies and buffers larger than the L2) ready to be timed."""

    def __init__(self, spec, rank, pack_flags, flags, local_rank, weights=None):
        import torch
        from paper_2308_07641_b200 import TSVDLinear, binding, device_activations
        self.spec, self.flags, self.binding = spec, flags, binding
        self.U, self.V, self.S = weights if weights is not None else gen.make_weights(spec)
        self.x_np = gen.make_x(rank_spec(spec, rank))
        self.layer = TSVDLinear(self.U, self.S, self.V, pack_flags)
        self.info = self.layer.info
        self.layer.reserve(spec.B, spec.x_dtype)
        self.x = device_activations(self.x_np, spec.x_dtype)
        self.y = self.layer.forward(self.x, flags=flags)
        torch.cuda.synchronize()
        # Rotating input/output buffers: together larger than twice the L2, so that every step
        # streams its activations from HBM and writes its results there.
        self.l2_bytes = int(torch.cuda.get_device_properties(local_rank).L2_cache_size)
        self.pair_bytes = self.x.numel() * self.x.element_size() + self.y.numel() * self.y.element_size()
        self.n_sets = int(min(64, max(2, -(-2 * self.l2_bytes // self.pair_bytes))))
        self.xs = [self.x] + [torch.roll(self.x, i, dims=0).contiguous() for i in range(1, self.n_sets)]
        self.ys = [self.y] + [torch.empty_like(self.y) for _ in range(1, self.n_sets)]
        # When the packed weights outweigh the activations (small batches) the weights are what must
        # come from HBM: pack the same layer several times and rotate over the copies as well.
        self.n_layers = 1
        if self.info["packed_bytes"] > self.pair_bytes:
            self.n_layers = int(min(64, max(2, -(-2 * self.l2_bytes // self.info["packed_bytes"]))))
        self.layers = [self.layer] + [TSVDLinear(self.U, self.S, self.V, pack_flags) for _ in range(1, self.n_layers)]
        for extra in self.layers[1:]:
            extra.reserve(spec.B, spec.x_dtype)
        self.plan = binding.tsvd_plan(self.layer.handle, spec.B, binding.DTYPES[spec.x_dtype], flags)
        self.l2_note = (f"inputs larger than L2: {self.n_sets} rotating x/y buffer pairs "
                        f"({self.n_sets * self.pair_bytes / 1e6:.0f} MB) and {self.n_layers} packed copies of the layer "
                        f"({self.n_layers * self.info['packed_bytes'] / 1e6:.0f} MB) against {self.l2_bytes / 1e6:.0f} MB of L2")

    def step(self, i):
        self.layers[i % self.n_layers].forward(self.xs[i % self.n_sets], out=self.ys[i % self.n_sets], flags=self.flags)

    def capture(self, steps, stamps=False):
        """`steps` forwards in one CUDA graph (no host launch latency between kernels).  With
        `stamps` every kernel also writes its own begin/end time; returns (graph, launches)."""
        import torch
        b = self.binding
        for L in self.layers:
            b.tsvd_profile_enable(L.handle, 2 if stamps else 0)
        side = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        n0 = b.tsvd_launch_count()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for i in range(steps):
                    self.step(i)
        return g, b.tsvd_launch_count() - n0

    def stage_times(self):
        """Summed in-graph kernel time (ms) and launches per stage over all rotating copies."""
        b = self.binding
        ms = [0.0] * b.N_STAGES
        n = [0] * b.N_STAGES
        for L in self.layers:
            m, c = b.tsvd_profile_read(L.handle)
            ms = [a + v for a, v in zip(ms, m)]
            n = [a + v for a, v in zip(n, c)]
            b.tsvd_profile_enable(L.handle, 0)
        return ms, n

    def close(self):
        for L in self.layers:
            L.close()


def replay_times(g, repeats, barrier):
    """`repeats` replays of a captured graph, each between its own pair of CUDA events, queued back to
    back; returns the per-replay times in ms and the wall-clock interval of the region."""
    import torch
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(repeats + 1)]
    g.replay()                         # one untimed replay (graph upload)
    barrier()
    t0 = time.time()
    ev[0].record()
    for i in range(repeats):
        g.replay()
        ev[i + 1].record()
    barrier()
    t1 = time.time()
    return [ev[i].elapsed_time(ev[i + 1]) for i in range(repeats)], (t0, t1)


def roofline_of(w, peaks, peaks_src, ms_per_step, stage_ms, stage_n, sm_mhz):
    """The dominant kernel of one workload against the roofline that bounds it."""
    b, spec, plan, info = w.binding, w.spec, w.plan, w.info
    per_launch = [m / c if c else 0.0 for m, c in zip(stage_ms, stage_n)]
    dom = int(np.argmax(per_launch))
    dom_ms = per_launch[dom]
    name = b.STAGE_NAMES[dom]
    rows, contr = (pad128(spec.K), pad128(spec.N)) if dom in (0, 1) else (pad128(spec.M), pad128(spec.K))
    out = {"kernel": name, "ms_per_launch": dom_ms, "plan": plan,
           "stage_us_per_launch": {n: 1e3 * v for n, v in zip(b.STAGE_NAMES, per_launch)},
           "timing": "time stamps written by the kernels inside a captured graph of the same steps "
                     "(begin: the first CTA once its wait for the previous kernel has ended; end: the last warp)"}
    if dom_ms <= 0:
        out.update(bound="hbm", achieved=None, peak=peaks["hbm_gbs"], unit="GB/s", frac=None, traffic=None)
        return out
    if dom in (1, 3) and plan["path"] in ("decode", "index"):
        if plan["path"] == "index":
            v_bytes, u_bytes = b.tsvd_index_bytes(w.layer.handle)
            byts, all_bytes = float(v_bytes if dom == 1 else u_bytes), float(v_bytes + u_bytes)
        else:
            byts, all_bytes = rows * contr / 4.0, float(info["packed_bytes"])   # 2 bits per padded entry
        achieved = byts / (dom_ms * 1e-3) / 1e9
        out.update(bound="hbm", achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s", frac=achieved / peaks["hbm_gbs"],
                   traffic=recorded_traffic(spec.name, name), bytes_per_launch=byts,
                   peak_source=f"{peaks_src} (of measured)",
                   step_hbm_gbs=all_bytes / (ms_per_step * 1e-3) / 1e9)
        out["step_hbm_frac"] = out["step_hbm_gbs"] / peaks["hbm_gbs"]
    elif dom in (1, 3):
        digits = max(1, plan["digits_x"] if dom == 1 else plan["digits_t"])
        ops = 2.0 * rows * contr * spec.B * digits        # executed dense operations of that launch
        useful = 2.0 * rows * contr * spec.B              # the same contraction without the digit split
        if plan["path"] == "tensor":
            peak, note = peaks["bf16_tflops"] * INT8_OVER_BF16, "int8 = measured bf16 burst x 2 (nominal ratio)"
        else:
            peak, note = peaks["bf16_tflops"], "measured bf16 burst"
        achieved = ops / (dom_ms * 1e-3) / 1e12
        out.update(bound="tensor", achieved=achieved, peak=peak, unit="TFLOP/s", frac=achieved / peak,
                   traffic=recorded_traffic(spec.name, name), ops_per_launch=ops, digits=digits,
                   peak_source=f"{note}; {peaks_src} (of measured)", useful_frac=useful / (dom_ms * 1e-3) / 1e12 / peak)
        if plan["path"] == "tensor" and sm_mhz:
            clock_peak = 148 * INT8_MAC_PER_CLK_PER_SM * 2 * sm_mhz * 1e6 / 1e12
            out["clock_peak"] = {"tops": clock_peak, "frac": achieved / clock_peak,
                                 "useful_frac": out["useful_frac"] * peak / clock_peak,
                                 "how": f"148 SMs x {INT8_MAC_PER_CLK_PER_SM} int8 MAC/clk x 2 x {sm_mhz:.0f} MHz "
                                        "(median sampled SM clock of the timed region)"}
    else:
        in_bytes = {"f32": 4, "bf16": 2, "i8": 1}[spec.x_dtype] if dom == 0 else 4
        nd = plan["digits_x"] if dom == 0 else plan["digits_t"]
        byts = float(spec.B * contr) * (in_bytes + nd)     # values read, digits written
        achieved = byts / (dom_ms * 1e-3) / 1e9
        out.update(bound="hbm", achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s", frac=achieved / peaks["hbm_gbs"],
                   traffic=None, bytes_per_launch=byts, peak_source=f"{peaks_src} (of measured)")
    if plan["path"] == "tensor":
        all_ops = 2.0 * spec.B * (pad128(spec.K) * pad128(spec.N) * plan["digits_x"] + pad128(spec.M) * pad128(spec.K) * plan["digits_t"])
        single = 2.0 * spec.B * (pad128(spec.K) * pad128(spec.N) + pad128(spec.M) * pad128(spec.K))
        int8_peak = peaks["bf16_tflops"] * INT8_OVER_BF16
        out["step_tensor_frac"] = all_ops / (ms_per_step * 1e-3) / 1e12 / int8_peak
        out["step_useful_frac_of_bf16_peak"] = single / (ms_per_step * 1e-3) / 1e12 / peaks["bf16_tflops"]
        if spec.B <= 32:
            # up to 32 tokens the tensor-core path runs one cluster kernel per stage and streaming the packed
            # codes is the other bound worth quoting
            out["step_hbm_gbs"] = float(info["packed_bytes"]) / (ms_per_step * 1e-3) / 1e9
            out["step_hbm_frac"] = out["step_hbm_gbs"] / peaks["hbm_gbs"]
    return out


def measure(w, steps, repeats, barrier, dist, world, sustained_s=0.0):
    """Median-of-replays step time of one workload and its in-graph kernel times."""
    import torch
    spec = w.spec
    g, launches = w.capture(steps)
    times, (t0, t1) = replay_times(g, repeats, barrier)
    med = max_over_ranks(dist, statistics.median(times), "cuda")
    ms_per_step = med / steps
    res = {"ms_per_step": ms_per_step, "ms_per_step_min": min(times) / steps, "ms_per_step_max": max(times) / steps,
           "tokens_per_s": aggregate_tokens_per_s(world, spec.B, ms_per_step), "launches_per_step": launches / steps,
           "launches": launches * repeats, "window": (t0, t1), "path": w.plan["path"]}
    if sustained_s > 0:
        n = max(2, int(sustained_s * 1e3 / max(med, 1e-3)) + 1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        s0 = time.time()
        a.record()
        for _ in range(n):
            g.replay()
        b.record()
        barrier()
        s1 = time.time()
        tot = max_over_ranks(dist, a.elapsed_time(b), "cuda")
        res["sustained"] = {"ms_per_step": tot / (n * steps), "seconds": tot * 1e-3, "steps": n * steps,
                            "tokens_per_s": aggregate_tokens_per_s(world, spec.B, tot / (n * steps)), "window": (s0, s1)}
    del g
    # the same steps once more with the kernels stamping their own begin and end
    g2, _ = w.capture(steps, stamps=True)
    stamp_times, _ = replay_times(g2, 2, barrier)
    stage_ms, stage_n = w.stage_times()
    del g2
    res["stage_ms"], res["stage_n"] = stage_ms, stage_n
    res["ms_per_step_with_stamps"] = statistics.median(stamp_times) / steps
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100, help="forwards per captured graph = steps of one timed region")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--repeats", type=int, default=10, help="timed replays of the graph; the median is reported")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default=HEADLINE, choices=sorted(gen.CONFIGS))
    ap.add_argument("--path", default="auto", choices=["auto", "simple", "decode", "tensor", "index"],
                    help="index = the index-list form (one to four tokens; meant for nonzero rates below 1/8)")
    ap.add_argument("--density", type=float, default=None,
                    help="override the workload's nonzero rate of U and V (the sparse sweep of the index-list form)")
    ap.add_argument("--wide-x", action="store_true", help="bf16 activations as four digits (TSVD_FLAG_WIDE_X)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="only the headline workload")
    ap.add_argument("--no-sustained", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer measurement (profiling runs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    spec = gen.CONFIGS[args.config]
    if args.density is not None:
        spec = gen.scaled(spec, name=f"{spec.name}_density{args.density:g}", density=args.density)

    if args.impl == "reference":
        run_reference(args, spec)
        return

    import torch
    from paper_2308_07641_b200 import binding, build as lib_build
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

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    flags = {"auto": 0, "simple": TSVD_FLAG_PATH_SIMPLE, "decode": TSVD_FLAG_PATH_DECODE,
             "tensor": TSVD_FLAG_PATH_TENSOR, "index": binding.TSVD_FLAG_PATH_INDEX}[args.path]
    if args.wide_x:
        flags |= binding.TSVD_FLAG_WIDE_X
    pack_flags = binding.TSVD_PACK_INDEX_LISTS if args.path == "index" else 0
    peaks, peaks_src = load_peaks()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.5)

    # ---- the headline workload ----
    w = Workload(spec, rank, pack_flags, flags, local_rank)
    for i in range(args.warmup):
        w.step(i)
    barrier()
    want_sustained = (not args.no_sustained) and spec.name in SUSTAINED
    head = measure(w, args.steps, args.repeats, barrier, dist, world, sustained_s=1.5 if want_sustained else 0.0)

    e2e = None
    w.layer.forward(w.x, out=w.y, flags=flags)
    torch.cuda.synchronize()
    y_gpu = w.y.float().double().cpu().numpy()
    if not args.no_e2e:
        # end to end: host buffers, copies inside the timed region
        x_host = torch.from_numpy(w.x_np.view(np.int16) if spec.x_dtype == "bf16" else w.x_np).pin_memory()
        y_bf16 = w.y.dtype == torch.bfloat16
        y_host = torch.empty((spec.B, spec.M), dtype=torch.int16 if y_bf16 else torch.float32).pin_memory()
        dt_code = binding.DTYPES[spec.x_dtype]
        e2e_steps = max(3, min(args.steps, 20))
        for _ in range(2):
            binding.tsvd_forward_host(w.layer.handle, x_host.data_ptr(), y_host.data_ptr(), spec.B, dt_code, flags)
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            binding.tsvd_forward_host(w.layer.handle, x_host.data_ptr(), y_host.data_ptr(), spec.B, dt_code, flags)
        torch.cuda.synchronize()
        e2e_s = (time.perf_counter() - t0) / e2e_steps
        e2e_s = max_over_ranks(dist, e2e_s, "cuda")
        e2e = {"value": aggregate_tokens_per_s(world, spec.B, e2e_s * 1e3), "unit": UNIT,
               "h2d_bytes_per_step": int(x_host.numel() * x_host.element_size()),
               "d2h_bytes_per_step": int(y_host.numel() * y_host.element_size()), "steps": e2e_steps,
               "ms_per_step": e2e_s * 1e3}
        y_e2e = (y_host.view(torch.bfloat16).float() if y_bf16 else y_host).double().numpy()
        w.layer.forward(w.x, out=w.y, flags=flags)
        torch.cuda.synchronize()
        y_gpu = w.y.float().double().cpu().numpy()
        e2e["matches_device_path"] = bool(np.array_equal(y_e2e, y_gpu))

    if rank != 0:
        w.close()
        if dist:
            dist.destroy_process_group()
        return

    # ---- every workload in the same line (one GPU only) ----
    per_config = None
    extra = {}
    if world == 1 and not args.no_per_config:
        per_config = {}
        for name in ALL_CONFIGS:
            if name == spec.name and args.path == "auto" and not args.wide_x:
                continue                  # the headline is filled in below
            s2 = gen.CONFIGS[name]
            w2 = Workload(s2, 0, 0, 0, local_rank)
            for i in range(3):
                w2.step(i)
            barrier()
            r2 = measure(w2, args.steps, args.repeats, barrier, None, 1,
                         sustained_s=1.5 if (not args.no_sustained and name in SUSTAINED) else 0.0)
            w2.layer.forward(w2.x, out=w2.y)
            torch.cuda.synchronize()
            y2 = w2.y.float().double().cpu().numpy()
            r2["parity"] = parity_against_checker(s2, w2.U, w2.S, w2.V, w2.x_np, y2, sample_tokens(s2.B))
            r2["status_word"] = binding.tsvd_last_status(w2.layer.handle)
            extra[name] = (w2, r2)
            # keep only what the summary needs; free the device memory before the next workload
            w2.xs, w2.ys, w2.x, w2.y = None, None, None, None
            for L in w2.layers[1:]:
                L.close()
            w2.layers = w2.layers[:1]
            torch.cuda.empty_cache()
        # the paper-shaped layer: prefill-sized and single-token batches
        try:
            Up, Vp, Sp, pinfo = paper_shaped_layer()
            for name, B in (("paper_layer_b3136", 3136), ("paper_layer_b1", 1)):
                s2 = gen.CaseSpec(name, M=PAPER_LAYER["M"], N=PAPER_LAYER["N"], K=PAPER_LAYER["K"], B=B,
                                  density=pinfo["nonzero_rate"], x_dtype="f32", s_dist="eq4", s_sorted=False, seed=60)
                w2 = Workload(s2, 0, 0, 0, local_rank, weights=(Up, Vp, Sp))
                for i in range(3):
                    w2.step(i)
                barrier()
                r2 = measure(w2, args.steps, args.repeats, barrier, None, 1)
                w2.layer.forward(w2.x, out=w2.y)
                torch.cuda.synchronize()
                r2["parity"] = parity_against_checker(s2, Up, Sp, Vp, w2.x_np, w2.y.float().double().cpu().numpy(),
                                                      sample_tokens(B))
                r2["status_word"] = binding.tsvd_last_status(w2.layer.handle)
                r2["operands"] = pinfo
                extra[name] = (w2, r2)
                w2.xs, w2.ys, w2.x, w2.y = None, None, None, None
                for L in w2.layers[1:]:
                    L.close()
                w2.layers = w2.layers[:1]
                torch.cuda.empty_cache()
        except Exception as exc:       # the decomposition is not the benchmark: report and go on
            extra_error = f"paper-shaped layer skipped: {exc!r}"
            per_config["paper_layer"] = extra_error
        # the other entry points that run kernels of their own: Algorithm 1 and a convolution form
        for name, fn in (("ternarize_4096x4096", measure_ternarize), ("conv3x3_c128_k256_8x56x56", measure_conv)):
            try:
                per_config[name] = fn()
            except Exception as exc:
                per_config[name] = f"skipped: {exc!r}"
            torch.cuda.empty_cache()
    sampler.stop()

    def summarise(wk, r):
        clocks = sampler.window(*r["window"])
        roof = roofline_of(wk, peaks, peaks_src, r["ms_per_step"], r["stage_ms"], r["stage_n"], clocks["sm_mhz"])
        out = {"us_per_step": 1e3 * r["ms_per_step"], "us_per_step_min": 1e3 * r["ms_per_step_min"],
               "us_per_step_max": 1e3 * r["ms_per_step_max"], "tokens_per_s": r["tokens_per_s"], "path": r["path"],
               "launches_per_step": r["launches_per_step"], "roofline": roof, "clocks": clocks,
               "us_per_step_with_stamps": 1e3 * r["ms_per_step_with_stamps"],
               "ms_x_mhz": r["ms_per_step"] * (clocks["sm_mhz"] or 0.0)}
        if "sustained" in r:
            s = dict(r["sustained"])
            sc = sampler.window(*s.pop("window"))
            s["clocks"] = sc
            s["ms_x_mhz"] = s["ms_per_step"] * (sc["sm_mhz"] or 0.0)
            if wk.plan["path"] == "tensor":
                all_ops = 2.0 * wk.spec.B * (pad128(wk.spec.K) * pad128(wk.spec.N) * wk.plan["digits_x"] +
                                             pad128(wk.spec.M) * pad128(wk.spec.K) * wk.plan["digits_t"])
                s["step_tensor_frac_of_sustained_peak"] = (all_ops / (s["ms_per_step"] * 1e-3) / 1e12 /
                                                           (peaks["bf16_tflops_sustained"] * INT8_OVER_BF16))
            out["sustained"] = s
        if "parity" in r:
            out["parity"] = r["parity"]
            out["status_word"] = r["status_word"]
        if "operands" in r:
            out["operands"] = r["operands"]
        return out

    head_sum = summarise(w, head)
    head_sum["parity"] = parity_against_checker(spec, w.U, w.S, w.V, w.x_np, y_gpu, sample_tokens(spec.B))
    head_sum["status_word"] = binding.tsvd_last_status(w.layer.handle)
    if per_config is not None:
        for name in ALL_CONFIGS + ("paper_layer_b3136", "paper_layer_b1"):
            if name in extra:
                w2, r2 = extra[name]
                per_config[name] = summarise(w2, r2)
                per_config[name]["roofline"].pop("timing", None)
                w2.close()
            elif name in ALL_CONFIGS:
                per_config[name] = "the headline of this line"

    plan = w.plan
    line = {"metric": METRIC, "value": head["tokens_per_s"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "int64" if plan["path"] == "index" else "int32" if plan["path"] in ("tensor", "decode") else {"f32": "f32", "bf16": "f32", "i8": "int32"}[spec.x_dtype],
            "data": "synthetic",
            "config": dict(workload_config(spec), l2=w.l2_note + f"; the {args.steps} steps are one CUDA graph"),
            "timing": {"repeats": args.repeats, "statistic": "median over the replays of the graph",
                       "ms_per_step_min": head["ms_per_step_min"], "ms_per_step_max": head["ms_per_step_max"],
                       "ms_per_step_with_stamps": head["ms_per_step_with_stamps"],
                       "ms_x_mhz": head_sum["ms_x_mhz"],
                       "kind": "burst: one replay lasts milliseconds; `sustained` holds the same replays back to back for seconds"},
            "e2e": e2e, "gpu_launches": int(head["launches"]), "roofline": head_sum["roofline"], "clocks": head_sum["clocks"],
            "packed_bytes": w.info["packed_bytes"],
            "algorithmic_adds_per_token": w.info["density_u"] * spec.M * spec.K + w.info["density_v"] * spec.K * spec.N,
            "path": args.path, "parity_on_cpu_sample": head_sum["parity"], "status_word": head_sum["status_word"]}
    if "sustained" in head_sum:
        line["sustained"] = head_sum["sustained"]
    if per_config is not None:
        line["per_config"] = per_config
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(spec, w.U, w.S, w.V, w.x_np)
    print(json.dumps(line), flush=True)
    w.close()
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
