#!/usr/bin/env python
"""Benchmark of the multi-tenant LoRA linear layer (forward + backward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3] [--impl reference]

One "step" is one pass of the whole hot path over one batch of synthetic input: index build, shrink,
base GEMM with the fused LoRA expand (forward), then g-shrink, dx GEMM with its fused expand and the dA/dB
reductions (backward).  The default workload is the training-shaped configuration (base W 4096x11008,
10 tenants of rank 32, 16384 tokens in lognormal per-tenant segments), the only single-projection
configuration that exercises every step; --workload cfg2 times the decode-shaped forward, cfg4 the
heterogeneous one, cfg5 the 7-projection decoder-layer set.

Prints ONE JSON line (rank 0).  `value` is whole-job tokens/s with inputs resident in HBM; `e2e` is the same
metric through the same calls with HOST inputs and outputs (pinned buffers, copies inside the timed region).
`--impl reference` times the CPU oracle on the host cores instead (a deliberately plain program).
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2605_08527_b200 import workloads as wl  # noqa: E402

METRIC = "multi-LoRA layer tokens/s (fwd+bwd)"
NOMINAL = {"bf16_tflops": 2250.0, "hbm_gbs": 8000.0}
FALLBACK = {"bf16_tflops": 1590.0, "hbm_gbs": 6650.0}


def profile_traffic(workload):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the workload's dominant kernel, from the committed ncu
    summaries under profiles/ (a line `bench-traffic <workload> <bytes per launch> <source file> <sha256[:16] of that
    file when the counters were taken>`).  None, with the reason, when no capture exists or the kernel's source has
    changed since."""
    import glob
    import hashlib
    for path in sorted(glob.glob(os.path.join(ROOT, "profiles", "*.txt"))):
        for line in open(path):
            f = line.split()
            if len(f) >= 5 and f[0] == "bench-traffic" and f[1] == workload:
                src = os.path.join(ROOT, f[3])
                if not os.path.exists(src):
                    return None, f"{os.path.basename(path)}: {f[3]} no longer exists"
                sha = hashlib.sha256(open(src, "rb").read()).hexdigest()[:16]
                if sha != f[4]:
                    return None, f"{os.path.basename(path)}: {f[3]} has changed since the counters were taken"
                return float(f[2]), os.path.basename(path)
    return None, "no ncu capture of this workload under profiles/"


CFG_OF = {"cfg1": 1, "cfg2": 2, "cfg3": 3, "cfg4": 4, "cfg5": 5}
CFG_DESC = {
    "cfg1": "tiny: W 512x512, 4 tenants r=8, 256 tokens, fwd+bwd",
    "cfg2": "rollout-decode shaped: W 4096x4096, 32 tenants r=16, 256 unsorted decode tokens, fwd only",
    "cfg3": "training shaped: W 4096x11008, 10 tenants r=32, 16384 tokens in lognormal segments, fwd+bwd",
    "cfg4": "heterogeneous tenants: W 5120x5120, 32 tenants r in {8,16,32,64}, 8192 Zipf tokens, fwd+bwd",
    "cfg5": "7B decoder-layer adapter set: 7 projections, 32 tenants r=16, 4096 training + 256 decode tokens",
}
SWEEPS = {
    # batch sizes x tenants of the rollout phases (the paper varies the number of concurrent tasks from 1 to 32)
    "decode": [f"decode-{T}-{n}" for T in (32, 64, 128, 256, 512, 1024) for n in (1, 8, 32)],
    "prefill": [f"prefill-{T}-{n}" for T in (8192, 16384, 32768) for n in (1, 8, 32)],
    # projections that share their input, fused into one call against one call each, on a decode batch
    "fused": [f"{k}-{T}-32" for T in (64, 256) for k in ("qkvseg", "qkv", "qkvsep", "gateupseg", "gateup", "gateupsep")],
    # decode batches over the projections of decoder layers of several sizes (hidden x intermediate of 7-8B, 14B and 32B
    # class models; q / o, gate / up and down shapes), 256 tokens and smaller batches
    "shapes": [f"decode{K}x{N}-{T}-32" for K, N, T in (
        (4096, 4096, 256), (4096, 12288, 256), (12288, 4096, 256), (4096, 14336, 256), (3584, 18944, 256),
        (5120, 5120, 256), (5120, 17408, 256), (17408, 5120, 256), (5120, 25600, 256), (25600, 5120, 256),
        (5120, 17408, 128), (5120, 17408, 64),
        # batches of 64 tokens: the kernels run with 64-token tiles
        (4096, 12288, 64), (12288, 4096, 64), (3584, 18944, 64), (17408, 5120, 64), (5120, 25600, 64), (5120, 34816, 32))],
}


def workload_desc(name):
    if name in CFG_DESC:
        return CFG_DESC[name]
    if name in wl.VARIANTS:
        return wl.VARIANTS[name]
    kind, T, n = name.split("-")
    if kind in ("qkv", "qkvsep", "qkvseg", "gateup", "gateupsep", "gateupseg"):
        shape = "q, k, v (4096x4096 each)" if kind.startswith("qkv") else "gate, up (4096x11008 each)"
        how = "one call each" if kind.endswith("sep") else \
            "one pool over the projections (B side by side), one call" if kind.endswith("seg") else \
            "fused into one projection (block-diagonal B), one call"
        return f"{shape}, {how}; {n} tenants r=16 per projection, {T} decode tokens, fwd only"
    what = "decode tokens (one per sequence, tenants uniform and unsorted)" if kind.startswith("decode") else \
        "prompt tokens in whole-prompt lognormal segments"
    shape = kind[6:] if kind.startswith("decode") and kind != "decode" else "4096x4096"
    return f"{kind} sweep point: W {shape}, {n} tenants r=16, {T} {what}, fwd only"


def run_sweep(args):
    """One bench.py process per sweep point (no CPU baseline, no end-to-end leg); prints their JSON lines."""
    import subprocess
    for name in SWEEPS[args.sweep]:
        cmd = [sys.executable, os.path.abspath(__file__), "--workload", name, "--steps", str(args.steps), "--warmup",
               str(args.warmup), "--no-cpu-baseline", "--e2e-steps", "0", "--flags", str(args.flags)] + (["--overlap"] if args.overlap else [])
        r = subprocess.run(cmd, capture_output=True, text=True)
        lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
        if r.returncode != 0 or not lines:
            print(json.dumps({"sweep": args.sweep, "workload": name, "failed": r.stderr.strip().splitlines()[-1:] }))
            continue
        d = json.loads(lines[-1])
        d["sweep"] = args.sweep
        print(json.dumps(d), flush=True)


def run_adamw(args, n_tenants):
    """Times the fused policy update + commit (marlaas_adapter_pool_adamw_commit) for n tenants of rank 16 on a
    4096 x 4096 projection: one call = one optimizer step of every tenant.  HBM-bound: 30 bytes per adapter element."""
    import torch
    from paper_2605_08527_b200 import binding as B
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the layer has no CPU path")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    K = N = 4096
    r = 16
    l2 = torch.cuda.get_device_properties(dev).L2_cache_size
    elems = n_tenants * r * (K + N)
    state_bytes = elems * 28                    # gradient, master, two moments read; master and moments written
    R = int(min(16, max(1, -(-3 * l2 // state_bytes))))
    copies = []
    for c in range(R):
        pool = B.AdapterPool(K, N, r, n_tenants, device=dev)
        st = {"pool": pool, "ids": list(range(1, n_tenants + 1))}
        gen = torch.Generator(device=dev).manual_seed(1234 + c)
        for nm, shape in (("dA", (K, r)), ("dB", (r, N)), ("A", (K, r)), ("B", (r, N))):
            st[nm] = [torch.randn(shape, generator=gen, device=dev, dtype=torch.float32) * (0.02 if nm in "AB" else 1.0)
                      for _ in range(n_tenants)]
        for nm, like in (("mA", "A"), ("vA", "A"), ("mB", "B"), ("vB", "B")):
            st[nm] = [torch.zeros_like(t) for t in st[like]]
        for i, tid in enumerate(st["ids"]):
            B.marlaas_adapter_pool_register(pool, tid, 0, r, 32.0, st["A"][i].to(torch.bfloat16), st["B"][i].to(torch.bfloat16))
        copies.append(st)

    def step(i):
        c = copies[i % R]
        B.marlaas_adapter_pool_adamw_commit(c["pool"], c["ids"], c["dA"], c["dB"], c["A"], c["B"], c["mA"], c["vA"], c["mB"],
                                            c["vB"], lr=1e-3, weight_decay=0.01, step=i + 1)

    for i in range(max(args.warmup, R)):
        step(i)
    torch.cuda.synchronize()
    # a call lasts tens of microseconds, less than Python needs to marshal its eight pointer tables: the K steps are
    # captured once into a CUDA graph (the call takes its pointers by value, so a capture can hold it) and replayed
    n0 = B.marlaas_kernel_launch_count()
    side = torch.cuda.Stream(device=dev)
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for i in range(args.steps):
                step(args.warmup + i)
    torch.cuda.current_stream().wait_stream(side)
    launches = B.marlaas_kernel_launch_count() - n0
    graph.replay()
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    reps = 20
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for a, b in evs:
        a.record()
        graph.replay()
        b.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = float(np.median([a.elapsed_time(b) for a, b in evs])) / args.steps
    peaks, peak_src = measured_peaks()
    bytes_per_step = elems * 30.0
    ach = bytes_per_step / (ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": "adapter AdamW updates + commits per second", "value": n_tenants / (ms * 1e-3), "unit": "tenant updates/s",
        "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload, "desc": f"AdamW + commit of {n_tenants} tenants, rank 16, on a 4096x4096 projection; "
                   "one call per step", "timed_as": "one CUDA graph of K steps, median of 20 replays", "l2": f"optimizer state of a step ({state_bytes / 1e6:.0f} MB) rotates over {R} copies"},
        "roofline": {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                     "traffic": None, "peak_source": f"of {peak_src}", "kernel": "k_adamw_commit",
                     "bytes_per_launch": bytes_per_step / max(launches / args.steps, 1)},
        "cpu_baseline": None, "e2e": None, "gpu_launches": int(launches), "clocks": clocks}))


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return {"bf16_tflops": float(d["bf16_tflops"]), "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    "hbm_gbs": float(d["hbm_gbs"])}, "measured"
        except Exception:
            pass
    return {"bf16_tflops": FALLBACK["bf16_tflops"], "bf16_tflops_sustained": 1400.0, "hbm_gbs": FALLBACK["hbm_gbs"]}, "fallback"


def algorithmic_work(w):
    """Flops and minimum bytes of one step (each operand touched once), per projection and summed.
    fwd: 2TKN + sum_i 2 r(K+N); bwd: 2TKN + sum_i r(4N+4K); rank padding and recomputation are not counted."""
    ts = w.tok_slot()
    out = {"fwd_flops": 0.0, "bwd_flops": 0.0, "fwd_bytes": 0.0, "bwd_bytes": 0.0, "gemm_flops": []}
    for p in w.projections:
        K, N = p.d_in, p.d_out
        np_ = len(p.parts) if p.parts else 1        # a pool over several projections holds one A per projection
        ranks = np.array([a.rank for a in p.adapters] + [0])
        r_tok = ranks[ts]
        Tb = 0 if p.dy_bits is None else p.dy_bits.shape[0]
        present = np.unique(ts[ts >= 0])
        ad_bytes = sum(2 * ranks[t] * (np_ * K + N) for t in present)
        out["fwd_flops"] += 2.0 * w.T * K * N + float(np.sum(2.0 * r_tok * (np_ * K + N)))
        out["fwd_bytes"] += 2.0 * (K * N + w.T * K + w.T * N) + ad_bytes
        out["gemm_flops"].append(2.0 * w.T * K * N + float(np.sum(2.0 * r_tok * N)))
        if Tb:
            rb = r_tok[:Tb]
            pres_b = np.unique(ts[:Tb][ts[:Tb] >= 0])
            out["bwd_flops"] += 2.0 * Tb * K * N + float(np.sum(rb * (4.0 * N + 4.0 * K)))
            out["bwd_bytes"] += 2.0 * (K * N + 2 * Tb * K + Tb * N) + sum(2 * ranks[t] * (K + N) for t in pres_b) \
                + sum(4 * ranks[t] * (K + N) for t in pres_b)
            out["gemm_flops"].append(2.0 * Tb * K * N + float(np.sum(2.0 * rb * K)))
    return out


class ClockSampler:
    """Clock / throttle-reason samples taken while the timed region runs: an NVML polling thread (a sample every 10 ms,
    no start-up delay, read-only queries), or nvidia-smi in a subprocess when the NVML bindings are missing."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc, self.path = None, None
        self.thread, self.samples, self.stop_flag = None, [], False
        self.nvml, self.handle = None, None
        try:
            import pynvml
            pynvml.nvmlInit()
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = gpu_index
            if vis:
                ids = [v.strip() for v in vis.split(",") if v.strip()]
                if gpu_index < len(ids) and ids[gpu_index].isdigit():
                    phys = int(ids[gpu_index])
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.nvml = pynvml
        except Exception:
            self.nvml = None

    def _poll(self):
        nv, h = self.nvml, self.handle
        bits = {"hw_slowdown": nv.nvmlClocksEventReasonHwSlowdown, "hw_thermal_slowdown": nv.nvmlClocksEventReasonHwThermalSlowdown,
                "sw_thermal_slowdown": nv.nvmlClocksEventReasonSwThermalSlowdown, "sw_power_cap": nv.nvmlClocksEventReasonSwPowerCap}
        while not self.stop_flag:
            try:
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(h)
                self.samples.append((float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)),
                                     float(nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)),
                                     nv.nvmlDeviceGetPowerUsage(h) / 1000.0, [k for k, b in bits.items() if r & b]))
            except Exception:
                pass
            time.sleep(0.01)

    def start(self):
        if self.nvml is not None:
            import threading
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
            return
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu_index)], stdout=f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.thread is not None:
            self.stop_flag = True
            self.thread.join(timeout=1.0)
            if not self.samples:
                return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
            sm, mx, pw = [x[0] for x in self.samples], [x[1] for x in self.samples], [x[2] for x in self.samples]
            reasons = sorted({r for x in self.samples for r in x[3]})
            return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "power_w_max": float(max(pw)),
                    "samples": len(sm), "reasons": reasons, "source": "nvml"}
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                c = [v.strip() for v in line.split(",")]
                if len(c) < 9:
                    continue
                try:
                    sm.append(float(c[1])); mx.append(float(c[2])); pw.append(float(c[3]))
                except ValueError:
                    continue
                for nm, v in zip(names, c[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(nm)
            os.unlink(self.path)
        except Exception:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "power_w_max": float(max(pw)),
                "samples": len(sm), "reasons": sorted(reasons)}


def oracle_step_sample(w, n_tok):
    """Time the oracle (as it stands) on the first n_tok tokens of every projection; returns seconds."""
    import oracle
    ts = w.tok_slot()
    total = 0.0
    for p in w.projections:
        r, s, A, Bm = oracle.adapters_of(p)
        n = min(n_tok, w.T)
        x = p.x[:n]
        t0 = time.perf_counter()
        oracle.forward(x, p.W, r, s, A, Bm, ts[:n])
        if p.dy_bits is not None:
            nb = min(n, p.dy_bits.shape[0])
            dy = p.dy[:nb]
            oracle.backward_dx(dy, p.W, r, s, A, Bm, ts[:nb])
            oracle.backward_dAdB(x[:nb], dy, r, s, A, Bm, ts[:nb])
        total += time.perf_counter() - t0
    return total


def max_over_ranks(ms: float, dist, device) -> float:
    """The slowest rank's time: every multi-GPU number is the maximum over ranks (replicas finish together or not at all)."""
    if dist is None:
        return float(ms)
    import torch
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tokens_per_s(tokens_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job throughput of `world` independent replicas (weak scaling: per-rank work is fixed)."""
    return tokens_per_rank * world / (ms_per_step * 1e-3)


def run_reference(args, rank, world):
    """--impl reference: the CPU oracle on the host cores, a bounded sample of the workload per step."""
    if rank != 0:
        return
    import oracle
    w = wl.make_named_workload(args.workload)
    n_tok = min(w.T, args.reference_tokens)
    for _ in range(args.warmup):
        oracle_step_sample(w, min(n_tok, 32))
    times = [oracle_step_sample(w, n_tok) for _ in range(args.steps)]
    sec = float(np.mean(times))
    val = n_tok / sec
    cores = oracle.num_threads()
    sample = f"first {n_tok} of {w.T} tokens of {args.workload}, all projections, forward" + \
             ("+backward" if w.T_bwd else "") + " per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32 storage / f64 accumulate", "data": "synthetic",
        "config": {"workload": args.workload, "desc": workload_desc(args.workload), "sample": sample},
        "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="cfg3",
                    help="cfg1 .. cfg5, a forward-only sweep point decode-T-n / prefill-T-n (T tokens, n tenants), or adamw-n "
                         "(the fused optimizer step + commit of n tenants)")
    ap.add_argument("--sweep", choices=sorted(SWEEPS),
                    help="run a grid of sweep points, one bench.py process and one JSON line each")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--reference-tokens", type=int, default=1024)
    ap.add_argument("--cpu-baseline-tokens", type=int, default=2048)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=6)
    ap.add_argument("--flags", type=int, default=0, help="extra MARLAAS_FLAG_* bits for every call (diagnostics)")
    ap.add_argument("--no-graph", action="store_true", help="time direct launches even for forward-only workloads")
    ap.add_argument("--repeats", type=int, default=5, help="replays of the captured K-step graph (median reported)")
    ap.add_argument("--overlap", action="store_true",
                    help="forward-only workloads: every call carries MARLAAS_FLAG_OVERLAP_PREVIOUS and has a workspace of its own, "
                         "as between two micro-batches that a serving loop interleaves (consecutive calls are independent)")
    ap.add_argument("--multi", action="store_true",
                    help="forward-only multi-projection workloads: q,k,v and gate,up through marlaas_lora_forward_multi (measured: no faster)")
    ap.add_argument("--headline-only", action="store_true", help="default workload without the `configs` entries of the other workloads")
    ap.add_argument("--sustained-seconds", type=float, default=2.0,
                    help="length of the sustained leg of the default run (steps issued back to back for this long)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "b200" else args.warmup
    if args.workload.startswith("adamw-") and args.workload[6:].isdigit():
        run_adamw(args, int(args.workload[6:]))
        return
    if args.sweep:
        if int(os.environ.get("WORLD_SIZE", "1")) != 1:
            raise SystemExit("bench.py --sweep runs on one GPU")
        run_sweep(args)
        return

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import torch
    from paper_2605_08527_b200 import binding as B

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the layer has no CPU path (use --impl reference for the oracle)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    ctx = {"torch": torch, "B": B, "dist": dist, "dev": dev, "rank": rank, "local_rank": local_rank, "world": world}
    w = wl.make_named_workload(args.workload)
    full = args.workload == "cfg3" and world == 1 and not args.headline_only
    out = measure(ctx, args, w, args.workload, args.steps, args.warmup, args.repeats, args.e2e_steps, not args.no_cpu_baseline,
                  sustained_s=args.sustained_seconds if full else 0.0)
    if full and rank == 0:
        # The metric names forward and forward+backward tokens/s and the fraction of the tensor / HBM roofline: the
        # headline above is the training-shaped configuration; the other configured workloads (and the variants that
        # show how much the segment table matters) follow in `configs`, each measured by the same code with fewer steps.
        configs = {}

        def extra(name, wk, steps=10, repeats=3):
            time.sleep(1.0)     # the sustained leg ran into the power cap: let the clocks come back before a burst measurement
            t0 = time.time()
            d = measure(ctx, args, wk, name, steps, 3, repeats, 0, False)
            configs[name] = summarize(d, time.time() - t0)

        extra("cfg3-fwd", wl.make_variant("cfg3-fwd", w))
        extra("cfg3-alltenants", wl.make_variant("cfg3-alltenants", w))
        del w
        extra("cfg2", wl.make_named_workload("cfg2"), steps=50, repeats=5)
        extra("cfg4", wl.make_named_workload("cfg4"))
        w5 = wl.make_named_workload("cfg5")
        extra("cfg5", w5)
        extra("cfg5-alltenants", wl.make_variant("cfg5-alltenants", w5))
        extra("cfg5-fused", wl.make_variant("cfg5-fused", w5))
        extra("cfg5-decode", wl.make_variant("cfg5-decode", w5), steps=20, repeats=5)
        extra("cfg5-decode-fused", wl.make_variant("cfg5-decode-fused", w5), steps=20, repeats=5)
        del w5
        # decode over a wider weight (gate / up of a 14B-class layer: 68 column strips for the 74 CTA pairs): the shape on
        # which the one-pass-over-W kernels come closest to the copy peak
        for nm in ("decode5120x17408-256-32", "decode5120x17408-64-32"):
            extra(nm, wl.make_named_workload(nm), steps=20, repeats=5)
        # the decode workloads once more with consecutive calls overlapped (independent calls, a workspace each: what a
        # serving loop that interleaves two micro-batches submits); reported beside, never instead of, the figures above
        import argparse as _ap
        args_ov = _ap.Namespace(**{**vars(args), "overlap": True})

        def extra_overlap(name, wk, steps=20, repeats=5):
            time.sleep(1.0)
            t0 = time.time()
            d = measure(ctx, args_ov, wk, name, steps, 3, repeats, 0, False)
            configs[name + "+overlap"] = summarize(d, time.time() - t0)

        extra_overlap("cfg2", wl.make_named_workload("cfg2"), steps=50)
        w5 = wl.make_named_workload("cfg5")
        extra_overlap("cfg5-decode-fused", wl.make_variant("cfg5-decode-fused", w5))
        del w5
        extra_overlap("decode5120x17408-256-32", wl.make_named_workload("decode5120x17408-256-32"))
        out["configs"] = configs
    if rank == 0:
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def summarize(d, seconds):
    """The figures of one extra workload that the one-line report carries."""
    r = d["roofline"]
    keep = {"metric": d["metric"], "tokens_per_s": d["value"], "ms_per_step": d["ms_per_step"], "ms_per_step_min": d["ms_per_step_min"],
            "steps": d["steps"], "timed_as": d["config"]["timed_as"], "calls": d["config"]["calls"], "segments": d["config"]["segments"],
            "tenants_present": d["config"]["tenants_present"], "gpu_launches": d["gpu_launches"], "clocks": d["clocks"],
            "work_per_step": d["work_per_step"], "wall_s": round(seconds, 1),
            "roofline": {k: r[k] for k in ("bound", "achieved", "peak", "unit", "frac", "traffic", "traffic_source", "peak_source", "kernel",
                                           "whole_step_frac", "whole_step_tflops", "frac_of_nominal_2250", "frac_of_nominal_8TBs",
                                           "frac_of_measured_sustained", "avg_launch_ms") if k in r}}
    return keep


def measure(ctx, args, w, wname, steps, warmup, repeats, e2e_steps, want_cpu, sustained_s=0.0):
    """One workload through the layer on this rank's GPU; returns the JSON-line dictionary (rank 0) or None."""
    torch, B, dist, dev = ctx["torch"], ctx["B"], ctx["dist"], ctx["dev"]
    rank, local_rank, world = ctx["rank"], ctx["local_rank"], ctx["world"]
    work = algorithmic_work(w)
    ts_np = w.tok_slot()

    def dev_bf16(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(dev)

    def pinned_bf16(bits):
        t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
        return t.pin_memory()

    # ---- device-resident state: one pool per projection, adapters registered, inputs uploaded -------------
    # L2 hygiene: R independent copies of everything a step touches (weights, pools, inputs, outputs), used in
    # rotation, with R chosen so that the copies' inputs exceed three times the L2; no step finds its operands
    # in cache and no flush (whose dirty lines the next step would have to write back) is needed.
    seg = B.Segments(torch.from_numpy(w.seg_offsets.astype(np.int32)).to(dev), torch.from_numpy(w.seg_slot.astype(np.int32)).to(dev))
    Tb = w.T_bwd
    seg_b = seg
    if 0 < Tb < w.T:
        keep = [s for s in range(len(w.seg_slot)) if w.seg_offsets[s] < Tb]
        off = np.array([min(int(w.seg_offsets[s]), Tb) for s in keep] + [Tb], dtype=np.int32)
        seg_b = B.Segments(torch.from_numpy(off).to(dev), torch.from_numpy(w.seg_slot[keep].astype(np.int32)).to(dev))
    l2_bytes = torch.cuda.get_device_properties(dev).L2_cache_size
    input_bytes = sum(p.W_bits.nbytes + (0 if p.dy_bits is None else p.dy_bits.nbytes) for p in w.projections) \
        + sum(x.nbytes for x in {id(p.x_bits): p.x_bits for p in w.projections}.values()) \
        + sum(2 * a.rank * (p.d_in + p.d_out) for p in w.projections for a in p.adapters)
    R = int(min(16, max(1, -(-3 * l2_bytes // input_bytes))))
    overlap = bool(getattr(args, "overlap", False)) and not Tb
    if overlap:
        R = max(R, 2)      # consecutive calls must not share a pool: a single projection alternates between two copies
    l2_note = f"inputs of a step ({input_bytes / 1e6:.0f} MB) rotate over {R} independent copies (> 3x the {l2_bytes / 1e6:.0f} MB L2)" \
        if R > 1 else f"inputs of a step ({input_bytes / 1e6:.0f} MB) are larger than 3x the {l2_bytes / 1e6:.0f} MB L2"
    pinned = {}

    def build_copy():
        projs, x_cache = [], {}
        for p in w.projections:
            pool = B.AdapterPool(p.d_in, p.d_out, w.max_rank, w.n_tenants, device=dev, parts=p.parts)
            for a in p.adapters:
                if p.parts and a.rank > 0:
                    cuts = np.concatenate([[0], np.cumsum(p.parts)])
                    B.marlaas_adapter_pool_register(pool, a.tenant_id, 0, a.rank, a.alpha,
                                                    [dev_bf16(a.A_bits[:, i * a.rank:(i + 1) * a.rank]) for i in range(len(p.parts))],
                                                    [dev_bf16(a.B_bits[:, cuts[i]:cuts[i + 1]]) for i in range(len(p.parts))])
                    continue
                B.marlaas_adapter_pool_register(pool, a.tenant_id, 0, a.rank, a.alpha, dev_bf16(a.A_bits), dev_bf16(a.B_bits))
            key = id(p.x_bits)
            if key not in x_cache:
                x_cache[key] = dev_bf16(p.x_bits)
            if key not in pinned:
                pinned[key] = pinned_bf16(p.x_bits)
            st = {"p": p, "pool": pool, "W": dev_bf16(p.W_bits), "x": x_cache[key], "x_host": pinned[key],
                  "y": torch.empty((w.T, p.d_out), dtype=torch.bfloat16, device=dev),
                  "h": torch.empty((pool.n_parts * w.T, pool.rank_stride), dtype=torch.float32, device=dev),
                  "ws": None}
            ws_bytes[0] = max(ws_bytes[0], B.marlaas_lora_workspace_bytes(pool, w.T))
            if Tb:
                st["dy"] = dev_bf16(p.dy_bits)
                if id(p.dy_bits) not in pinned:
                    pinned[id(p.dy_bits)] = pinned_bf16(p.dy_bits)
                st["dy_host"] = pinned[id(p.dy_bits)]
                st["dx"] = torch.empty((Tb, p.d_in), dtype=torch.bfloat16, device=dev)
                st["dA"] = [torch.empty((pool.n_parts * p.d_in, a.rank), dtype=torch.float32, device=dev) for a in p.adapters]
                # a pool over several projections keeps h as one plane of T rows per projection: the backward rows (a prefix
                # of the batch) are gathered into planes of T_bwd rows before the backward call
                if pool.n_parts > 1 and Tb < w.T:
                    st["h_b"] = torch.empty((pool.n_parts, Tb, pool.rank_stride), dtype=torch.float32, device=dev)
                st["dB"] = [torch.empty((a.rank, p.d_out), dtype=torch.float32, device=dev) for a in p.adapters]
            projs.append(st)
        return projs

    ws_bytes = [0]
    copies = [build_copy() for _ in range(R)]
    # one workspace for every call of the step loop: it is scratch, the calls are ordered on one stream, and a caller
    # would not keep one per projection either
    shared_ws = torch.empty(max(ws_bytes[0], 256), dtype=torch.uint8, device=dev)
    for c in copies:
        for st_ in c:
            st_["ws"] = shared_ws
    projs = copies[0]
    all_projs = [s for c in copies for s in c]

    # A step is all forwards of the layer's projections, then all backwards (as a training step runs them).  The
    # projections see the same mixed batch, so the second and later calls of each pass reuse the plan the first one
    # left in the shared workspace (MARLAAS_FLAG_REUSE_PLAN): the plan is built once per pass, not once per projection.
    # Forward-only steps over several projections (a decode step of a decoder layer): the projections that read the same
    # activations -- q, k, v and gate, up -- do not depend on one another and go through ONE marlaas_lora_forward_multi
    # call each, which may run them side by side; o and down stay calls of their own (in a model they wait for attention
    # and for the activation function).  Concurrent calls need a workspace each.
    GROUPS = (("q", "k", "v"), ("o",), ("gate", "up"), ("down",))
    use_multi = (not Tb) and len(w.projections) > 1 and args.multi and not overlap
    if use_multi or overlap:
        for c in copies:
            for st_ in c:
                st_["ws"] = torch.empty(max(B.marlaas_lora_forward_workspace_bytes(st_["pool"], w.T), 256), dtype=torch.uint8, device=dev)

    def step(i=0, x_of=lambda s: s["x"], dy_of=lambda s: s["dy"], cs=None, seg=seg):
        cs = copies[i % R] if cs is None else cs
        if use_multi:
            by_name = {s["p"].name: s for s in cs}
            done = set()
            for grp in GROUPS:
                members = [by_name[nm] for nm in grp if nm in by_name]
                if members:
                    B.marlaas_lora_forward_multi([dict(pool=s["pool"], x=x_of(s), W=s["W"], seg=seg, y=s["y"], h_save=s["h"],
                                                       workspace=s["ws"]) for s in members], flags=args.flags)
                    done.update(s["p"].name for s in members)
            for s in cs:
                if s["p"].name not in done:
                    B.marlaas_lora_forward(s["pool"], x_of(s), s["W"], seg, y=s["y"], h_save=s["h"], workspace=s["ws"], flags=args.flags)
            return
        for j, s in enumerate(cs):
            fl = args.flags | (B.MARLAAS_FLAG_REUSE_PLAN if j > 0 else 0)
            if overlap:
                # the call before this one used another pool, another workspace and other outputs (the previous projection
                # of this copy, or the last one of the previous copy), and its x, W and table are constants here
                fl = args.flags | B.MARLAAS_FLAG_OVERLAP_PREVIOUS
            B.marlaas_lora_forward(s["pool"], x_of(s), s["W"], seg, y=s["y"], h_save=s["h"], workspace=s["ws"], flags=fl)
        if Tb:
            for j, s in enumerate(cs):
                fl = args.flags | (B.MARLAAS_FLAG_REUSE_PLAN if j > 0 else 0)
                hb = s["h"][:Tb]
                if "h_b" in s:
                    s["h_b"].copy_(s["h"].view(s["pool"].n_parts, w.T, -1)[:, :Tb])
                    hb = s["h_b"]
                B.marlaas_lora_backward(s["pool"], x_of(s)[:Tb], s["W"], dy_of(s), seg_b, dx=s["dx"], dA=s["dA"], dB=s["dB"],
                                        h_saved=hb, workspace=s["ws"], flags=fl)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(warmup, R)):
        step(i)
    for s in all_projs:
        B.marlaas_check_status(s["pool"])
    barrier()

    # Forward-only (decode-shaped) steps last about ten microseconds, less than the host needs to issue one through
    # Python, so the K timed steps are captured once into a CUDA graph and replayed; training-shaped steps are
    # issued directly (their gradient pointer tables come from pageable host memory, which a capture cannot hold).
    graph = None
    if not Tb and not args.no_graph:
        try:
            side = torch.cuda.Stream(device=dev)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                g_ = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g_, stream=side):
                    for i in range(steps):
                        step(i)
            torch.cuda.current_stream().wait_stream(side)
            graph = g_
            wa, wb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            graph.replay()
            wa.record()
            for _ in range(3):
                graph.replay()
            wb.record()
            barrier()
            # enough replays for the clock sampler to see the GPU under this load (about 0.3 s), at least --repeats
            repeats = int(min(5000, max(repeats, 0.3e3 / max(wa.elapsed_time(wb) / 3, 1e-3))))
        except Exception as e:  # noqa: BLE001
            print(f"bench.py: CUDA graph capture failed ({e}); timing direct launches", file=sys.stderr)
            graph = None

    def run_steps():
        if graph is not None:
            graph.replay()
        else:
            for i in range(steps):
                step(i)

    # ---- timed region: device-resident inputs ------------------------------------------------------------------
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    reps = max(1, repeats)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    barrier()
    n0 = B.marlaas_kernel_launch_count()
    if graph is None:
        evs[0][0].record()
        run_steps()
        evs[0][1].record()
        barrier()
        launches = B.marlaas_kernel_launch_count() - n0
        rep_ms = [evs[0][0].elapsed_time(evs[0][1])]
    else:
        # the graph holds exactly K steps; it is replayed `reps` times and the median replay is reported
        for a, b in evs:
            a.record()
            run_steps()
            b.record()
        barrier()
        launches = None
        rep_ms = [a.elapsed_time(b) for a, b in evs]
    clocks = sampler.stop() if rank == 0 else None
    total_ms = max_over_ranks(float(np.median(rep_ms)), dist, dev)
    ms_per_step = total_ms / steps
    tokens_per_step = w.T * world
    value = aggregate_tokens_per_s(w.T, world, ms_per_step)

    # ---- dominant kernel, timed live with events on the launching stream ---------------------------------------
    for s in all_projs:
        B.marlaas_kernel_timing_begin(s["pool"])
    n1 = B.marlaas_kernel_launch_count()
    for i in range(steps):
        step(i)
    launches_direct = B.marlaas_kernel_launch_count() - n1
    if launches is None:
        launches = launches_direct      # what one replay of the captured graph launches
    gemm_ms, gemm_n = 0.0, 0
    for s in all_projs:
        ms, n = B.marlaas_kernel_timing_end(s["pool"])
        gemm_ms += ms
        gemm_n += n
    peaks, peak_src = measured_peaks()
    traffic, traffic_src = profile_traffic(wname)
    gemm_flops_per_step = float(sum(work["gemm_flops"]))
    avg_launch_ms = gemm_ms / max(gemm_n, 1)
    flops_per_launch = gemm_flops_per_step / max(len(work["gemm_flops"]), 1)
    # forward-only batches below the machine balance (flops per byte of the measured peaks) are bound by the one pass
    # over W; everything else by the tensor cores
    hbm_bound = (not Tb) and work["fwd_flops"] / work["fwd_bytes"] < peaks["bf16_tflops"] * 1e12 / (peaks["hbm_gbs"] * 1e9)
    if hbm_bound:
        ach = work["fwd_bytes"] / (ms_per_step * 1e-3) / 1e9
        roofline = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": ach / peaks["hbm_gbs"], "traffic": traffic, "traffic_source": traffic_src, "peak_source": f"of {peak_src}",
                    "kernel": "whole forward call: k_decode_shrink and the decode GEMM (base product + expand), overlapped; "
                              "bytes = W + x + y + present adapters, each once",
                    "bytes_per_launch": work["fwd_bytes"], "avg_launch_ms": ms_per_step,
                    "direct_launch_event_ms": avg_launch_ms,
                    "frac_of_nominal_8TBs": ach / NOMINAL["hbm_gbs"]}
    else:
        ach = flops_per_launch / (avg_launch_ms * 1e-3) / 1e12 if gemm_n else 0.0
        # One denominator: the measured burst figure (the GEMM launches are timed one by one with events, inside a loop of
        # tens of milliseconds).  The sustained and nominal figures are reported beside it, never substituted for it.
        peak_t = peaks["bf16_tflops"]
        whole = (work["fwd_flops"] + work["bwd_flops"]) / (ms_per_step * 1e-3) / 1e12
        roofline = {"bound": "tensor", "achieved": ach, "peak": peak_t, "unit": "TFLOP/s",
                    "frac": ach / peak_t, "traffic": traffic, "traffic_source": traffic_src,
                    "peak_source": f"of {peak_src} (burst)",
                    "kernel": "base GEMM with fused LoRA expand (forward y and backward dx launches)" if Tb else "base GEMM with fused LoRA expand (forward launches)",
                    "launches_timed": gemm_n, "avg_launch_ms": avg_launch_ms, "flops_per_launch": flops_per_launch,
                    "frac_of_nominal_2250": ach / NOMINAL["bf16_tflops"],
                    "frac_of_measured_sustained": ach / peaks["bf16_tflops_sustained"],
                    "whole_step_tflops": whole, "whole_step_frac": whole / peak_t,
                    "whole_step_frac_of_nominal_2250": whole / NOMINAL["bf16_tflops"]}

    # ---- sustained leg: the same steps issued back to back for seconds, clocks sampled throughout -------------------
    sustained = None
    if sustained_s > 0 and rank == 0:
        n_sus = int(max(steps, sustained_s * 1e3 / max(ms_per_step, 1e-3)))
        sampler2 = ClockSampler(local_rank)
        sampler2.start()
        a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a_.record()
        for i in range(n_sus):
            step(i)
        b_.record()
        torch.cuda.synchronize()
        clk2 = sampler2.stop()
        sus_ms = a_.elapsed_time(b_) / n_sus
        whole_s = (work["fwd_flops"] + work["bwd_flops"]) / (sus_ms * 1e-3) / 1e12
        bins = {}
        for smp in sampler2.samples:
            k = int(round(smp[0] / 100.0) * 100)
            bins[k] = bins.get(k, 0) + 1
        sustained = {"steps": n_sus, "seconds": a_.elapsed_time(b_) / 1e3, "ms_per_step": sus_ms, "tokens_per_s": w.T / (sus_ms * 1e-3),
                     "whole_step_tflops": whole_s, "whole_step_frac_of_measured_sustained": whole_s / peaks["bf16_tflops_sustained"],
                     "whole_step_frac_of_measured_burst": whole_s / peaks["bf16_tflops"], "clocks": clk2,
                     "sm_mhz_histogram_100mhz_bins": {str(k): v for k, v in sorted(bins.items())},
                     "ms_per_step_times_median_sm_ghz": sus_ms * (clk2.get("sm_mhz") or 0) / 1e3}

    # ---- end to end: host inputs -> device -> layer -> host outputs, all inside the timed region ------------
    e2e = None
    if e2e_steps > 0:
        host_out = []
        for s in projs:
            o = {"y": torch.empty((w.T, s["p"].d_out), dtype=torch.bfloat16).pin_memory()}
            if Tb:
                o["dx"] = torch.empty((Tb, s["p"].d_in), dtype=torch.bfloat16).pin_memory()
                o["dA"] = [torch.empty(t.shape, dtype=torch.float32).pin_memory() for t in s["dA"]]
                o["dB"] = [torch.empty(t.shape, dtype=torch.float32).pin_memory() for t in s["dB"]]
            host_out.append(o)
        seg_off_h = torch.from_numpy(w.seg_offsets.astype(np.int32)).pin_memory()
        seg_slot_h = torch.from_numpy(w.seg_slot.astype(np.int32)).pin_memory()

        # Two sets of device buffers, used in turn, and three streams: the host-to-device copies of step i + 1 and the
        # device-to-host copies of step i - 1 run beside the layer calls of step i (the link is full duplex), as a caller
        # that feeds the layer from host memory would arrange it.  Every step still copies all of its inputs in and all of
        # its results out inside the timed region.
        sets = [projs, copies[1] if R > 1 else build_copy()]
        for st_ in sets[1]:
            if st_["ws"] is None:
                st_["ws"] = shared_ws if not use_multi else \
                    torch.empty(max(B.marlaas_lora_forward_workspace_bytes(st_["pool"], w.T), 256), dtype=torch.uint8, device=dev)
        host_outs = [host_out, host_out]      # the results of every step land in the same pinned buffers
        segs = [seg, B.Segments(torch.empty_like(seg.seg_offsets), torch.empty_like(seg.seg_slot))]
        main = torch.cuda.current_stream()
        s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_done = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]
        used = [False, False]

        def e2e_step(i):
            k = i % 2
            cs, sg = sets[k], segs[k]
            h2d = d2h = 0
            with torch.cuda.stream(s_in):
                if used[k]:
                    s_in.wait_event(ev_done[k])       # the step that last read these input buffers has finished
                sg.seg_offsets.copy_(seg_off_h, non_blocking=True)
                sg.seg_slot.copy_(seg_slot_h, non_blocking=True)
                h2d += seg_off_h.numel() * 4 + seg_slot_h.numel() * 4
                done = set()
                for s in cs:
                    if id(s["x"]) not in done:
                        s["x"].copy_(s["x_host"], non_blocking=True)
                        h2d += s["x"].numel() * 2
                        done.add(id(s["x"]))
                    if Tb:
                        s["dy"].copy_(s["dy_host"], non_blocking=True)
                        h2d += s["dy"].numel() * 2
                ev_in[k].record(s_in)
            main.wait_event(ev_in[k])
            if used[k]:
                main.wait_event(ev_out[k])            # the results this set held two steps ago are on the host
            step(cs=cs, seg=sg)
            ev_done[k].record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[k])
                for s, o in zip(cs, host_outs[k]):
                    o["y"].copy_(s["y"], non_blocking=True)
                    d2h += s["y"].numel() * 2
                    if Tb:
                        o["dx"].copy_(s["dx"], non_blocking=True)
                        d2h += s["dx"].numel() * 2
                        for hbuf, dbuf in zip(o["dA"] + o["dB"], s["dA"] + s["dB"]):
                            hbuf.copy_(dbuf, non_blocking=True)
                            d2h += dbuf.numel() * 4
                ev_out[k].record(s_out)
            used[k] = True
            return h2d, d2h

        for i in range(2):
            e2e_step(i)
        main.wait_stream(s_out)
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(e2e_steps):
            h2d, d2h = e2e_step(i)
        main.wait_stream(s_in)
        main.wait_stream(s_out)
        b.record()
        barrier()
        e_ms = max_over_ranks(a.elapsed_time(b), dist, dev)
        e2e = {"value": tokens_per_step / (e_ms / e2e_steps * 1e-3), "unit": "tokens/s",
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e2e_steps,
               "ms_per_step": e_ms / e2e_steps,
               "how": "pinned host buffers; two sets of device buffers and three streams, so that a step's copies in, "
                      "its layer calls and its copies out overlap the neighbouring steps' (every step copies all inputs "
                      "in and all results out inside the timed region)"}

    for s in all_projs:
        B.marlaas_check_status(s["pool"])

    # ---- the oracle on the host cores, bounded sample (rank 0, single-GPU runs only) ------------------------
    cpu_baseline = None
    if rank == 0 and world == 1 and want_cpu:
        import oracle
        n_tok = min(w.T, args.cpu_baseline_tokens)
        sec = oracle_step_sample(w, n_tok)
        cpu_baseline = {"value": n_tok / sec, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
                        "sample": f"first {n_tok} of {w.T} tokens of {wname}, all projections, one timed execution "
                                  f"({sec:.1f} s)"}

    out = None
    if rank == 0:
        out = {
            "metric": METRIC if Tb else "multi-LoRA layer tokens/s (fwd)", "value": value, "unit": "tokens/s",
            "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wname, "desc": workload_desc(wname), "tokens_per_step_per_gpu": w.T,
                       "backward_tokens": Tb, "segments": int(len(w.seg_slot)),
                       "tenants_present": int(len(set(int(v) for v in ts_np.tolist() if v >= 0))), "l2": l2_note,
                       "timed_as": "one CUDA graph of K steps, median of %d replays" % reps if graph is not None else "K direct steps",
                       "calls": "q,k,v and gate,up through marlaas_lora_forward_multi (independent projections side by side)" if use_multi else ("one call per projection, each started beside the end of the one before (MARLAAS_FLAG_OVERLAP_PREVIOUS: consecutive calls "
                                 "are independent, as between two interleaved micro-batches; a workspace per call)" if overlap else
                                 "one call per projection and pass"),
                       "multi_gpu": "replicas only (independent copies of the batch per GPU, no collective)"},
            "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e, "sustained": sustained, "gpu_launches": int(launches),
            "clocks": clocks,
            "work_per_step": {"fwd_gflop": work["fwd_flops"] / 1e9, "bwd_gflop": work["bwd_flops"] / 1e9,
                              "fwd_mb": work["fwd_bytes"] / 1e6, "bwd_mb": work["bwd_bytes"] / 1e6},
            "ms_per_step_min": float(min(rep_ms)) / steps,
        }
    for c in copies:
        for st_ in c:
            st_.clear()
    del copies, projs, all_projs
    torch.cuda.empty_cache()
    return out if rank == 0 else None


if __name__ == "__main__":
    main()
