"""Benchmark of the Step-Ahead Error Feedback hot path (one Algorithm-1 iteration = one step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 0..4] [--avg-period p] [--impl reference]

Prints ONE JSON line.  `value` = steps/s over all N GPUs with the gradients already resident in HBM
(a ring of pre-generated gradient sets, each far larger than L2, cycled step by step); `e2e` = the
same step driven through the host-buffer entry points (pinned host gradients copied in, parameters
copied out, inside the timed region); `roofline` = the dominant kernel (the worker pass) against the
measured HBM copy bandwidth; `cpu_baseline` = the CPU oracle timed on a bounded sample of the same
workload.  The path does not shard (the workers are a batch axis on one GPU), so N > 1 runs N
independent replicas: no data-path collective, "scaling": "weak".

`--impl reference` times the CPU oracle alone (there is no reference implementation of this paper).
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "step-ahead EF steps/sec at W workers x d params"
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic of one worker-pass launch per worker-element, from the committed ncu capture
# (dram__bytes_read.sum + dram__bytes_write.sum of a smaller case of the same kernel, which grows in
# proportion to the elements processed).  None until a capture exists for the variant.
# sign_p1: 13.64 B at K = 4 = 12 B per worker-element + (8 B of ebar + sign words) per parameter.
# topk_p1: 1324.2 MB for 4 x 25.56 M worker-elements = 12 B per worker-element + 3.81 B per parameter (ebar);
# topk_general: 2027.4 MB = 19.83 B per worker-element (candidate lists included);
# topk_p1_folded: 2765.3 MB for 8 x 25.56 M worker-elements = 12 B per worker-element + 12.18 B per parameter.
# sign_p1_folded: 43.752 GB for 32 x 109.48 M worker-elements, captured on config 4 itself with one-pass metrics
# (profiles/worker_and_server_pass_cfg4_dram_bytes.md) = 12 B per worker-element + 15.63 B per parameter.
WORKER_PASS_DRAM_BYTES = {"sign_p1": (12.0, 6.56), "sign_general": (19.64, 0.0),      # (per worker-element, per parameter)
                          "sign_p1_folded": (12.0, 15.63),
                          "topk_p1": (12.0, 3.81), "topk_general": (19.83, 0.0),      # profiles/worker_pass_sign_cfg2shapes_4workers.md,
                          "topk_p1_folded": (12.0, 12.18), "mu0": None}                                                # profiles/topk_passes_cfg3shapes_4workers.md


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, stream copy)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in out.splitlines():
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def sample_tensors(sizes, budget):
    """A bounded sample of whole tensors (largest that fits, smallest, median, then a seeded shuffle)."""
    import numpy as np
    order = np.argsort(sizes)
    pick = [int(j) for j in order[::-1] if sizes[j] <= budget][:1] + [int(order[0]), int(order[len(order) // 2])]
    pick += [int(j) for j in np.random.default_rng(0).permutation(len(sizes))]
    out, total = [], 0
    for j in dict.fromkeys(pick):
        if total + sizes[j] <= budget or not out:
            out.append(j)
            total += sizes[j]
    return sorted(out)


def cpu_baseline(w, avg_period, seed, steps, warmup, target_elems=40_000_000):
    """The oracle, as it stands, on a sample of whole tensors of the workload (all K workers)."""
    import numpy as np
    from oracle import sae_oracle as so
    from paper_2008_05823_b200 import synth
    K, sizes = w.num_workers, w.tensor_sizes
    offs = np.concatenate([[0], np.cumsum(sizes)])
    js = sample_tensors(sizes, max(1, target_elems // K))
    sub = [sizes[j] for j in js]
    n_sub = int(sum(sub))
    scales = synth.workload_scales(w, seed)
    threads = max(1, min(so.max_threads(), len(os.sched_getaffinity(0))))
    x0 = np.concatenate([synth.x0_numpy_range(seed, int(offs[j]), sizes[j]) for j in js])
    orc = so.Oracle(K, sub, x0, compressor=w.compressor, server_compress=w.server_compress, mode=w.mode,
                    avg_period=avg_period, momentum=w.momentum, weight_decay=w.weight_decay, topk_num=w.topk_num,
                    topk_den=w.topk_den, threads=threads)
    grads = [np.stack([np.concatenate([synth.grads_numpy_range(seed, t, k, int(offs[j]), sizes[j], scales[j],
                                                               w.outlier_per_65536, w.outlier_mult) for j in js])
                       for k in range(K)]) for t in range(2)]
    for t in range(warmup):
        t0 = time.perf_counter()
        orc.step(grads[t % 2], w.lr)
        warm_dt = time.perf_counter() - t0
    if steps <= 0:                      # aim at ~15 s of CPU work
        steps = int(max(2, min(1000, 15.0 / max(warm_dt, 1e-3))))
    t0 = time.perf_counter()
    for t in range(steps):
        orc.step(grads[t % 2], w.lr)
    dt = time.perf_counter() - t0
    frac = n_sub / w.d
    # the same oracle on one core (a few steps): the plain single-threaded figure
    orc1 = so.Oracle(K, sub, x0, compressor=w.compressor, server_compress=w.server_compress, mode=w.mode,
                     avg_period=avg_period, momentum=w.momentum, weight_decay=w.weight_decay, topk_num=w.topk_num,
                     topk_den=w.topk_den, threads=1)
    orc1.step(grads[0], w.lr)
    n1 = int(max(1, min(steps, 3.0 / max(warm_dt * threads / 4, 1e-3))))
    t0 = time.perf_counter()
    for t in range(n1):
        orc1.step(grads[(t + 1) % 2], w.lr)
    dt1 = time.perf_counter() - t0
    single = {"value": n1 / dt1 * frac, "unit": "steps/s", "cores": 1, "steps": n1, "seconds": dt1}
    return {"value": steps / dt * frac, "unit": "steps/s", "cores": threads, "kind": "oracle", "single_thread": single,
            "sample": f"{len(js)} of {len(sizes)} whole tensors ({n_sub} of {w.d} params = {100 * frac:.2f}%), all "
                      f"{K} workers, {steps} steps in {dt:.2f} s; value = sample steps/s x sampled fraction",
            "sample_seconds": dt, "ms_per_sample_step": 1e3 * dt / steps}


def run_reference(args, w, avg_period, rank):
    if rank != 0:
        return
    steps, warmup = max(1, args.steps), max(1, args.warmup)
    cb = cpu_baseline(w, avg_period, args.seed, steps, warmup, target_elems=30_000_000)
    line = {"impl": "reference", "metric": METRIC, "value": cb["value"], "unit": "steps/s", "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": 1e3 / cb["value"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "num_workers": w.num_workers, "d": w.d, "avg_period": avg_period,
                       "note": "no reference implementation exists for this paper: this arm is the CPU oracle"},
            "cpu_baseline": cb,
            "e2e": {"value": cb["value"], "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def max_over_ranks(value, device=None):
    """Max of a per-rank scalar over the process group (a no-op without one).  Works on CPU tensors
    (gloo) and CUDA tensors (nccl)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(steps, ms_total_max, world):
    """steps/s of all replicas together: every rank runs `steps` steps in at most ms_total_max."""
    return world * steps / (ms_total_max * 1e-3)


def algorithmic_bytes(w, avg_period):
    """Bytes the method itself must move per step (each gradient read once, each persistent state word
    read and written once) and per launch of the worker pass."""
    Wd, d = w.num_workers * w.d, w.d
    topk = w.compressor != 1
    if avg_period == 1:
        step = 12 * Wd + 24 * d              # g R, m RW | x RW, e_srv RW, ebar RW
        # scaled sign: g R, m RW | ebar RW (the pending average is formed in this pass);
        # Top-K: g R, m RW | ebar R (Delta is not stored: the server pass recomputes it from m)
        # Top-K with 8 or 16 workers and no weight decay, folded form: ebar R and W, and the worker-axis sum W
        folded = topk and w.num_workers in (8, 16) and w.weight_decay == 0.0
        # scaled sign with 32 workers, no weight decay, above the small-problem limit: the worker pass also writes
        # the ordered sum of the previous step's messages (the folded server pass)
        sign_folded = (not topk) and w.num_workers >= 32 and w.weight_decay == 0.0 and Wd > (1 << 24)
        worker = (12 * Wd + (12 if folded else 4) * d) if topk else 12 * Wd + (12 if sign_folded else 8) * d
        variant = ("topk_p1_folded" if folded else "topk_p1") if topk else ("sign_p1_folded" if sign_folded else "sign_p1")
    elif w.momentum == 0.0:
        step = 12 * Wd + 16 * d              # g R, e RW | x RW, e_srv RW  (mu = 0: no momentum rows)
        worker = 12 * Wd                     # g R, Delta(e) RW
        variant = "mu0"
    else:
        step = 20 * Wd + 16 * d              # g R, m RW, e RW | x RW, e_srv RW
        worker = 20 * Wd                     # g R, m RW, Delta(e) RW
        variant = "topk_general" if topk else "sign_general"
    return step, worker, variant


def run_sharded(args, w, p, rank, local_rank, world):
    """One job whose K workers are split over the ranks (scaled sign).  Each rank runs the worker lines of
    its own workers; the server pass of every rank reads all K messages in place from their owners."""
    import torch
    import torch.distributed as dist
    from paper_2008_05823_b200 import binding as sb
    from paper_2008_05823_b200 import configs, synth
    from paper_2008_05823_b200.sharded import sharded_sae, worker_range

    if w.compressor == configs.IDENTITY:
        raise SystemExit("--sharded: scaled sign or Top-K")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)
    stream = torch.cuda.Stream(device=dev)
    torch.cuda.set_stream(stream)
    K, d = w.num_workers, w.d
    begin, count = worker_range(K, world, rank)
    scales = synth.workload_scales(w, args.seed)
    gen = synth.DeviceGenerator(w.tensor_sizes, scales, device=dev)
    x0 = torch.empty(d, device=dev)
    gen.x0(x0, args.seed)
    grad_bytes = 4 * count * d
    ring = args.ring or int(max(2, min(4, (40 << 30) // grad_bytes, args.steps + args.warmup)))
    grads = []
    for t in range(ring):
        g = torch.empty(count, d, device=dev)
        gen.grads(g, count, args.seed + 1000 * rank, t, w.outlier_per_65536, w.outlier_mult)   # timing only
        grads.append(g)
    kw = dict(compressor=w.compressor, server_compress=w.server_compress, mode=w.mode, avg_period=p,
              momentum=w.momentum, weight_decay=w.weight_decay, topk_num=w.topk_num, topk_den=w.topk_den)
    if world > 1:
        run = sharded_sae(K, w.tensor_sizes, x0, **kw)
        eng = run.engine
        step = lambda g: run.step(g, w.lr)
        finish = run.finish
    else:
        eng = sb.Sae(K, w.tensor_sizes, x0, shard=(0, K), **kw)
        eng.shard_attach(eng.shard_export())

        def step(g):                       # one stream: begin is ordered before end, end before the next begin
            eng.step_begin(g, w.lr)
            eng.step_end()
        finish = lambda: None
    for t in range(args.warmup):
        step(grads[t % ring])
    finish()
    eng.sync()
    sampler = ClockSampler(local_rank)
    launches0 = eng.kernel_launches
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    sampler.start()
    t0 = time.perf_counter()               # the barriers between the phases are host-side: wall clock around
    for t in range(args.steps):            # a synchronised region (device events would miss the waits)
        step(grads[(args.warmup + t) % ring])
    finish()
    torch.cuda.synchronize()
    ms_total = 1e3 * (time.perf_counter() - t0)
    clocks = sampler.stop()
    gpu_launches = eng.kernel_launches - launches0
    eng.sync()
    ms_total = max_over_ranks(ms_total, dev)
    ms_per_step = ms_total / args.steps
    eng.set_profiling(True)
    for t in range(args.steps):
        step(grads[(args.warmup + t) % ring])
    finish()
    ktimes = eng.get_kernel_times()
    eng.set_profiling(False)
    total_k = sum(ms for ms, _ in ktimes.values())
    kernels = {name: {"launches": cnt, "ms_per_launch": ms / cnt, "share": ms / total_k}
               for name, (ms, cnt) in ktimes.items()}
    peak, peak_source = measured_peak()
    worker_bytes = 20 * count * d          # g R, m RW, Delta RW: the differences are always stored when sharded
    wk_ms = kernels["worker_pass"]["ms_per_launch"]
    achieved = worker_bytes / (wk_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "worker_pass", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": None, "algorithmic_bytes_per_launch": worker_bytes,
                "ms_per_launch": wk_ms, "peak_source": peak_source, "kernels": kernels,
                # what a rank reads from its peers per step (1 bit per element + 1 scale per tensor and
                # worker), against the ring all-reduce of fp32 model differences it replaces
                "exchange_bytes_per_rank_per_step": (K - count) * (w.num_tensors * 4 + ((d + 31) // 32) * 4),
                "fp32_ring_allreduce_bytes_per_rank_per_step": (2 * 4 * d * (world - 1)) // world}
    if world > 1:
        run.close()
    else:
        eng.close()
    if rank == 0:
        line = {"metric": METRIC, "value": 1e3 * args.steps / ms_total, "unit": "steps/s", "n_gpus": world,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "strong", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": w.name + "_sharded", "num_workers": K, "workers_per_rank": count, "d": d,
                           "num_tensors": w.num_tensors,
                           "compressor": {1: "scaled_sign", 2: "topk"}[w.compressor], "avg_period": p,
                           "parallelism": f"sharded: {K} workers over {world} rank(s); every rank's server pass reads "
                                          "all messages in place through row tables",
                           "l2": f"inputs larger than L2: each step reads a fresh {grad_bytes / 1e9:.2f} GB gradient "
                                 f"set (ring of {ring})"},
                "clocks": clocks, "e2e": None, "gpu_launches": gpu_launches, "roofline": roofline, "cpu_baseline": None}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", type=int, default=4, help="index of the benchmark configuration, 0..4 (default: the largest)")
    ap.add_argument("--avg-period", type=int, default=1,
                    help="error-averaging period p (1 = average inside every step; 0 = never)")
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--ring", type=int, default=0, help="gradient sets kept in HBM (0 = auto)")
    ap.add_argument("--workers", type=int, default=0,
                    help="override the workload's worker count (smaller cases of the same kernels for ncu captures)")
    # the paper's variant grid "(EF,SAEF)-(SGD,SGDM,SignSGD,SignSGDM)-(SC,DC)-(TopK)" on the same kernels
    ap.add_argument("--mode", choices=["saef", "ef"], default=None, help="step-ahead or plain local error feedback")
    ap.add_argument("--single-way", action="store_true", help="server sends its Delta uncompressed (SC)")
    ap.add_argument("--momentum", type=float, default=None, help="0 gives the SGD / SignSGD variants")
    ap.add_argument("--topk-percent", type=float, default=None, help="Top-K sparsity in percent (Table 1: 1, 5, 10)")
    ap.add_argument("--block-size", type=int, default=0,
                    help="block-wise compression: cut every tensor into segments of this many elements")
    ap.add_argument("--local-steps", type=int, default=1,
                    help="communicate the model differences every H iterations (needs --avg-period 0); a step is "
                         "still one iteration, so the figure averages H - 1 local iterations and one communicating one")
    ap.add_argument("--sharded", action="store_true",
                    help="sharded operation: the workers are split over the ranks (strong scaling of one job); "
                         "with one rank it times the same two-phase, table-driven path on one GPU")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "native" else args.warmup

    from paper_2008_05823_b200 import configs
    w = configs.workload(args.workload)
    if args.workers > 0:
        w.num_workers = args.workers
        w.name += f"_workers{args.workers}"
    if args.mode is not None:
        w.mode = configs.SAEF if args.mode == "saef" else configs.EF
        w.name += f"_{args.mode}"
    if args.single_way:
        w.server_compress = 0
        w.name += "_sc"
    if args.momentum is not None:
        w.momentum = args.momentum
        w.name += f"_mu{args.momentum:g}"
    if args.topk_percent is not None:
        w.compressor = configs.TOPK
        w.topk_num, w.topk_den = int(round(args.topk_percent * 10)), 1000
        w.name += f"_top{args.topk_percent:g}pct"
    if args.block_size > 0:
        w.tensor_sizes = configs.blockwise_sizes(w.tensor_sizes, args.block_size)
        w.name += f"_blk{args.block_size}"
    p = args.avg_period
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, w, p, rank)
        return
    if args.sharded:
        run_sharded(args, w, p, rank, local_rank, world)
        return

    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2008_05823_b200 import binding as sb
    from paper_2008_05823_b200 import synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # Everything runs on one non-default stream: on such a stream sae_step replays cached CUDA graphs.
    stream = torch.cuda.Stream(device=dev)
    torch.cuda.set_stream(stream)

    K, d = w.num_workers, w.d
    scales = synth.workload_scales(w, args.seed)
    gen = synth.DeviceGenerator(w.tensor_sizes, scales, device=dev)
    x0 = torch.empty(d, device=dev)
    gen.x0(x0, args.seed)
    grad_bytes = 4 * K * d
    ring = args.ring or int(max(2, min(4, (40 << 30) // grad_bytes, args.steps + args.warmup)))
    grads = []
    for t in range(ring):
        g = torch.empty(K, d, device=dev)
        gen.grads(g, K, args.seed, t, w.outlier_per_65536, w.outlier_mult)
        grads.append(g)

    def make():
        return sb.Sae(K, w.tensor_sizes, x0, compressor=w.compressor, server_compress=w.server_compress, mode=w.mode,
                      avg_period=p, momentum=w.momentum, weight_decay=w.weight_decay, topk_num=w.topk_num,
                      topk_den=w.topk_den, local_steps=args.local_steps)

    # ---- device-resident throughput ------------------------------------------------------------------
    sae = make()
    for t in range(args.warmup):
        sae.step(grads[t % ring], w.lr)
    sae.sync()
    sampler = ClockSampler(local_rank)
    launches0 = sae.kernel_launches
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    ev0.record()
    for t in range(args.steps):
        sae.step(grads[(args.warmup + t) % ring], w.lr)
    ev1.record()
    barrier()
    clocks = sampler.stop()
    ms_total = ev0.elapsed_time(ev1)
    gpu_launches = sae.kernel_launches - launches0
    sae.sync()                                    # raises if the device flagged a range error
    ms_total = max_over_ranks(ms_total, dev)
    ms_per_step = ms_total / args.steps
    value = whole_job_value(args.steps, ms_total, world)

    # ---- per-kernel times (same steps again, every launch bracketed by events on the library's stream) ----
    sae.set_profiling(True)
    for t in range(args.steps):
        sae.step(grads[(args.warmup + t) % ring], w.lr)
    ktimes = sae.get_kernel_times()
    sae.set_profiling(False)
    total_k = sum(ms for ms, _ in ktimes.values())
    kernels = {name: {"launches": cnt, "ms_per_launch": ms / cnt, "share": ms / total_k}
               for name, (ms, cnt) in ktimes.items()}
    step_bytes, worker_bytes, variant = algorithmic_bytes(w, p)
    peak, peak_source = measured_peak()
    wk_ms = kernels["worker_pass"]["ms_per_launch"]
    achieved = worker_bytes / (wk_ms * 1e-3) / 1e9
    per = WORKER_PASS_DRAM_BYTES.get(variant)
    roofline = {"bound": "hbm", "kernel": "worker_pass", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": (per[0] * K * d + per[1] * d) if per else None,
                "algorithmic_bytes_per_launch": worker_bytes, "ms_per_launch": wk_ms, "peak_source": peak_source,
                "frac_of_nominal_8TBs": achieved / 8000.0,
                "step": {"algorithmic_bytes": step_bytes, "achieved_GBs": step_bytes / (ms_per_step * 1e-3) / 1e9,
                         "frac": step_bytes / (ms_per_step * 1e-3) / 1e9 / peak,
                         "frac_of_nominal_8TBs": step_bytes / (ms_per_step * 1e-3) / 1e9 / 8000.0},
                "kernels": kernels}
    sae.close()
    del sae

    # ---- small workloads: the whole trajectory as ONE captured graph ----------------------------------
    # Configs 0-1 are bound by launch and pipeline latency; with all iterations' gradients resident their
    # steps can be captured into a single CUDA graph (sae_step joins a capture the caller has open), which
    # takes the per-step graph launch off the host as well.  Valid to replay because the launch sequence
    # is periodic: the number of steps is even (scale buffers alternate) and a multiple of p.
    whole_graph = None
    n_traj = w.iterations
    if K * d <= (1 << 23) and n_traj % 2 == 0 and (p == 0 or n_traj % p == 0):
        g_all = []
        for t in range(n_traj):
            g = torch.empty(K, d, device=dev)
            gen.grads(g, K, args.seed, t, w.outlier_per_65536, w.outlier_mult)
            g_all.append(g)
        sae = make()
        for t in range(n_traj):                      # same phase of every schedule at the start of the capture
            sae.step(g_all[t], w.lr)
        sae.sync()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for t in range(n_traj):
                sae.step(g_all[t], w.lr)
        reps = max(3, min(200, 20000 // n_traj))
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        ev0.record()
        for _ in range(reps):
            graph.replay()
        ev1.record()
        torch.cuda.synchronize()
        ms = ev0.elapsed_time(ev1)
        sae.sync()
        sae.close()
        del sae, graph, g_all
        whole_graph = {"steps_per_graph": n_traj, "replays": reps, "steps_per_s": 1e3 * reps * n_traj / ms,
                       "ms_per_step": ms / (reps * n_traj)}

    # ---- end to end through the host-buffer entry points --------------------------------------------
    e2e = None
    if not args.no_e2e:
        import psutil
        if psutil.virtual_memory().available > 3 * grad_bytes + (8 << 30):
            host_g = torch.empty(K, d, dtype=torch.float32, pin_memory=True)
            host_g.copy_(grads[0])
            host_x = torch.empty(d, dtype=torch.float32, pin_memory=True)
            sae = make()
            e2e_steps = max(2, min(args.steps, int(4e9 // grad_bytes) + 2))
            for _ in range(2):
                sae.step_host(host_g, w.lr)
                sae.get_params_host(host_x)
            barrier()
            t0 = time.perf_counter()
            for _ in range(e2e_steps):
                sae.step_host(host_g, w.lr)          # H2D of this step's gradients + the step
                sae.get_params_host(host_x)          # D2H of the step's result, synchronises
            torch.cuda.synchronize()
            dt = time.perf_counter() - t0
            dt = max_over_ranks(dt, dev)
            sae.sync()
            sae.close()
            e2e = {"value": world * e2e_steps / dt, "unit": "steps/s", "h2d_bytes_per_step": grad_bytes,
                   "d2h_bytes_per_step": 4 * d, "steps": e2e_steps, "ms_per_step": 1e3 * dt / e2e_steps,
                   "api": "sae_step_host + sae_get_params_host (pinned host buffers)"}
            del host_g, host_x
        else:
            e2e = {"value": None, "unit": "steps/s", "skipped": "not enough host memory to pin one gradient set"}

    cb = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cb = cpu_baseline(w, p, args.seed, steps=0, warmup=1)

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": "steps/s", "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": w.name, "num_workers": K, "d": d, "num_tensors": w.num_tensors,
                           "compressor": {0: "identity", 1: "scaled_sign", 2: "topk"}[w.compressor],
                           "avg_period": p, "momentum": w.momentum, "lr": w.lr, "weight_decay": w.weight_decay,
                           "mode": "saef" if w.mode == configs.SAEF else "ef",
                           "server_compress": "double-way" if w.server_compress else "single-way",
                           "topk": f"{w.topk_num}/{w.topk_den}" if w.compressor == configs.TOPK else None,
                           "local_steps": args.local_steps,
                           "parallelism": "replicas only" if world > 1 else "1 GPU, workers are a batch axis",
                           "l2": f"inputs larger than L2: each step reads a fresh {grad_bytes / 1e9:.2f} GB gradient set "
                                 f"(ring of {ring})"},
                "clocks": clocks, "e2e": e2e, "gpu_launches": gpu_launches, "roofline": roofline, "cpu_baseline": cb}
        if whole_graph is not None:
            line["whole_trajectory_graph"] = whole_graph
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
