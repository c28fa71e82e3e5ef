"""Benchmark of the Step-Ahead Error Feedback hot path (one Algorithm-1 iteration = one step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 0..4] [--avg-period p] [--impl reference]

Prints ONE JSON line.  `value` = steps/s over all N GPUs with the gradients already resident in HBM
(a ring of pre-generated gradient sets, each far larger than L2, cycled step by step) for a caller that
does not read the state between steps; `with_step_ahead` = the same loop when the caller fetches the
step-ahead point x - e^(k) (where Algorithm 1 evaluates the next gradient) after every step; `e2e` = the
same step driven through the host-buffer entry points (pinned host gradients copied in, parameters
copied out, inside the timed region); `roofline` = the dominant kernel (the worker pass) against the
measured HBM copy bandwidth; `all_configs` = every benchmark configuration under both averaging
schedules (p = 1, and the paper's finite period), a short timed region each; `cpu_baseline` = the CPU
oracle timed on whole steps of the same workload at full size where the host can hold it.  The path does
not shard (the workers are a batch axis on one GPU), so N > 1 runs N independent replicas: no data-path
collective, "scaling": "weak".

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
NOMINAL_HBM_GBS = 8000.0
L2_BYTES = 126 << 20

# DRAM traffic of one worker-pass launch (ncu: dram__bytes_read.sum + dram__bytes_write.sum), as
# (bytes per worker-element, bytes per parameter, where the figure comes from).  The two-term form holds
# because the traffic of these streaming passes grows in proportion to the elements processed; captures
# on a smaller worker count of the same kernel are scaled by it.  The run itself cannot measure DRAM
# counters: the source string says which capture a figure rests on, so a stale one is visible.
WORKER_PASS_DRAM_BYTES = {
    "sign_p1": (12.0, 6.56, "ncu capture of the folded-averaging worker pass, config-2 shapes at 4 workers"),
    "sign_general": (19.64, 0.0, "ncu capture of the plain worker pass, config-2 shapes at 4 workers"),
    "sign_p1_folded": (12.0, 15.63, "ncu capture of k_worker_fused<32> on config 4 itself (one-pass metrics), "
                                    "43.752 GB per launch"),
    "sign_p1_folded16": (12.0, 12.51, "ncu capture of k_worker_fused<16> on config 2 itself (one-pass metrics), "
                                      "5.227 GB per launch"),
    "topk_p1": (12.0, 3.81, "ncu capture of the Top-K worker pass, config-3 shapes at 4 workers"),
    "topk_general": (19.83, 0.0, "ncu capture of the Top-K worker pass with stored differences, config-3 shapes at 4 workers"),
    "topk_p1_folded": (12.0, 12.18, "ncu capture of k_worker_fused<8, Top-K> on config 3"),
    "mu0": None,
}


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


def _oracle_threads():
    from oracle import sae_oracle as so
    return max(1, min(so.max_threads(), len(os.sched_getaffinity(0))))


def _oracle_for(w, avg_period, sizes, x0, threads):
    from oracle import sae_oracle as so
    return so.Oracle(w.num_workers, sizes, x0, compressor=w.compressor, server_compress=w.server_compress,
                     mode=w.mode, avg_period=avg_period, momentum=w.momentum, weight_decay=w.weight_decay,
                     topk_num=w.topk_num, topk_den=w.topk_den, threads=threads)


def _sampled_inputs(w, seed, js):
    """x0 and two gradient sets restricted to the whole tensors `js` (host generator)."""
    import numpy as np
    from paper_2008_05823_b200 import synth
    sizes = w.tensor_sizes
    offs = np.concatenate([[0], np.cumsum(sizes)])
    scales = synth.workload_scales(w, seed)
    x0 = np.concatenate([synth.x0_numpy_range(seed, int(offs[j]), sizes[j]) for j in js])
    grads = [np.stack([np.concatenate([synth.grads_numpy_range(seed, t, k, int(offs[j]), sizes[j], scales[j],
                                                               w.outlier_per_65536, w.outlier_mult) for j in js])
                       for k in range(w.num_workers)]) for t in range(2)]
    return x0, grads


def _full_inputs(w, seed, sets):
    """x0 and `sets` whole gradient sets on the host.  With a CUDA device the seeded device generator makes
    them (the same bits as the host generator, far faster) and they are copied over; otherwise numpy does."""
    import numpy as np
    from paper_2008_05823_b200 import synth
    scales = synth.workload_scales(w, seed)
    try:
        import torch
        cuda = torch.cuda.is_available()
    except Exception:
        cuda = False
    if cuda:
        dev = torch.device("cuda", torch.cuda.current_device())
        gen = synth.DeviceGenerator(w.tensor_sizes, scales, device=dev)
        x0d = torch.empty(w.d, device=dev)
        gen.x0(x0d, seed)
        x0 = x0d.cpu().numpy()
        grads = []
        for t in range(sets):
            g = torch.empty(w.num_workers, w.d, device=dev)
            gen.grads(g, w.num_workers, seed, t, w.outlier_per_65536, w.outlier_mult)
            grads.append(g.cpu().numpy())
            del g
        torch.cuda.synchronize()
        torch.cuda.empty_cache()
        return x0, grads, "device generator, copied to the host"
    x0 = synth.x0_numpy(seed, w.d)
    grads = [synth.workload_grads_numpy(w, seed, t, scales) for t in range(sets)]
    return x0, grads, "host generator"


def _time_steps(orc, grads, lr, steps):
    t0 = time.perf_counter()
    for t in range(steps):
        orc.step(grads[t % len(grads)], lr)
    return time.perf_counter() - t0


def cpu_baseline(w, avg_period, seed, steps, warmup, wall_budget_s=200.0, sample_elems=40_000_000):
    """The oracle, as it stands, on the host cores: whole steps of the workload at FULL size when the host can
    hold it and (warmup + steps) of them fit the wall budget, otherwise on a bounded sample of whole tensors
    (all K workers) scaled by the sampled fraction and marked as an extrapolation.  steps <= 0: as many
    full-size steps as fit ~15 s, at least 2.  Used unchanged by the native arm's `cpu_baseline` and by
    `--impl reference`, so the two cannot disagree about what was timed."""
    import numpy as np
    import psutil
    K, sizes, d = w.num_workers, w.tensor_sizes, w.d
    threads = _oracle_threads()
    warmup = max(1, warmup)
    # ---- a small sample first: the single-thread figure, the sampled estimate, and a guess of the full-size step time
    js = sample_tensors(sizes, max(1, sample_elems // K))
    sub = [sizes[j] for j in js]
    n_sub = int(sum(sub))
    frac = n_sub / d
    x0s, gs = _sampled_inputs(w, seed, js)
    orc = _oracle_for(w, avg_period, sub, x0s, threads)
    orc.step(gs[0], w.lr)
    dt_probe = _time_steps(orc, gs[1:] + gs[:1], w.lr, 2) / 2
    n_s = int(max(2, min(200, 4.0 / max(dt_probe, 1e-4))))
    dt_s = _time_steps(orc, gs, w.lr, n_s)
    sampled = {"value": n_s / dt_s * frac, "unit": "steps/s", "cores": threads, "steps": n_s, "seconds": dt_s,
               "sample": f"{len(js)} of {len(sizes)} whole tensors ({n_sub} of {d} params = {100 * frac:.2f}%), all {K} "
                         f"workers; value = sample steps/s x sampled fraction (an extrapolation: small tensors sit in cache)"}
    del orc
    orc1 = _oracle_for(w, avg_period, sub, x0s, 1)
    orc1.step(gs[0], w.lr)
    n1 = int(max(1, min(n_s, 3.0 / max(dt_s / n_s * threads / 2, 1e-4))))
    dt1 = _time_steps(orc1, gs[1:] + gs[:1], w.lr, n1)
    single = {"value": n1 / dt1 * frac, "unit": "steps/s", "cores": 1, "steps": n1, "seconds": dt1,
              "sample": "the same sample of whole tensors on one thread, scaled by the sampled fraction"}
    del orc1
    est_full_step = 1.25 * (dt_s / n_s) / frac         # (a margin: the sample's small tensors sit in cache)
    # ---- full size, if memory and time allow
    sets = 1 if 4 * K * d > (4 << 30) else 2
    need = 4 * (4 * K * d + sets * K * d + 8 * d)       # oracle state m, e, Delta, C(Delta) + gradient sets
    avail = psutil.virtual_memory().available
    want_steps = steps if steps > 0 else 2
    reason = None
    if need * 1.1 + (6 << 30) > avail:
        reason = (f"host memory: the full-size oracle needs {need / 1e9:.1f} GB, {avail / 1e9:.1f} GB available "
                  f"(short by {(need * 1.1 + (6 << 30) - avail) / 1e9:.1f} GB)")
    elif est_full_step * (warmup + want_steps) + need / 2.5e9 > wall_budget_s:
        reason = (f"time: a full-size step is estimated at {est_full_step:.1f} s, {warmup + want_steps} of them plus "
                  f"set-up exceed the {wall_budget_s:.0f} s budget")
    if reason is None:
        x0, grads, how = _full_inputs(w, seed, sets)
        orc = _oracle_for(w, avg_period, sizes, x0, threads)
        warm_dt = _time_steps(orc, grads, w.lr, warmup) / warmup
        if steps <= 0:
            steps = int(max(2, min(1000, 15.0 / max(warm_dt, 1e-3))))
        dt = _time_steps(orc, grads[::-1], w.lr, steps)
        del orc, grads
        return {"value": steps / dt, "unit": "steps/s", "cores": threads, "kind": "oracle", "full_size": True,
                "extrapolated": False, "steps": steps, "warmup": warmup, "seconds": dt, "ms_per_step": 1e3 * dt / steps,
                "sample": f"whole workload ({d} params x {K} workers), {steps} full-size steps in {dt:.2f} s after "
                          f"{warmup} warm-up; {sets} gradient set(s) from the {how}",
                "single_thread": single, "sampled_estimate": sampled}
    # ---- bounded sample: K steps of a sample sized to fit the budget
    if steps <= 0:
        steps = n_s
        dt = dt_s
    else:
        orc = _oracle_for(w, avg_period, sub, x0s, threads)
        _time_steps(orc, gs, w.lr, warmup)
        dt = _time_steps(orc, gs, w.lr, steps)
        del orc
    return {"value": steps / dt * frac, "unit": "steps/s", "cores": threads, "kind": "oracle", "full_size": False,
            "extrapolated": True, "steps": steps, "warmup": warmup, "seconds": dt, "ms_per_step": 1e3 * dt / steps / frac,
            "not_full_size_because": reason, "sample": sampled["sample"], "single_thread": single,
            "sampled_estimate": sampled}


def config_dict(w, p, args, world):
    """The `config` object of the JSON line: the same for the native and the reference arm."""
    from paper_2008_05823_b200 import configs
    grad_bytes = 4 * w.num_workers * w.d
    ring = ring_length(args, grad_bytes, p, w.compressor == configs.TOPK)
    return {"workload": w.name, "num_workers": w.num_workers, "d": w.d, "num_tensors": w.num_tensors,
            "compressor": {0: "identity", 1: "scaled_sign", 2: "topk"}[w.compressor],
            "avg_period": p, "momentum": w.momentum, "lr": w.lr, "weight_decay": w.weight_decay,
            "mode": "saef" if w.mode == configs.SAEF else "ef",
            "server_compress": "double-way" if w.server_compress else "single-way",
            "topk": f"{w.topk_num}/{w.topk_den}" if w.compressor == configs.TOPK else None,
            "local_steps": args.local_steps,
            "caller_reads_state_between_steps": bool(getattr(args, "read_step_ahead", False)),
            "parallelism": "replicas only" if world > 1 else "1 GPU, workers are a batch axis",
            "l2": l2_note(grad_bytes, ring)}


def ring_length(args, grad_bytes, period=1, topk=False):
    """Gradient sets kept in HBM and cycled, at most 40 GB of them.  Large sets: four, or two.  Sets smaller than
    L2: enough of them that the ring as a whole is twice L2 (a set is evicted before its turn comes again),
    rounded up to a multiple of the step pattern's period -- lcm(4, p): scale buffers alternate, record
    buffers rotate by four, every p-th step averages -- so that a given set always meets the same kind of step
    and the library's cache of step graphs (keyed on the gradient pointer) stays small.
    Top-K: as many sets as 40 GB hold, up to 48.  A short ring makes the gradients periodic, and with them the
    momentum and the Top-K thresholds, which then jump from step to step by more than stochastic gradients make
    them (the thresholds of about thirty (worker, tensor) pairs leave their candidate windows on every step of a
    ring of 2 or 4 sets, none with a fresh set every step): work that a training run would not see."""
    import math
    if args.ring:
        return args.ring
    pattern = math.lcm(4, max(1, period))
    if grad_bytes > L2_BYTES and topk:
        n = int(min(48, (40 << 30) // grad_bytes))
        return n // pattern * pattern if n >= pattern else max(2, n // 2 * 2)
    if grad_bytes > L2_BYTES:
        return 4 if 4 * grad_bytes <= (40 << 30) else 2     # (powers of two divide the step pattern's period)
    need = -(-2 * L2_BYTES // grad_bytes)
    return int(-(-need // pattern) * pattern)


def l2_note(grad_bytes, ring):
    if grad_bytes > L2_BYTES:
        return (f"inputs larger than L2: each step reads a fresh {grad_bytes / 1e9:.2f} GB gradient set "
                f"(ring of {ring})")
    return (f"inputs larger than L2: a ring of {ring} gradient sets of {grad_bytes / 1e6:.1f} MB = "
            f"{ring * grad_bytes / 1e6:.0f} MB is cycled, so a set is evicted before it is read again; the K x d "
            f"state of this workload is itself smaller than L2 and stays there")


def run_reference(args, w, avg_period, rank, world):
    if rank != 0:
        return
    steps, warmup = max(1, args.steps), max(1, args.warmup)
    cb = cpu_baseline(w, avg_period, args.seed, steps, warmup, wall_budget_s=300.0)
    line = {"impl": "reference", "metric": METRIC, "value": cb["value"], "unit": "steps/s", "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": 1e3 / cb["value"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": config_dict(w, avg_period, args, world),
            "note": "no reference implementation exists for this paper: this arm is the CPU oracle on the host cores",
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
        # scaled sign from 16 workers on, no weight decay, above the small-problem limit: the worker pass also writes
        # the ordered sum of the previous step's messages (the folded server pass)
        sign_folded = (not topk) and w.num_workers >= 16 and w.weight_decay == 0.0 and Wd > (1 << 24)
        worker = (12 * Wd + (12 if folded else 4) * d) if topk else 12 * Wd + (12 if sign_folded else 8) * d
        sign_variant = ("sign_p1_folded" if w.num_workers >= 32 else "sign_p1_folded16") if sign_folded else "sign_p1"
        variant = ("topk_p1_folded" if folded else "topk_p1") if topk else sign_variant
    elif w.momentum == 0.0:
        step = 12 * Wd + 16 * d              # g R, e RW | x RW, e_srv RW  (mu = 0: no momentum rows)
        worker = 12 * Wd                     # g R, Delta(e) RW
        variant = "mu0"
    else:
        step = 20 * Wd + 16 * d              # g R, m RW, e RW | x RW, e_srv RW
        worker = 20 * Wd                     # g R, m RW, Delta(e) RW
        variant = "topk_general" if topk else "sign_general"
    return step, worker, variant


def step_ahead_bytes(w, avg_period):
    """Bytes a step must move when the caller reads the step-ahead point x - e^(k) after it (one vector).
    p = 1: the averaged error needs every worker's scale (threshold), and a scale needs the worker's whole
    tensor, so the K momentum rows are read a second time (or the K differences written and read back, which
    is more): 16 W d; then ebar R+W, the server error R+W twice (the server's own scale separates forming
    Delta from subtracting C(Delta)), x R+W, the point W.  Other periods: the general step plus x, one
    worker's stored difference R and the point W."""
    Wd, d = w.num_workers * w.d, w.d
    if avg_period == 1:
        return 16 * Wd + 36 * d, "16 W d + 36 d (g R, m R+W+R | ebar R+W, e_srv (R+W) x 2, x R+W, point W)"
    step, _, _ = algorithmic_bytes(w, avg_period)
    return step + 12 * d, "general step + 12 d (x R, one worker's difference R, point W)"


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
    ring = args.ring or int(max(2, min(4, (40 << 30) // grad_bytes)))
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
    ap.add_argument("--no-step-ahead", action="store_true", help="skip the arm that reads the step-ahead point every step")
    ap.add_argument("--read-step-ahead", action="store_true",
                    help="make the headline itself the loop that fetches the step-ahead point after every step "
                         "(the default run reports that loop beside the headline, as `with_step_ahead`)")
    ap.add_argument("--no-all-configs", dest="all_configs", action="store_false",
                    help="skip the short runs of every configuration under both schedules (default run only)")
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
    overridden = (args.workers > 0 or args.mode is not None or args.single_way or args.momentum is not None or
                  args.topk_percent is not None or args.block_size > 0 or args.local_steps != 1 or p != 1 or
                  args.read_step_ahead)
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, w, p, rank, world)
        return
    if args.sharded:
        run_sharded(args, w, p, rank, local_rank, world)
        return

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
    peak, peak_source = measured_peak()

    def make_inputs(wl, n_sets):
        scales = synth.workload_scales(wl, args.seed)
        gen = synth.DeviceGenerator(wl.tensor_sizes, scales, device=dev)
        x0 = torch.empty(wl.d, device=dev)
        gen.x0(x0, args.seed)
        grads = []
        for t in range(n_sets):
            g = torch.empty(wl.num_workers, wl.d, device=dev)
            gen.grads(g, wl.num_workers, args.seed, t, wl.outlier_per_65536, wl.outlier_mult)
            grads.append(g)
        return gen, x0, grads

    def make(wl, x0, period, local_steps=1):
        return sb.Sae(wl.num_workers, wl.tensor_sizes, x0, compressor=wl.compressor, server_compress=wl.server_compress,
                      mode=wl.mode, avg_period=period, momentum=wl.momentum, weight_decay=wl.weight_decay,
                      topk_num=wl.topk_num, topk_den=wl.topk_den, local_steps=local_steps)

    def measure(wl, x0, grads, period, steps, warmup, read_step_ahead=False, profile=True, local_steps=1):
        """`steps` timed steps (CUDA events on the library's stream, max over ranks), then the same steps again
        with every launch bracketed by events for the per-kernel shares.  read_step_ahead: the caller fetches
        worker 0's step-ahead point x - e^(0) after every step, inside the timed region -- with p = 1 that one
        vector is every worker's gradient point."""
        ring = len(grads)
        sae = make(wl, x0, period, local_steps)
        out = torch.empty(wl.d, device=dev) if read_step_ahead else None

        def one(t):
            sae.step(grads[t % ring], wl.lr)
            if read_step_ahead:
                sae.get_step_ahead(0, out)

        for t in range(warmup):
            one(t)
        sae.sync()
        topk = wl.compressor == configs.TOPK
        fb0 = sae.get_state(sb.STATE_TOPK_FALLBACKS).cpu().tolist() if topk else None
        sampler = ClockSampler(local_rank)
        launches0 = sae.kernel_launches
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        sampler.start()
        ev0.record()
        for t in range(steps):
            one(warmup + t)
        ev1.record()
        barrier()
        clocks = sampler.stop()
        ms_total = ev0.elapsed_time(ev1)
        launches = sae.kernel_launches - launches0
        sae.sync()                                    # raises if the device flagged a range error
        ms_total = max_over_ranks(ms_total, dev)
        res = {"steps": steps, "ms_total": ms_total, "ms_per_step": ms_total / steps,
               "steps_per_s": whole_job_value(steps, ms_total, world), "gpu_launches": launches, "clocks": clocks,
               "kernels": None}
        if topk:     # (row, tensor) pairs whose candidate window missed the threshold during the timed steps
            fb1 = sae.get_state(sb.STATE_TOPK_FALLBACKS).cpu().tolist()
            res["topk_window_misses_per_step"] = {"workers": (fb1[0] - fb0[0]) / steps, "server": (fb1[1] - fb0[1]) / steps,
                                                  "pairs": {"workers": wl.num_workers * wl.num_tensors,
                                                            "server": wl.num_tensors}}
        if profile:
            sae.set_profiling(True)
            for t in range(steps):
                one(warmup + t)
            ktimes = sae.get_kernel_times()
            sae.set_profiling(False)
            total_k = sum(ms for ms, _ in ktimes.values())
            res["kernels"] = {name: {"launches": cnt, "ms_per_launch": ms / cnt, "share": ms / total_k}
                              for name, (ms, cnt) in ktimes.items()}
        sae.close()
        return res

    def fractions(nbytes, ms):
        gbs = nbytes / (ms * 1e-3) / 1e9
        return gbs, gbs / peak, gbs / NOMINAL_HBM_GBS

    def config_entry(wl, period, r, n_sets):
        sb_, wb_, _ = algorithmic_bytes(wl, period)
        gbs, f_meas, f_nom = fractions(sb_, r["ms_per_step"])
        wk = r["kernels"]["worker_pass"]["ms_per_launch"]
        entry = {"workload": wl.name, "avg_period": period, "steps": r["steps"],
                 "steps_per_s": r["steps_per_s"], "ms_per_step": r["ms_per_step"],
                 "step_algorithmic_bytes": sb_, "step_achieved_GBs": gbs,
                 "step_frac_of_measured": f_meas, "step_frac_of_nominal": f_nom,
                 "worker_pass_ms": wk, "worker_pass_algorithmic_bytes": wb_,
                 "worker_pass_frac": fractions(wb_, wk)[1], "worker_pass_frac_of_nominal": fractions(wb_, wk)[2],
                 "kernels": {n: {"launches": v["launches"], "ms_per_launch": v["ms_per_launch"]}
                             for n, v in r["kernels"].items()},
                 "gpu_launches": r["gpu_launches"], "clocks": r["clocks"],
                 "l2": l2_note(4 * wl.num_workers * wl.d, n_sets)}
        if "topk_window_misses_per_step" in r:
            entry["topk_window_misses_per_step"] = r["topk_window_misses_per_step"]
        return entry

    # ---- every benchmark configuration, both averaging schedules, a short timed region each ---------------
    # The smaller configurations come first, before the headline workload has driven the GPU into its power cap
    # (their steps are microseconds long and feel the clock); the headline's own entries are added further down.
    all_configs = None
    do_all = args.all_configs and world == 1 and args.workload == 4 and not overridden
    if do_all:
        all_configs = []
        for idx in range(configs.NUM_WORKLOADS - 1):
            wl = configs.workload(idx)
            gb = 4 * wl.num_workers * wl.d
            _, xs, gs = make_inputs(wl, ring_length(args, gb, wl.avg_period_paper, wl.compressor == configs.TOPK))
            n_steps = {0: 400, 1: 400, 2: 100, 3: 100}[idx]
            for period in (1, wl.avg_period_paper):
                # warm-up: every (gradient set, step kind) pair once, so that its step graph exists before the timed region
                r = measure(wl, xs, gs, period, n_steps, max(args.warmup, 2 * period if period > 1 else 3, len(gs) + 4))
                all_configs.append(config_entry(wl, period, r, len(gs)))
            del xs, gs
            torch.cuda.empty_cache()

    # ---- headline: device-resident throughput, state not read between steps ------------------------------
    K, d = w.num_workers, w.d
    grad_bytes = 4 * K * d
    ring = ring_length(args, grad_bytes, p, w.compressor == configs.TOPK)
    gen, x0, grads = make_inputs(w, ring)
    # (warm-up: every gradient set at least once, so that its step graph exists before the timed region)
    head = measure(w, x0, grads, p, args.steps, max(args.warmup, ring + 1),
                   read_step_ahead=args.read_step_ahead, local_steps=args.local_steps)
    ms_per_step, value, kernels = head["ms_per_step"], head["steps_per_s"], head["kernels"]
    step_bytes, worker_bytes, variant = algorithmic_bytes(w, p)
    if args.read_step_ahead:                   # this loop's own byte count, and the plain worker pass it runs
        step_bytes, _ = step_ahead_bytes(w, p)
        if p == 1:
            worker_bytes, variant = 12 * K * d + 4 * d, "uniform_error_pass"
    wk_ms = kernels["worker_pass"]["ms_per_launch"]
    achieved, frac, frac_nom = fractions(worker_bytes, wk_ms)
    per = WORKER_PASS_DRAM_BYTES.get(variant)
    sgbs, sfrac, sfrac_nom = fractions(step_bytes, ms_per_step)
    roofline = {"bound": "hbm", "kernel": "worker_pass", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "topk_window_misses_per_step": head.get("topk_window_misses_per_step"),
                "frac": frac, "traffic": (per[0] * K * d + per[1] * d) if per else None,
                "traffic_source": per[2] if per else None,
                "algorithmic_bytes_per_launch": worker_bytes, "ms_per_launch": wk_ms, "peak_source": peak_source,
                "frac_of_nominal_8TBs": frac_nom,
                "step": {"algorithmic_bytes": step_bytes, "achieved_GBs": sgbs, "frac": sfrac,
                         "frac_of_nominal_8TBs": sfrac_nom},
                "kernels": kernels}

    # ---- the loop of Algorithm 1 as the paper runs it: the gradient point is read after every step --------
    with_step_ahead = None
    if not args.no_step_ahead and not args.read_step_ahead and args.local_steps == 1:
        sa_steps = max(3, min(args.steps, 30))
        sa = measure(w, x0, grads, p, sa_steps, args.warmup, read_step_ahead=True)
        sa_bytes, sa_formula = step_ahead_bytes(w, p)
        gbs, f_meas, f_nom = fractions(sa_bytes, sa["ms_per_step"])
        with_step_ahead = {"steps_per_s": sa["steps_per_s"], "ms_per_step": sa["ms_per_step"], "steps": sa_steps,
                           "algorithmic_bytes": sa_bytes, "algorithmic_bytes_formula": sa_formula,
                           "achieved_GBs": gbs, "frac_of_measured": f_meas, "frac_of_nominal": f_nom,
                           "gpu_launches": sa["gpu_launches"], "kernels": sa["kernels"], "clocks": sa["clocks"],
                           "api": "sae_step + sae_get_step_ahead(worker 0) every step, device buffers"}

    # the headline workload's entries of the all-configurations block (its p = 1 entry is the headline itself)
    if do_all:
        n_steps = max(10, min(args.steps, 30))
        for period in (1, w.avg_period_paper):
            r = head if period == p else measure(w, x0, grads, period, n_steps, max(args.warmup, 2 * period if period > 1 else 3))
            all_configs.append(config_entry(w, period, r, len(grads)))

    # ---- small workloads: the whole trajectory as ONE captured graph ----------------------------------
    # Configs 0-1 are bound by launch and pipeline latency; with all iterations' gradients resident their
    # steps can be captured into a single CUDA graph (sae_step joins a capture the caller has open), which
    # takes the per-step graph launch off the host as well.  Valid to replay because the launch sequence
    # is periodic: the number of steps is even (scale buffers alternate) and a multiple of p.
    whole_graph = None
    n_traj = w.iterations
    if K * d <= (1 << 23) and n_traj % 2 == 0 and (p == 0 or n_traj % p == 0) and args.local_steps == 1:
        g_all = []
        for t in range(n_traj):
            g = torch.empty(K, d, device=dev)
            gen.grads(g, K, args.seed, t, w.outlier_per_65536, w.outlier_mult)
            g_all.append(g)
        sae = make(w, x0, p)
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
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
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
            sae = make(w, x0, p, args.local_steps)
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

    # the device buffers are no longer needed; the oracle's inputs are generated afresh
    del grads, x0
    torch.cuda.empty_cache()
    cb = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cb = cpu_baseline(w, p, args.seed, steps=0, warmup=1)

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": "steps/s", "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": config_dict(w, p, args, world),
                "clocks": head["clocks"], "e2e": e2e, "gpu_launches": head["gpu_launches"], "roofline": roofline,
                "cpu_baseline": cb, "with_step_ahead": with_step_ahead}
        if all_configs is not None:
            line["all_configs"] = all_configs
        if whole_graph is not None:
            line["whole_trajectory_graph"] = whole_graph
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
