#!/usr/bin/env python
"""Benchmark of the Q-GenX hot path on B200.

One "step" is one extra-gradient iteration of Algorithm 1 on the scale workload: K = 32 simulated
workers, d = 2^26 fp32 coordinates each, Gaussian-mixture oracle noise (0.9 N(0,1) + 0.1 N(0,100)),
diagonal operator V(x) = D x, bucket 16384, 17 adaptive levels, Huffman code, sub-blocks of 64
coordinates.  A step runs both exchanges (quantize -> encode -> decode -> average), the operator,
the half/dual/primal updates, the adaptive step size, and -- every `--refit-every` steps -- the
histogram and level refit.

Metric: GB/s of the quantize -> encode -> decode -> average path, counted in algorithmic bytes per
exchange  4 K d (read the dual vectors) + 2 S (write, then read, the streams; S = padded stream bytes
+ 4 K nb length words, measured) + 4 d (write the mean), two exchanges per step, divided by the
device time of whole steps (so the operator, updates and refits are inside the time but add no bytes).

  python bench.py [--gpus N] [--steps K] [--warmup W]            # this library
  python bench.py --impl reference [--steps K] [--warmup W]      # the CPU oracle on a bounded sample

With N > 1 (torchrun, one rank per GPU) every rank runs an independent replica of the workload
(the library has no exchange between GPUs): weak scaling, no collective on the data path.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "Q-GenX quantize->code->decode->average GB/s (% of HBM peak); EG iterations/sec"
WORKLOAD = "c5-scale: K=32, d=2^26, mixture noise, diagonal operator, bucket 16384, 17 adaptive levels"


def profile_constants():
    """DRAM bytes and executed thread instructions per coordinate of the encode kernel, as counted by ncu on the
    small case: read from the line "bench: ..." of the committed summary, so that they change together with it.
    (None, None) when the summary does not carry them, e.g. after the kernel changed and before a new capture."""
    import re
    try:
        text = open(os.path.join(ROOT, "profiles", "exchange_kernels_K8_d16M.txt")).read()
        m = re.search(r"^bench: dram_bytes_per_coordinate=([0-9.]+) instructions_per_coordinate=([0-9.]+)", text, re.M)
        return (float(m.group(1)), float(m.group(2))) if m else (None, None)
    except OSError:
        return None, None


def exchange_bytes(K, d, nb, stream_words):
    """Algorithmic bytes of one exchange: read V, write + read the streams and their length words, write the mean."""
    S = 4 * int(stream_words) + 4 * K * nb
    return 4 * K * d + 2 * S + 4 * d


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi clock and throttle-reason samples taken while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.QUERY,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
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
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def max_over_ranks(ms, world):
    """Largest per-rank time; the only collective of the benchmark (timing, not data)."""
    if world == 1:
        return ms
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([ms], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def make_problem(args, device):
    import qgx_inputs as gen
    return gen.c5_diagonal(K=args.workers, d=args.d, device=device, bucket=args.bucket)


def run_ours(args):
    import torch
    import torch.distributed as dist
    import qgx_inputs as gen
    import paper_2308_09187_b200 as qgx

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl")
    torch.cuda.set_device(local)
    device = "cuda:%d" % local
    K, d, bucket, nlev = args.workers, args.d, args.bucket, 17
    nb = (d + bucket - 1) // bucket

    prob = make_problem(args, device)
    ctx = qgx.qgx_create(local)
    cb = qgx.qgx_build_codebook_fixed(nlev, args.subblock)
    cfg = qgx.make_quant_cfg(gen.uniform_levels(nlev).tolist(), bucket, cb, prob.seed,
                             code_type=qgx.QGX_CODE_HUFFMAN, nbins=1024)
    op = qgx.make_operator(qgx.QGX_OP_DIAGONAL, prob.D)
    st = qgx.EgState(prob.x0, K)
    qgx.qgx_eg_init(ctx, st)

    def step():
        t = st.t
        refit = qgx.QGX_REFIT_FIRST if t == 1 else (qgx.QGX_REFIT_CONTINUE if (t - 1) % args.refit_every == 0 else qgx.QGX_REFIT_NONE)
        qgx.qgx_eg_step(ctx, st, op, prob.noise[0], prob.noise[1], cfg, refit=refit)

    for _ in range(max(args.warmup, 1)):
        step()
    qgx.qgx_sync_status(ctx)

    # ---- device-resident timed region --------------------------------------------------------
    qgx.qgx_timing_enable(ctx, 8 * args.steps + 64)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = qgx.qgx_launch_count(ctx)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None
    launches = qgx.qgx_launch_count(ctx) - launches0
    qgx.qgx_sync_status(ctx)
    ms_max = max_over_ranks(ms, world)

    # stream sizes of the last step (both exchanges), for the byte count
    words = []
    for slot in (0, 1):
        _, bbits, _ = qgx.exchange_stream_tensors(ctx, slot, K, nb)
        words.append(int(((bbits.to(torch.int64) + 31) // 32).sum().item()))
    total_bits = [int(qgx.exchange_stream_tensors(ctx, s, K, nb)[2].sum().item()) for s in (0, 1)]
    bytes_step = sum(exchange_bytes(K, d, nb, w) for w in words)
    value = world * bytes_step * args.steps / (ms_max * 1e-3) / 1e9
    peak, peak_kind = measured_peak_gbs()

    n_enc, ms_enc = qgx.qgx_timing_read(ctx, qgx.QGX_KERNEL_ENCODE)
    n_dec, ms_dec = qgx.qgx_timing_read(ctx, qgx.QGX_KERNEL_DECODE)
    n_his, ms_his = qgx.qgx_timing_read(ctx, qgx.QGX_KERNEL_HISTOGRAM)
    n_op, ms_op = qgx.qgx_timing_read(ctx, qgx.QGX_KERNEL_OPERATOR)
    n_fin, ms_fin = qgx.qgx_timing_read(ctx, qgx.QGX_KERNEL_FINISH, reset=True)
    qgx.qgx_timing_enable(ctx, 0)
    # the dominant kernel is the fused quantize+encode pass: it reads the K noise vectors and the
    # operator value once and writes the streams, their lengths, offsets and norms
    enc_bytes = 4 * K * d + 4 * d + 4 * (sum(words) / 2.0) + 12 * K * nb
    enc_ms = ms_enc / max(n_enc, 1)
    achieved = enc_bytes / (enc_ms * 1e-3) / 1e9 if n_enc else None
    # DRAM bytes per launch of that kernel: counted by ncu on a smaller case of the same kernel (see
    # profiles/exchange_kernels_K8_d16M.txt: 655.2 MB read + written for K * d = 2^27 coordinates) and scaled by
    # the coordinates of a launch, which the traffic is proportional to.  Set to None when the kernel changes.
    dram_per_coord, instr_per_coord = profile_constants()
    traffic = args.traffic_bytes
    if traffic is None and dram_per_coord is not None:
        traffic = dram_per_coord * K * d
    # The same kernel against the issue ceiling that actually binds it: executed thread instructions per second
    # (ncu's count per coordinate x coordinates per launch / the event time) over 148 SMs x 128 lanes x the SM clock
    # seen during the timed region.
    alu = None
    if n_enc and instr_per_coord is not None:
        sm_mhz = (clocks or {}).get("sm_mhz") or 1965.0
        alu_peak = 148 * 128 * sm_mhz * 1e6 / 1e12
        alu_ach = instr_per_coord * K * d / (enc_ms * 1e-3) / 1e12
        alu = {"achieved": alu_ach, "peak": alu_peak, "unit": "T thread-instructions/s", "frac": alu_ach / alu_peak}
    roofline = {"bound": "hbm", "kernel": "k_exchange_encode", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": (achieved / peak) if achieved else None, "peak_kind": "of " + peak_kind,
                "traffic": traffic, "ms_per_launch": enc_ms, "alu": alu,
                "kernels_ms_per_step": {"encode": ms_enc / args.steps, "decode": ms_dec / args.steps,
                                        "histogram": ms_his / args.steps, "operator": ms_op / args.steps,
                                        "finish": ms_fin / args.steps}}

    # ---- end to end: host buffers, H2D of the step's inputs and D2H of its result inside the time ----
    e2e = None
    if rank == 0 or world > 1:
        try:
            e2e = run_e2e(args, qgx, ctx, st, op, cfg, prob, world, bytes_step)
        except Exception as ex:  # e.g. not enough pinned host memory
            e2e = {"value": None, "unit": "GB/s", "error": str(ex)[:200]}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(args, cfg, prob)

    others = None
    if rank == 0 and world == 1 and not args.no_other_configs:
        del prob                                      # the scale workload's 17 GB of noise
        try:
            others = other_configs(qgx, ctx)
        except Exception as ex:
            others = {"error": str(ex)[:200]}

    if rank == 0:
        s_val, g_val = st.read_scalars()
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_max / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": WORKLOAD if (K, d, bucket) == (32, 1 << 26, 16384) else "K=%d d=%d bucket=%d" % (K, d, bucket),
                       "K": K, "d": d, "bucket": bucket, "nlev": nlev, "subblock": args.subblock, "code": "huffman",
                       "refit_every": args.refit_every, "parallelism": "replicas x%d" % world,
                       "l2": "inputs (%.1f GB per exchange) larger than L2" % (4e-9 * K * d)},
            "pct_hbm_peak_measured": 100.0 * value / world / peak, "pct_of_8TBps": 100.0 * value / world / 8000.0,
            "eg_iterations_per_s": world * args.steps / (ms_max * 1e-3),
            "bits_per_coordinate": sum(total_bits) / (2.0 * K * d),
            "algorithmic_bytes_per_step": bytes_step,
            "gpu_launches": launches, "clocks": clocks, "roofline": roofline, "e2e": e2e, "cpu_baseline": cpu,
            "gamma": g_val, "sum_sq": s_val, "other_configs": others,
        }
        print(json.dumps(line))
    qgx.qgx_destroy(ctx)
    if world > 1:
        dist.destroy_process_group()


def other_configs(qgx, ctx):
    """The smaller configurations, timed on the device with CUDA events around the calls (the context's stream is
    torch's current stream); they are launch- and latency-bound: supplementary figures, not the headline."""
    import numpy as np
    import torch
    import qgx_inputs as gen

    def timed(fn, n, warm=3):
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e-3 / n

    out = {}
    g = gen.c1_bilinear(T=100, device="cuda")
    cfg = qgx.make_quant_cfg(gen.uniform_levels(9).numpy(), g.bucket, qgx.qgx_build_codebook_fixed(9, 32), g.seed)
    op = qgx.make_operator(qgx.QGX_OP_BILINEAR, g.A)
    st = qgx.EgState(g.z0, g.K)
    qgx.qgx_eg_init(ctx, st)
    i = [0]

    def c1_step():
        t = i[0] % 100
        i[0] += 1
        qgx.qgx_eg_step(ctx, st, op, g.noise[t, 0], g.noise[t, 1], cfg)
    out["c1_bilinear_n1024_K4_iterations_per_s"] = 1.0 / timed(c1_step, 200)

    vi = gen.c4_affine(device="cuda")
    cfg4 = qgx.make_quant_cfg(gen.uniform_levels(17).numpy(), vi.bucket, qgx.qgx_build_codebook_fixed(17, 32), vi.seed,
                              code_type=qgx.QGX_CODE_HUFFMAN)
    op4 = qgx.make_operator(qgx.QGX_OP_DENSE_AFFINE, vi.M, vi.b)
    st4 = qgx.EgState(vi.x0, vi.K)
    qgx.qgx_eg_init(ctx, st4)
    nz = vi.noise(1)
    qgx.qgx_eg_step(ctx, st4, op4, nz[0], nz[1], cfg4, refit=qgx.QGX_REFIT_FIRST)
    out["c4_affine_n8192_K8_iterations_per_s"] = 1.0 / timed(lambda: qgx.qgx_eg_step(ctx, st4, op4, nz[0], nz[1], cfg4), 100)
    del vi, op4, st4

    c2 = gen.c2_gaussian(device="cuda")
    cfg2 = qgx.make_quant_cfg(np.linspace(0, 1, 17), c2.bucket, qgx.qgx_build_codebook_fixed(17, 64), c2.seed,
                              code_type=qgx.QGX_CODE_HUFFMAN)
    qgx.qgx_update_levels(ctx, c2.v, cfg2, qgx.QGX_REFIT_FIRST)
    K2, d2 = c2.v.shape
    mean, tot = qgx.qgx_exchange(ctx, c2.v, cfg2, 3, slot=0)
    sec = timed(lambda: qgx.qgx_exchange(ctx, c2.v, cfg2, 3, slot=0), 20)
    nb2 = d2 // c2.bucket
    words = int(((tot.cpu().numpy().astype(np.int64) + 31) // 32).sum()) + K2 * nb2
    out["c2_exchange_K8_d2p24_GBps"] = exchange_bytes(K2, d2, nb2, words) / sec / 1e9
    del c2

    lw = gen.c3_layerwise(K=16, device="cuda")
    cfgs, at = [], 0
    for n in lw.sizes:
        c = qgx.make_quant_cfg(np.linspace(0, 1, lw.nlev), lw.bucket, qgx.qgx_build_codebook_fixed(lw.nlev, 32), lw.seed,
                               code_type=qgx.QGX_CODE_HUFFMAN)
        qgx.qgx_update_levels(ctx, lw.v[:, at:at + n].contiguous(), c, qgx.QGX_REFIT_FIRST)
        cfgs.append(c)
        at += n
    out["c3_layerwise_16_tensors_K16_ms_per_exchange"] = 1e3 * timed(lambda: qgx.qgx_exchange_segments(ctx, lw.v, lw.sizes, cfgs, 9), 20)
    qgx.qgx_sync_status(ctx)
    return out


def run_e2e(args, qgx, ctx, st, op, cfg, prob, world, bytes_step):
    """The same step through the public call with HOST inputs: the step's noise is copied from pinned host
    memory to the device and the step's result (the new iterate, with the sum of squared differences and the step
    size) is read back."""
    import torch
    import torch.distributed as dist
    K, d = args.workers, args.d
    host_noise = torch.empty((2, K, d), dtype=torch.float32, pin_memory=True)
    host_noise.copy_(prob.noise)
    host_out = torch.empty(2, dtype=torch.float64, pin_memory=True)
    host_x = torch.empty((d,), dtype=torch.float32, pin_memory=True)      # the step's result: the new iterate
    dev_noise = prob.noise                       # destination of the per-step copy
    steps = max(1, min(args.steps, args.e2e_steps))

    def step():
        dev_noise.copy_(host_noise, non_blocking=True)
        qgx.qgx_eg_step(ctx, st, op, dev_noise[0], dev_noise[1], cfg, refit=qgx.QGX_REFIT_NONE)
        host_out.copy_(st.scalars, non_blocking=True)
        host_x.copy_(st.X, non_blocking=True)

    step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = max_over_ranks(e0.elapsed_time(e1), world)
    qgx.qgx_sync_status(ctx)
    return {"value": world * bytes_step * steps / (ms * 1e-3) / 1e9, "unit": "GB/s", "steps": steps,
            "ms_per_step": ms / steps, "h2d_bytes_per_step": 2 * K * d * 4, "d2h_bytes_per_step": 4 * d + 16,
            "eg_iterations_per_s": world * steps / (ms * 1e-3)}


def oracle_sample_problem(args, seed=1005):
    """A bounded sample of the workload for the single-threaded oracle: the same K and bucket, fewer buckets."""
    import qgx_inputs as gen
    d_s = args.cpu_buckets * args.bucket
    return gen.c5_diagonal(K=args.workers, d=d_s, device="cpu", seed=seed, bucket=args.bucket), d_s


def cpu_model():
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


class pinned_to_one_core:
    """Runs the enclosed code on one host core (where the system allows it)."""

    def __enter__(self):
        self.before = None
        try:
            self.before = os.sched_getaffinity(0)
            os.sched_setaffinity(0, {min(self.before)})
        except (AttributeError, OSError):
            self.before = None
        return self

    def __exit__(self, *exc):
        if self.before is not None:
            os.sched_setaffinity(0, self.before)


def cpu_baseline(args, cfg, prob):
    """The oracle, as it stands, on a bounded sample of the same workload: pinned to one host core, and again
    with one thread per worker (each thread runs one worker's quantize -> encode -> decode; timing only)."""
    import numpy as np
    from concurrent.futures import ThreadPoolExecutor
    from oracle import qgx_oracle as o
    K, bucket = args.workers, args.bucket
    d_s = args.cpu_buckets * bucket
    a = (prob.D[:d_s] * prob.x0[:d_s]).cpu().numpy()
    V = (prob.noise[0, :, :d_s].cpu().numpy() + a[None, :]).astype(np.float32)
    lev = np.array(cfg.level_list(), dtype=np.float32)
    cbo = o.codebook_from(cfg.cb.lengths(), cfg.cb.codes(), subblock=cfg.cb.subblock)
    with pinned_to_one_core():
        t0 = time.perf_counter()
        mean, total = o.exchange(V, bucket, lev, cbo, int(cfg.seed), 2)
        dt = time.perf_counter() - t0
    nb = d_s // bucket
    words = int(np.sum((total.astype(np.int64) + 31) // 32)) + K * nb      # upper estimate of padded words
    by = exchange_bytes(K, d_s, nb, words)
    threads = max(1, min(K, os.cpu_count() or 1))
    slices = [np.ascontiguousarray(V[k:k + 1]) for k in range(K)]
    with ThreadPoolExecutor(max_workers=threads) as pool:               # the C calls release the interpreter lock
        t0 = time.perf_counter()
        list(pool.map(lambda vk: o.exchange(vk, bucket, lev, cbo, int(cfg.seed), 2), slices))
        dt_threads = time.perf_counter() - t0
    return {"value": by / dt / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle",
            "cpu": cpu_model(), "host_cores": os.cpu_count(),
            "threads_value": by / dt_threads / 1e9, "threads": threads,
            "sample": "one exchange of K=%d workers x %d buckets of %d coordinates (%.1f M coordinates): %.1f s on one "
                      "core, %.1f s with %d threads (one worker per thread)"
                      % (K, args.cpu_buckets, bucket, K * d_s / 1e6, dt, dt_threads, threads)}


def run_reference(args):
    """--impl reference: the CPU oracle's own iteration on a bounded sample of the workload, one host core."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    import qgx_inputs as gen
    from oracle import qgx_oracle as o
    K, bucket, nlev = args.workers, args.bucket, 17
    nbk = max(1, args.ref_buckets)
    d_s = nbk * bucket
    prob = gen.c5_diagonal(K=K, d=d_s, device="cpu", bucket=bucket)
    opo = o.Op(o.OP_DIAGONAL, prob.D.numpy())
    st = o.EgState(prob.x0.numpy(), K)
    lev = gen.uniform_levels(nlev).numpy().copy()
    cbo = o.codebook_fixed(nlev, args.subblock)
    n0, n1 = prob.noise[0].numpy(), prob.noise[1].numpy()
    bits = 0

    def step():
        t = st.t
        refit = 2 if t == 1 else (1 if (t - 1) % args.refit_every == 0 else 0)
        return o.eg_step(st, opo, n0, n1, bucket, lev, cbo, prob.seed, refit=refit, code_type=o.CODE_HUFFMAN, nbins=1024)

    with pinned_to_one_core():
        for _ in range(max(args.warmup, 1)):
            step()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            bits = step()
        dt = time.perf_counter() - t0
    words = bits // 32 + 2 * K * nbk                      # both exchanges, padded estimate
    by = 2 * (4 * K * d_s + 4 * d_s) + 2 * (4 * words + 2 * 4 * K * nbk)
    value = by * args.steps / dt / 1e9
    sample = "each step: one full iteration (2 exchanges) on K=%d workers x %d buckets of %d coordinates" % (K, nbk, bucket)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD + " (bounded sample)", "K": K, "d": d_s, "bucket": bucket, "nlev": nlev,
                   "subblock": args.subblock, "code": "huffman", "refit_every": args.refit_every},
        "eg_iterations_per_s": args.steps / dt,
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample, "cpu": cpu_model(),
                         "host_cores": os.cpu_count()},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workers", type=int, default=32, help="K, simulated workers")
    ap.add_argument("--d", type=int, default=1 << 26)
    ap.add_argument("--bucket", type=int, default=16384)
    ap.add_argument("--subblock", type=int, default=64)
    ap.add_argument("--refit-every", type=int, default=10)
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-buckets", type=int, default=320, help="buckets per worker in the timed oracle sample")
    ap.add_argument("--ref-buckets", type=int, default=2, help="buckets per worker per step of --impl reference")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true", help="skip the supplementary timings of the smaller configurations")
    ap.add_argument("--traffic-bytes", type=float, default=None,
                    help="dram bytes per launch of the dominant kernel from the last ncu capture (null once the kernel changed)")
    args = ap.parse_args()
    if args.steps is None:
        args.steps = 100 if args.impl == "ours" else 10
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
