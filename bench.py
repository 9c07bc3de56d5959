#!/usr/bin/env python
"""EFCP optimizer-step benchmark (one JSON line on stdout, printed by rank 0).

A "step" is one pass of the whole hot path over one synthetic gradient:
error feedback -> exact Top-k -> residual -> ring insert -> scalar products ->
m x m coefficients -> linear combination (one efcp_step call).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME]
  python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...
  python bench.py --impl reference ...        # the CPU oracle, timed on the host cores

N > 1 runs N independent replicas (one optimizer state per GPU, no data-path
collective): weak scaling.  Before timing, the ring window is filled completely
(m untimed steps) so that the timed steps are steady-state steps.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2306_06098_b200 import gradgen  # noqa: E402

METRIC = "efcp_steps_per_sec"
UNIT = "steps/s"

# DRAM traffic per launch of the dominant kernels from the ncu captures summarised under
# profiles/ (dram__bytes_read.sum + dram__bytes_write.sum), keyed by workload; None until
# a capture of that workload exists.  Scaled from a smaller capture where noted there.
# Captured on a quarter-size copy of c4_bert_base (same slab width and segment lengths, see
# profiles/): DRAM traffic / bytes to move was 1.103 for k_sp_rows and 1.079 for k_lcg, and it
# is proportional to the bytes streamed, so the C4 figures are those ratios times the C4 bytes
# per launch.
NCU_TRAFFIC_BYTES = {
    "c4_bert_base": {"sp": int(1.103 * 6 * 1024 * 1_094_822),
                     "lcg": int(1.079 * (6 * 1024 * 1_094_822 + 4 * 109_482_240))},
}


def load_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (earlier pool measurement)"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while timing."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, pw = [], [], []
        reasons = set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.strip().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                pw.append(float(parts[2]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def dist_setup(n_gpus):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        backend = "nccl" if torch.cuda.is_available() else "gloo"
        dist.init_process_group(backend=backend)
    return world, rank, local


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(x, world, device):
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def make_oracle(d, m, k, lam, precond):
    """The CPU oracle of the preconditioner being timed (None when it cannot hold the case:
    the Sparse GGT oracle keeps a dense m x d window)."""
    from oracle import ref
    if precond == "ggt":
        if d * m * 8 > (4 << 30):
            return None
        from oracle import ggt
        return ggt.RefSparseGGT(d, m, k, lam)
    return ref.RefEFCP(d, m, k, lam)


def oracle_steps_per_sec(w, grads_host, n_steps, precond="mfac", threads=None):
    """Times the CPU oracle as it stands on `n_steps` gradients of workload w; `threads`
    limits its OpenMP team (None: every core the process may use)."""
    from oracle import ref
    o = make_oracle(w.d, w.m, w.k, w.lam, precond)
    if o is None:
        return None
    all_threads = ref.num_threads()
    if threads is not None:
        ref.set_num_threads(threads)
    try:
        used = ref.num_threads()
        t0 = time.perf_counter()
        for i in range(n_steps):
            o.step(grads_host[i % len(grads_host)])
        dt = time.perf_counter() - t0
    finally:
        ref.set_num_threads(all_threads)
    o.close()
    return n_steps / dt, used, dt


REFERENCE_BUDGET_S = 240.0  # the reference arm's timed + warm-up steps stay within this


def run_reference(args, world, rank):
    """The reference arm: the CPU oracle on the benchmark's own workload.  The first step on
    the full workload is timed; only if warm-up + steps at that pace would exceed the budget
    is the workload cut down (leading d / 2^j coordinates of the same gradients, k scaled
    alike), and then the line reports what was timed, with the extrapolation in a key of its
    own."""
    if rank != 0:
        return
    from oracle import ref
    w = get_workload(args.workload)
    total = max(1, args.steps + args.warmup)
    # inputs only: the workload's generator, on the GPU when there is one (the same bytes the
    # main arm's gradients have), copied to the host
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    gs = gradgen.GradStream.for_workload(w, dev)
    grads = [gs.next().cpu().numpy() for _ in range(min(4, total))]
    del gs
    if dev == "cuda":
        torch.cuda.empty_cache()
    o = make_oracle(w.d, w.m, w.k, w.lam, args.precond)
    if o is None:
        print(json.dumps({"impl": "reference",
                          "unavailable": "the Sparse GGT oracle keeps a dense m x d window"}))
        return
    t0 = time.perf_counter()
    o.step(grads[0])  # counts as the first warm-up step when there is one
    first = time.perf_counter() - t0
    done = 1
    shrink = 1
    d, k = w.d, w.k
    while first * total / shrink > REFERENCE_BUDGET_S and w.d // (shrink * 2) >= 4096:
        shrink *= 2
    if shrink > 1:
        o.close()
        d, k = w.d // shrink, max(1, w.k // shrink)
        grads = [g[:d].copy() for g in grads]
        o = make_oracle(d, w.m, k, w.lam, args.precond)
        done = 0
    for i in range(done, args.warmup):
        o.step(grads[i % len(grads)])
    # exactly args.steps timed steps; without warm-up the sizing step above is the first of them
    n_timed = args.steps
    carried = min(done, max(0, done - args.warmup))
    t0 = time.perf_counter()
    for i in range(carried, n_timed):
        o.step(grads[(args.warmup + i) % len(grads)])
    dt = time.perf_counter() - t0 + (first if carried else 0.0)
    o.close()
    value = n_timed / dt
    sample = (f"{n_timed} oracle steps on the full workload, window filling from empty (the "
              f"oracle loops over all m rows whether written or not), {dt:.1f} s")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": args.gpus, "steps": n_timed, "warmup": args.warmup,
        "ms_per_step": 1e3 / value, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "d": d, "m": w.m, "k": k, "lambda": w.lam,
                   "preconditioner": {"mfac": "Sparse M-FAC", "ggt": "Sparse GGT"}[args.precond]},
        "gpu_launches": 0,
    }
    if shrink > 1:
        sample = (f"{n_timed} oracle steps on the leading d/{shrink} = {d} coordinates of the "
                  f"workload's gradients with k = {k} (one full-size step took {first:.1f} s, "
                  f"too slow for {total} steps), {dt:.1f} s")
        line["extrapolated_full_workload"] = {
            "value": value / shrink, "unit": UNIT, "d": w.d, "k": w.k,
            "how": f"timed steps/s divided by {shrink}: the oracle's cost is linear in d at "
                   f"fixed density and m; the one full-size step measured gives "
                   f"{1.0 / first:.4f} steps/s"}
    line["cpu_baseline"] = {"value": value, "unit": UNIT, "cores": ref.num_threads(),
                            "kind": "oracle", "sample": sample}
    line["e2e"] = {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    print(json.dumps(line), flush=True)


def run_local_shards(args):
    """The coordinate-sharded step with all shards on one GPU of this process (exchange buffers
    summed on the device): what splitting the step at its exchange points costs, without any
    interconnect.  Not the benchmark's metric: a diagnostic line."""
    from paper_2306_06098_b200 import binding, sharded
    torch.cuda.set_device(0)
    w = get_workload(args.workload)
    n = args.local_shards
    shards, ranges = sharded.create_local_shards(binding, w.d, w.m, w.k, w.lam, n)
    stepper = sharded.ShardedStep(shards, sharded.sum_in_process)
    gs = gradgen.GradStream.for_workload(w, "cuda")
    ubuf = torch.empty(w.d, dtype=torch.float32, device="cuda")
    split = lambda t: [t[lo:hi] for lo, hi in ranges]
    prefill = w.m if args.prefill < 0 else args.prefill
    for _ in range(prefill):
        stepper.step(split(gs.next()), split(ubuf))
    pool = [gs.next().clone() for _ in range(min(args.steps + args.warmup, 64))]
    del gs
    for i in range(args.warmup):
        stepper.step(split(pool[i % len(pool)]), split(ubuf))
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for i in range(args.steps):
        stepper.step(split(pool[(args.warmup + i) % len(pool)]), split(ubuf))
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / args.steps
    assert all(s.status() == 0 for s in shards)
    print(json.dumps({"metric": METRIC, "value": 1e3 / ms, "unit": UNIT, "n_gpus": 1,
                      "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
                      "higher_is_better": True, "data": "synthetic", "dtype": "f32",
                      "config": {"workload": w.name, "d": w.d, "m": w.m, "k": w.k,
                                 "parallelism": f"{n} coordinate shards on one GPU, buffers "
                                                f"summed on the device (no interconnect)",
                                 "ranges": ranges, "prefill_steps": prefill}}), flush=True)


def get_workload(name):
    if name.startswith("custom:"):
        f = name.split(":", 1)[1].split(",")
        return gradgen.Workload(name, int(f[0]), int(f[1]), int(f[2]), float(f[3]), 200, int(f[4]),
                                int(f[5]) if len(f) > 5 else None)
    return gradgen.WORKLOADS[name]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=gradgen.C4.name,
                    help="one of %s, or custom:d,m,k,lambda,rank[,scale_block] (profiling cases)"
                    % ", ".join(sorted(gradgen.WORKLOADS)))
    ap.add_argument("--rhs", default="compressed", choices=["compressed", "accumulator"],
                    help="precondition c_t (Algorithm 1, default) or the whole accumulator a_t")
    ap.add_argument("--values", default="fp32", choices=["fp32", "bf16"],
                    help="window value format (bf16: Section 3.1 'Format for V', not the default)")
    ap.add_argument("--precond", default="mfac", choices=["mfac", "ggt"],
                    help="ggt: Sparse GGT (appendix), lambda of the workload is its eps; m <= 160")
    ap.add_argument("--lcg", default="fixed", choices=["fixed", "fp32"],
                    help="accumulator of the linear combination: int32 fixed point with an fp32 "
                         "fallback per slab (the library's default) or fp32 atomics (EFCP_LCG_FP32)")
    ap.add_argument("--block", type=int, default=0,
                    help="block-wise Top-k with blocks of this many coordinates (Section 3.1 "
                         "'Sparsity Pattern'); 0 = global Top-k, the default")
    ap.add_argument("--apply-update", action="store_true",
                    help="time efcp_step_apply: the step plus theta <- (1 - gamma eta) theta - "
                         "eta s u on a resident parameter vector (eta 1e-3, gamma 1e-4)")
    ap.add_argument("--no-u", action="store_true",
                    help="with --apply-update and no clipping: do not materialise u (the linear "
                         "combination updates theta directly)")
    ap.add_argument("--clip", type=float, default=0.0,
                    help="with --apply-update: clip |u| to this norm (adds the norm kernels)")
    ap.add_argument("--prefill", type=int, default=-1,
                    help="untimed steps before warm-up; -1 = m (fill the whole window)")
    ap.add_argument("--local-shards", type=int, default=0,
                    help="diagnostic: run the coordinate-sharded step with this many shards, all "
                         "on GPU 0 of this process")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-steps", type=int, default=5)
    ap.add_argument("--cpu-single-steps", type=int, default=2,
                    help="steps of the oracle's single-thread leg of the CPU baseline (0: skip)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        # rank 0 alone runs the oracle; no process group is needed for that
        run_reference(args, int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")))
        return
    if args.local_shards > 1:
        run_local_shards(args)
        return
    world, rank, local = dist_setup(args.gpus)

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback)")
    from paper_2306_06098_b200 import binding  # fails loudly when the library is missing

    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    w = get_workload(args.workload)
    K, W = args.steps, args.warmup
    gs = gradgen.GradStream(w.d, w.rank, w.seed + rank, w.scale_block, w.noise, str(device))
    acc = args.rhs == "accumulator"
    bf16 = args.values == "bf16"
    opt = binding.Efcp(w.d, w.m, w.k, w.lam,
                       (binding.RHS_ACCUMULATOR if acc else binding.RHS_COMPRESSED) |
                       (binding.VALUES_BF16 if bf16 else 0) |
                       (binding.PRECOND_GGT if args.precond == "ggt" else 0) |
                       (binding.LCG_FP32 if args.lcg == "fp32" else 0), args.block)
    if args.block:  # rows are a little longer than k: count the bytes of what is really kept
        w = gradgen.Workload(w.name, w.d, w.m, opt.k, w.lam, w.steps, w.rank, w.scale_block,
                             w.seed, w.noise)
    gbuf = torch.empty(w.d, dtype=torch.float32, device=device)
    ubuf = torch.empty(w.d, dtype=torch.float32, device=device)

    theta = torch.randn(w.d, dtype=torch.float32, device=device) if args.apply_update else None

    def one_step(g, stream=None):
        if theta is None:
            opt.step(g, ubuf, stream)
        else:
            opt.step_apply(g, theta, None if args.no_u else ubuf, 1e-3, 1e-4, args.clip, stream)

    prefill = w.m if args.prefill < 0 else args.prefill
    for _ in range(prefill):
        gs.next(out=gbuf)
        opt.step(gbuf, ubuf)
    torch.cuda.synchronize()
    assert opt.status() == 0, binding.strerror(opt.status())

    # inputs of the timed region: resident in HBM before it starts
    pool_n = min(K + W, 128)
    pool = [gs.next().clone() for _ in range(pool_n)]
    del gs  # frees U
    torch.cuda.empty_cache()

    for i in range(W):
        one_step(pool[i % pool_n])
    torch.cuda.synchronize()
    barrier(world)
    try:  # nvidia-smi numbering ignores CUDA_VISIBLE_DEVICES: address the GPU by UUID
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(local).uuid).replace("GPU-", "")
    except Exception:
        gpu_id = str(local)
    sampler = ClockSampler(gpu_id)
    sampler.start()
    time.sleep(0.3)
    stream = torch.cuda.current_stream()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    opt.profile_begin(K)
    torch.cuda.synchronize()
    ev0.record(stream)
    for i in range(K):
        one_step(pool[(W + i) % pool_n], stream)
    ev1.record(stream)
    torch.cuda.synchronize()
    barrier(world)
    clocks = sampler.stop()
    ms_total = max_over_ranks(ev0.elapsed_time(ev1), world, device)
    stages, n_rec = opt.profile_end()
    launches = opt.launches_per_step * K
    assert opt.status() == 0, binding.strerror(opt.status())
    ms_per_step = ms_total / K
    value = world * K / (ms_total * 1e-3)

    # end to end: host buffers, copies inside the timed region
    e2e = None
    if args.e2e_steps > 0:
        gh = torch.empty(w.d, dtype=torch.float32).pin_memory()
        uh = torch.empty(w.d, dtype=torch.float32).pin_memory()
        gh.copy_(pool[0])
        opt.step_host(gh, uh)  # allocates the staging buffers
        barrier(world)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for i in range(args.e2e_steps):
            opt.step_host(gh, uh)
        torch.cuda.synchronize()
        dt = max_over_ranks(time.perf_counter() - t0, world, device)
        e2e = {"value": world * args.e2e_steps / dt, "unit": UNIT,
               "h2d_bytes_per_step": 4 * w.d, "d2h_bytes_per_step": 4 * w.d,
               "steps": args.e2e_steps}

    # roofline of the dominant kernel (HBM bound): bytes per launch / its time.  The headline
    # figures (`achieved`, `frac`) count the bytes the kernel has to read and write as it is
    # built: a 16-bit slab-relative index and an fp32 (bf16) value per window entry, 6 (4) bytes,
    # plus the dense vectors.  `algorithmic` repeats them for the method's own (I, V) format
    # with int32 indices, 8 (6) bytes per entry, the count of the scope table; that figure can
    # exceed the peak because the kernel moves fewer bytes than it is credited with.
    # x = a_t adds one read of xi to SP and one to LCG.
    peak, peak_src = load_peak()
    mk = w.m * w.k
    xi_read = 4 * w.d if acc else 0
    val_b = 2 if bf16 else 4
    alg = {"sp": (4 + val_b) * mk + xi_read, "lcg": (4 + val_b) * mk + 4 * w.d + xi_read}
    mov = {"sp": (2 + val_b) * mk + xi_read, "lcg": (2 + val_b) * mk + 4 * w.d + xi_read}
    kern = max(("sp", "lcg"), key=lambda s: stages[s])
    avg_ms = stages[kern] / max(n_rec, 1)
    achieved_alg = alg[kern] / (avg_ms * 1e-3) / 1e9
    moved = mov[kern] / (avg_ms * 1e-3) / 1e9
    traffic = None
    if not (acc or bf16 or args.block or args.precond != "mfac" or
            (kern == "lcg" and (args.lcg != "fixed" or args.apply_update))):
        traffic = NCU_TRAFFIC_BYTES.get(w.name, {}).get(kern)
    roofline = {"bound": "hbm", "kernel": {"sp": "k_sp_rows", "lcg": "k_lcg"}[kern],
                "achieved": moved, "peak": peak, "unit": "GB/s", "frac": moved / peak,
                "bytes_per_launch": mov[kern],
                "traffic": traffic,
                "traffic_source": (None if traffic is None else
                                   "ncu dram bytes of a quarter-size capture scaled to a full "
                                   "launch (profiles/)"),
                "peak_source": peak_src, "avg_launch_ms": avg_ms,
                "algorithmic": {"bytes_per_launch": alg[kern], "achieved": achieved_alg,
                                "frac": achieved_alg / peak}}
    step_bytes = 2 * (4 + val_b) * mk + 16 * w.d + 8 * w.k + 2 * xi_read
    step_moved = 2 * (2 + val_b) * mk + 16 * w.d + 10 * w.k + 2 * xi_read
    if args.apply_update:  # theta read and written, u read; the norm reads u once more
        extra = (4 * w.d if args.no_u else 12 * w.d) + (4 * w.d if args.clip > 0 else 0)
        step_bytes += extra
        step_moved += extra
    step_gbs = step_bytes / (ms_per_step * 1e-3) / 1e9
    step_moved_gbs = step_moved / (ms_per_step * 1e-3) / 1e9
    stage_ms = {s: stages[s] / max(n_rec, 1) for s in stages}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and args.cpu_steps > 0:
        grads_host = [pool[i].cpu().numpy() for i in range(min(2, pool_n))]
        timed = oracle_steps_per_sec(w, grads_host, args.cpu_steps, args.precond)
        if timed is not None:
            v, cores, dt = timed
            cpu_baseline = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                            "sample": f"{args.cpu_steps} full steps of {w.name} from an empty "
                                      f"window (the oracle loops over all m rows whether written "
                                      f"or not), {dt:.1f} s"}
            if args.cpu_single_steps > 0:
                v1, c1, dt1 = oracle_steps_per_sec(w, grads_host, args.cpu_single_steps,
                                                   args.precond, threads=1)
                cpu_baseline["single_thread"] = {
                    "value": v1, "unit": UNIT, "cores": c1,
                    "sample": f"{args.cpu_single_steps} full steps, {dt1:.1f} s"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": W, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "d": w.d, "m": w.m, "k": w.k, "lambda": w.lam,
                       "rhs": args.rhs, "window_values": args.values,
                       "lcg_accumulator": ("int32 fixed point, fp32 fallback per slab (%d slabs "
                                           "fell back)" % opt.fixed_point_fallbacks()
                                           if args.lcg == "fixed" and not acc else "fp32"),
                       "preconditioner": {"mfac": "Sparse M-FAC", "ggt": "Sparse GGT"}[args.precond],
                       "topk": f"blockwise({args.block})" if args.block else "global",
                       "prefill_steps": prefill,
                       "parameter_update": (f"efcp_step_apply (eta 1e-3, gamma 1e-4, clip "
                                            f"{args.clip:g}{', u not materialised' if args.no_u else ''})"
                                            if args.apply_update else "none"),
                       "parallelism": f"replicas x{world}",
                       "l2": "inputs larger than L2 (window %.2f GB, gradient %.2f GB)" % (
                           8 * w.m * w.k / 1e9, 4 * w.d / 1e9)},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
            "roofline": roofline,
            "step_hbm": {"bytes_per_step": step_moved, "achieved_gbs": step_moved_gbs,
                         "frac_of_peak": step_moved_gbs / peak,
                         "frac_of_8tbs": step_moved_gbs / 8000.0,
                         "algorithmic": {"bytes_per_step": step_bytes, "achieved_gbs": step_gbs,
                                         "frac_of_peak": step_gbs / peak,
                                         "frac_of_8tbs": step_gbs / 8000.0}},
            "stage_ms": stage_ms,
            "cpu_baseline": cpu_baseline,
        }
        print(json.dumps(line), flush=True)
    opt.close()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
