#!/usr/bin/env python
"""Benchmark of the CD-Adam step (Algorithm 1, all stages) on synthetic gradients.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C4] [--impl cdadam|reference]

A "step" is one call of cdadam_step: worker stage for all n workers, server stage and the
worker-side AMSGrad update.  The default workload is C4 (d = 110,000,000, n = 8 workers,
scaled sign per tensor, heavy-tailed gradients); C1..C5 can be chosen with --workload.
The path is pinned to one GPU and does not shard: with --gpus N every rank runs an
independent replica of the same problem ("replicas only"), value is the sum over ranks.

Prints one JSON line (rank 0).  `value` is steps/s with the gradients already resident in
device memory; `e2e` is the same through cdadam_step_host with pinned HOST gradients, the
host->device copy of n*d floats and the device->host copy of x inside the timed region.
The timed region is R blocks of exactly K steps (R >= 5 and enough for about a second in
all); `ms_per_step` and `value` come from the median block, `repeats` gives the spread.
`roofline` is for the dominant kernel (the worker pass), timed with CUDA events recorded by
the library on the launching stream in a separate pass of the same K steps.  The default
run (C4, one GPU) then times C5, C3 and C2 the same way and reports them in
`other_workloads`; C4 stays the headline.
`--impl reference` times the CPU oracle (tests/-only code, as it stands, one core) on a
bounded sample of the same workload.
"""
import argparse
import hashlib
import re
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "compressed-AMSGrad steps/s"
UNIT = "steps/s"
FALLBACK_HBM_GBS = 6650.0

# ncu capture of the dominant kernel: dram__bytes_read.sum + dram__bytes_write.sum per launch,
# keyed by workload, with the hash of the kernel sources at capture time.  A changed source
# makes the figure stale and bench reports null.
NCU_TRAFFIC = {
    # k_worker_sign_ring: 2.673 GB measured on C4 scaled by 0.25 (same tile), x4 by the units
    "C4": {"hash": "43a020d7013fe046", "bytes_per_launch": 4 * (1.814689e+09 + 8.5882368e+08),
           "note": "extrapolated from an ncu capture of the same kernel on the workload scaled by 0.25 "
                   "(same tile and kernel variant), multiplied by 4: traffic is proportional to n*d"},
}


def kernel_source_hash():
    """Hash of the kernel sources without comments and blank space (a reworded comment does
    not make the captured counters stale; any change of code does)."""
    h = hashlib.sha256()
    for f in ("common.cuh", "sign_kernels.cu"):
        with open(os.path.join(ROOT, "paper_2111_00705_b200", "csrc", f), "r") as fh:
            src = fh.read()
        src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
        src = re.sub(r"//[^\n]*", "", src)
        h.update("".join(src.split()).encode())
    return h.hexdigest()[:16]


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def algorithmic_bytes(w, bf16=False):
    """Bytes Algorithm 1 must move per step with every vector touched once.
    scaled sign: worker 4 (g) + 8 (ghat r/w) + 1/8 (bits) per worker element; server and
    update n/8 + 48.25 per element.  top-k: 8 per worker element + 44 per element."""
    from paper_2111_00705_b200 import synth
    if w.compressor == synth.SIGN:
        gb = 2.0 if bf16 else 4.0
        return w.d * ((8.25 + gb) * w.n + 48.25), w.n * w.d * (8.125 + gb)
    if w.compressor == synth.TOPK:
        return w.d * (8.0 * w.n + 44.0), w.n * w.d * 8.0
    if w.compressor == synth.RANDK:      # sparse: 3 sectors-worth of floats per kept entry + dense AMSGrad
        return w.d * 36.0 + (w.n + 1) * w.k * 20.0, w.d * 36.0
    return w.d * (12.0 * w.n + 48.0), w.d * (12.0 * w.n + 48.0)


class ClockSampler:
    """nvidia-smi samples of SM clock and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "20"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush(); self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.f:
            parts = [s.strip() for s in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons),
                       samples=len(sm))
        return out


def oracle_sample(w, frac, steps):
    """Time the CPU oracle on the first `frac` of the coordinates (same recipe) for `steps`
    steps; returns seconds per step of the sample and the sample workload."""
    import oracle as orc
    from paper_2111_00705_b200 import synth
    ws = synth.workload(w.name, scale=frac) if frac < 1.0 else w
    o = orc.Oracle(ws.d, ws.n, ws.compressor, k=ws.k, offsets=ws.offsets, x0=ws.x0("cpu").numpy(),
                   beta1=ws.beta1, beta2=ws.beta2, lr=ws.lr, eps=ws.eps)
    grads = [ws.grads(t, "cpu").numpy() for t in (1, 2)]
    t0 = time.perf_counter()
    for t in range(steps):
        o.step(grads[t % 2])
    dt = (time.perf_counter() - t0) / steps
    o.close()
    return dt, ws


SAMPLE = {"C1": (1.0, 20), "C2": (0.25, 4), "C3": (0.01, 4), "C4": (0.1, 5), "C5": (0.01, 5)}


def run_reference(args, rank):
    """The oracle, as it stands, on the host cores (rank 0 only)."""
    if rank != 0:
        return
    from paper_2111_00705_b200 import synth
    w = synth.workload(args.workload)
    frac, sample_steps = SAMPLE[w.name]
    for _ in range(args.warmup and 1):
        oracle_sample(w, frac, 1)
    times = []
    for _ in range(args.steps):
        dt, ws = oracle_sample(w, frac, sample_steps)
        times.append(dt)
    sec_full = statistics.mean(times) / frac          # cost is linear in d
    value = 1.0 / sec_full
    sample = "first %g of the coordinates (d=%d, same recipe, n=%d), %d oracle steps per bench step; " \
             "seconds per step scaled by 1/%g" % (frac, ws.d, ws.n, sample_steps, frac)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec_full * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "params_per_s": value * w.d,
            "config": {"workload": describe(w), "replicas": 1, "l2": l2_note(w)},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def max_over_ranks_ms(ms, device):
    """Device time of a region on this rank -> the maximum over all ranks (N = 1: itself)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replicas_throughput(world, steps, total_ms):
    """N independent replicas ("replicas only"): units all ranks processed over the slowest
    rank's time."""
    return world * steps / (total_ms * 1e-3)


def run_distributed(args, w, dev, rank, world):
    """The distributed deployment (one process per GPU, each with its share of the n workers,
    messages over NCCL): device-timed K iterations, max over ranks.  Total work is fixed as N
    grows, so scaling is "strong".  Rank 0 prints one JSON line."""
    import torch
    import torch.distributed as dist
    from paper_2111_00705_b200 import distributed as dd
    from paper_2111_00705_b200 import synth
    if w.compressor not in (synth.SIGN, synth.TOPK):
        raise SystemExit("--layout %s: the distributed deployment takes the scaled-sign and top-k workloads" % args.layout)
    if not dist.is_initialized():                      # a single process: a group of one
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", str(29000 + os.getpid() % 2000))
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=dev)
    args.warmup = max(args.warmup, 3)
    if args.layout == "range":
        run_range(args, w, dev, rank, world)
        dist.destroy_process_group()
        return
    server_rank = 0 if args.layout == "server" else None
    opt = dd.DistributedCDAdam(w.d, w.n, None, server_rank, beta1=w.beta1, beta2=w.beta2, lr=w.lr, eps=w.eps,
                               offsets=w.offsets, x0=w.x0(dev), device=dev, compressor=w.compressor, k=w.k)
    first, per = dd.partition(w.n, world, rank, server_rank)
    grads = [w.grads(t + 1, dev).reshape(w.n, w.d)[first:first + per].contiguous().reshape(-1) if per else None
             for t in range(2)]
    stream = torch.cuda.current_stream()
    for t in range(args.warmup):
        opt.step(grads[t % 2])
    dist.barrier(); torch.cuda.synchronize()
    sampler = ClockSampler(dev.index) if rank == 0 else None
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for t in range(args.steps):
        opt.step(grads[t % 2])
    b.record(stream)
    dist.barrier(); torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else None
    total_ms = max_over_ranks_ms(a.elapsed_time(b), dev)
    opt.shard.device_status()
    value = args.steps / (total_ms * 1e-3)
    words = (w.d + 31) // 32
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": describe(w), "layout": args.layout, "workers_per_rank": per,
                       "l2": "inputs larger than L2" if per * w.d * 4 >= 2 * 126e6 else "not flushed"},
            "params_per_s": value * w.d,
            "message_bytes_per_worker": words * 4 + 4 * w.q if w.compressor == synth.SIGN else 8 * w.k,
            "gpu_launches": opt.shard.launches_per_step() * args.steps, "clocks": clocks}))
    opt.close()
    dist.destroy_process_group()


def run_range(args, w, dev, rank, world):
    """The coordinate-sharded deployment: every process owns d / N coordinates of all n workers
    and of the server; the l1 parts (scaled sign) or the histograms and tie counts (top-k) are
    all-gathered.  Strong scaling.  With --of-ranges R on ONE process the context is range 0 of
    R: the time of one rank's share, its gathers being one-rank collectives - a projection of
    the N = R step without the latency of R-rank collectives, said so in the line."""
    import torch
    import torch.distributed as dist
    from paper_2111_00705_b200 import binding as cd
    from paper_2111_00705_b200 import distributed as dd
    ranges = args.of_ranges if (world == 1 and args.of_ranges > 1) else world
    lo, hi = dd.range_partition(w.d, ranges, rank)
    if ranges != world:
        opt = dd.RangeShardedCDAdam.__new__(dd.RangeShardedCDAdam)
        opt.group, opt.world, opt.rank, opt.lo, opt.hi = None, 1, 0, lo, hi
        opt.range = cd.CDAdamRange(w.d, w.n, lo, hi, 0, ranges, beta1=w.beta1, beta2=w.beta2, lr=w.lr, eps=w.eps,
                                   offsets=w.offsets, x0=w.x0(dev)[lo:hi].contiguous(), device=dev,
                                   compressor=w.compressor, k=w.k)
    else:
        opt = dd.RangeShardedCDAdam(w.d, w.n, offsets=w.offsets, x0=w.x0(dev)[lo:hi].contiguous(), beta1=w.beta1,
                                    beta2=w.beta2, lr=w.lr, eps=w.eps, device=dev, compressor=w.compressor, k=w.k)
    grads = [w.grads(t + 1, dev).reshape(w.n, w.d)[:, lo:hi].contiguous().reshape(-1) for t in range(2)]
    stream = torch.cuda.current_stream()

    def step(t):
        if ranges == world:
            opt.step(grads[t % 2])
            return
        r = opt.range                                  # one range of several: its gathers stay on this process
        if r.compressor == cd.TOPK:
            for stage in range(r.TOPK_STAGES):
                r.range_topk(stage, grads[t % 2] if stage <= 4 else None)
                buf = r.range_topk_buffer(stage)
                if buf is not None:
                    dist.all_gather_into_tensor(buf[0], buf[0].clone())
        else:
            r.range_workers(grads[t % 2])
            b = r.range_buffers()["worker_sums"]; dist.all_gather_into_tensor(b[0].view(-1), b[0].reshape(-1).clone())
            r.range_server()
            b = r.range_buffers()["server_sums"]; dist.all_gather_into_tensor(b[0].view(-1), b[0].reshape(-1).clone())
            r.range_update()

    for t in range(args.warmup):
        step(t)
    dist.barrier(); torch.cuda.synchronize()
    sampler = ClockSampler(dev.index) if rank == 0 else None
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for t in range(args.steps):
        step(t)
    b.record(stream)
    dist.barrier(); torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else None
    total_ms = max_over_ranks_ms(a.elapsed_time(b), dev)
    opt.range.device_status()
    value = args.steps / (total_ms * 1e-3)
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": describe(w), "layout": "range", "ranges": ranges,
                       "coordinates_per_rank": hi - lo,
                       "projection": None if ranges == world else
                       "one process timed as range 0 of %d (its share of the work, one-rank gathers): "
                       "not a %d-GPU measurement" % (ranges, ranges)},
            "params_per_s": value * w.d,
            "gpu_launches": opt.range.launches_per_step() * args.steps, "clocks": clocks}))
    opt.close()


def l2_small(w):
    return w.n * w.d * 4 < 2 * 126e6


def l2_note(w):
    """How the timed steps are kept from finding their inputs in L2 (the GPU arm's protocol)."""
    return ("flushed between steps" if l2_small(w) else
            "inputs larger than L2 (%.2f GB of gradients per step)" % (w.n * w.d * 4 / 1e9))


def describe(w):
    from paper_2111_00705_b200 import synth
    comp = {synth.SIGN: "scaled-sign", synth.TOPK: "top-k k=%d" % w.k, synth.IDENTITY: "identity",
            synth.RANDK: "rand-k k=%d" % w.k}[w.compressor]
    return "%s d=%d n=%d %s q=%d %s fp32" % (w.name, w.d, w.n, comp, w.q, w.dist)


def run_workload(args, w, dev, rank, world, barrier, headline):
    """Times one workload on this rank's GPU: W warm-up steps, then R repeats of a block of
    exactly K steps (device time per block, max over ranks; R >= 5 and enough for the timed
    region to last about a second), the clock sampler running from before the warm-up to
    after the last repeat; then a per-kernel pass for the roofline of the dominant kernel.
    The headline workload also gets the end-to-end leg through the host-buffer entry point."""
    import torch
    from paper_2111_00705_b200 import binding as cd
    from paper_2111_00705_b200 import synth

    opt = cd.CDAdam(w.d, w.n, w.compressor, k=w.k, offsets=w.offsets, x0=w.x0(dev),
                    beta1=w.beta1, beta2=w.beta2, lr=w.lr, eps=w.eps, device=dev,
                    mode={"markov": cd.MARKOV, "ef": cd.EF, "naive": cd.NAIVE}[args.mode])
    if args.tile:
        opt.set_tile(args.tile)
    if w.compressor == synth.RANDK:      # the draws are inputs; one set of draws serves all steps
        import numpy as np
        opt.set_random_sets(torch.from_numpy(synth.random_sets(w.d, w.k, w.n, w.seed, 1).view(np.int32)).to(dev),
                            torch.from_numpy(synth.random_sets(w.d, w.k, 1, w.seed + 1, 1)[0].view(np.int32)).to(dev))
    # two gradient sets, alternated; each is far larger than L2 except for C1, where L2 is
    # flushed between steps instead
    nbuf = 2 if w.n * w.d * 4 * 2 < 60e9 else 1
    grads = [w.grads(t + 1, dev).reshape(-1) for t in range(nbuf)]
    bf16 = headline and args.grads == "bf16"
    step = opt.step
    if bf16:
        grads = [g.to(torch.bfloat16) for g in grads]
        step = opt.step_bf16
    # L2 holds 126 MB.  A step whose gradients alone are at least twice that (and whose worker
    # state is as large again) cannot find its inputs there; smaller workloads get the flush.
    small = l2_small(w)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if small else None
    stream = torch.cuda.current_stream()
    K = args.steps

    def block():
        """K steps; returns the device milliseconds spent in the steps (flushes not counted)."""
        if flush is None:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for t in range(K):
                step(grads[t % nbuf], stream)
            b.record(stream)
            return [(a, b)]
        pairs = []
        for t in range(K):              # time each step alone so that the L2 flush is not counted
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); step(grads[t % nbuf], stream); b.record(stream)
            pairs.append((a, b))
        return pairs

    barrier()
    sampler = ClockSampler(dev.index) if rank == 0 else None     # runs from here to the last repeat
    for t in range(args.warmup):
        if flush is not None:
            flush.zero_()
        step(grads[t % nbuf], stream)
    barrier()
    probe = block()                      # one untimed block sizes the number of repeats
    barrier()
    est_ms = max(sum(a.elapsed_time(b) for a, b in probe), 1e-3)
    repeats = args.repeats if args.repeats > 0 else int(min(400, max(5, -(-args.region_ms // est_ms))))

    # ---- timed region: R blocks of K steps, device time per block, max over ranks --------
    blocks = []
    barrier()
    for r in range(repeats):
        blocks.append(block())
        if flush is not None or r % 8 == 7:
            barrier()                    # bound the queue depth (events, flushes)
    barrier()
    block_ms = [sum(a.elapsed_time(b) for a, b in pairs) for pairs in blocks]
    block_ms = max_over_ranks_list(block_ms, dev)
    clocks = sampler.stop() if sampler else None
    med = statistics.median(block_ms)
    ms_per_step = med / K
    if clocks and clocks.get("sm_mhz"):
        clocks["ms_per_step_x_sm_mhz"] = ms_per_step * clocks["sm_mhz"]

    # ---- per-kernel pass for the roofline ------------------------------------------------
    opt.profile_enable(True)
    for t in range(K):
        if flush is not None:
            flush.zero_()
        step(grads[t % nbuf], stream)
    stage_ms, psteps = opt.profile_read()
    opt.profile_enable(False)
    stage_ms = {k: v / max(psteps, 1) for k, v in stage_ms.items()}
    step_bytes, dom_bytes = algorithmic_bytes(w, bf16)
    dom_name = max(stage_ms, key=stage_ms.get)
    peak, peak_kind = measured_peak()
    achieved = dom_bytes / (stage_ms[dom_name] * 1e-3) / 1e9 if stage_ms[dom_name] > 0 else 0.0
    traffic = traffic_note = None
    cap = NCU_TRAFFIC.get(w.name)
    if cap and cap.get("hash") == kernel_source_hash() and not bf16 and args.mode == "markov":
        traffic = cap["bytes_per_launch"]
        traffic_note = cap["note"]
    roofline = {"bound": "hbm", "kernel": dom_name, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_source": "%s copy bandwidth" % peak_kind,
                "traffic": traffic, "traffic_source": traffic_note,
                "algorithmic_bytes_per_launch": dom_bytes,
                "ms_per_launch": stage_ms[dom_name],
                "timed": "separate pass of the same %d steps with events around every kernel" % K}

    # ---- end to end: host gradients in, x out, copies inside the timed region ------------
    e2e = None
    if headline:
        try:
            if args.e2e_steps < 1:
                raise RuntimeError("skipped (--e2e-steps 0)")
            if bf16:
                raise RuntimeError("skipped (host path takes binary32 gradients)")
            gh = [g.cpu().pin_memory() for g in grads[:1]]
            xh = torch.empty(w.d, dtype=torch.float32).pin_memory()
            opt.step_host(gh[0], xh, stream)                       # allocates the staging buffer
            barrier()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for t in range(args.e2e_steps):
                opt.step_host(gh[0], xh, stream)
            b.record(stream)
            barrier()
            e_ms = max_over_ranks_ms(a.elapsed_time(b), dev)
            e2e = {"value": replicas_throughput(world, args.e2e_steps, e_ms), "unit": UNIT,
                   "h2d_bytes_per_step": w.n * w.d * 4, "d2h_bytes_per_step": w.d * 4,
                   "steps": args.e2e_steps}
            del gh, xh
        except Exception as exc:                                   # e.g. not enough pinned memory
            e2e = {"value": None, "unit": UNIT, "error": str(exc)[:200]}

    launches = opt.launches_per_step() * K * repeats
    opt.device_status()          # raises if a kernel reported a bounded wait that ran out
    opt.close()
    del grads, flush
    torch.cuda.empty_cache()
    gbs = step_bytes / (ms_per_step * 1e-3) / 1e9
    return {"workload": describe(w), "ms_per_step": ms_per_step,
            "value": replicas_throughput(world, K, med),
            "repeats": {"count": repeats, "steps_per_repeat": K, "statistic": "median",
                        "ms_per_step_min": min(block_ms) / K, "ms_per_step_max": max(block_ms) / K,
                        "timed_region_ms": sum(block_ms)},
            "l2": l2_note(w),
            "step_hbm": {"algorithmic_bytes": step_bytes, "gbs": gbs, "frac_of_8tbs": gbs / 8e3,
                         "frac_of_measured": gbs / peak},
            "stage_ms": stage_ms, "roofline": roofline, "e2e": e2e, "gpu_launches": launches,
            "clocks": clocks}


def max_over_ranks_list(ms_list, device):
    """Per-block device times of this rank -> elementwise maximum over all ranks."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1):
        return list(ms_list)
    t = torch.tensor(ms_list, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="C4")
    ap.add_argument("--impl", default="cdadam", choices=["cdadam", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--repeats", type=int, default=0,
                    help="blocks of --steps steps that are timed (the median is reported); 0 = at least 5 "
                         "and enough for the timed region to last --region-ms")
    ap.add_argument("--region-ms", type=float, default=1200.0,
                    help="minimum total length of the timed region when --repeats is 0")
    ap.add_argument("--others", default="auto", choices=["auto", "on", "off"],
                    help="after the headline workload, also time C5, C3 and C2 and report them in "
                         "`other_workloads` (auto: on for the default C4 run on one GPU)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--compressor", default=None, choices=[None, "randk"],
                    help="randk: run the workload's shapes with the rand-k compressor (k as in C3: d/100)")
    ap.add_argument("--grads", default="f32", choices=["f32", "bf16"],
                    help="bf16: gradients given in bfloat16 through cdadam_step_bf16 (not the headline config)")
    ap.add_argument("--mode", default="markov", choices=["markov", "ef", "naive"],
                    help="markov = Algorithm 1 (default); ef = classical error feedback, naive = naive "
                         "compression (the comparison schemes of Section 4; their bytes differ, so the "
                         "roofline figures of such a run are not the headline's)")
    ap.add_argument("--of-ranges", type=int, default=0,
                    help="--layout range on one process: time range 0 of this many ranges (a projection)")
    ap.add_argument("--layout", default="replicas", choices=["replicas", "sharded", "server", "range"],
                    help="replicas (default): every rank runs the whole n-worker problem on its own.  "
                         "sharded: the distributed deployment, n/N workers per rank, worker messages "
                         "all-gathered over NCCL, server stage computed on every rank (scaled sign only; "
                         "strong scaling).  server: rank 0 is the server and holds no worker (N >= 2).  "
                         "range: the coordinate-sharded deployment, d/N coordinates of all workers per rank, "
                         "only the l1 parts / top-k histograms gathered")
    ap.add_argument("--tile", type=int, default=0,
                    help="force the kernels' tile size (profiler captures of scaled-down cases)")
    ap.add_argument("--scale", type=float, default=1.0,
                    help="shrink d (same recipe) for profiler captures; not a bench line")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2111_00705_b200 import synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    w = synth.workload(args.workload, scale=args.scale)
    if args.layout != "replicas":
        run_distributed(args, w, dev, rank, world)
        return
    if args.compressor == "randk":
        w.compressor, w.k, w.offsets = synth.RANDK, max(1, w.d // 100), None
    if args.warmup < 3:
        args.warmup = 3
    head = run_workload(args, w, dev, rank, world, barrier, True)

    # the other full-size configurations, same protocol, shorter record
    others = None
    plain = (args.scale == 1.0 and args.mode == "markov" and args.grads == "f32" and not args.compressor
             and not args.tile)
    if args.others == "on" or (args.others == "auto" and world == 1 and w.name == "C4" and plain):
        others = {}
        for name in ("C5", "C3", "C2"):
            if name == w.name:
                continue
            try:
                r = run_workload(args, synth.workload(name), dev, rank, world, barrier, False)
                rf = r["roofline"]
                others[name] = {"workload": r["workload"], "ms_per_step": r["ms_per_step"],
                                "steps_per_s": r["value"], "repeats": r["repeats"], "l2": r["l2"],
                                "algorithmic_gbs": r["step_hbm"]["gbs"],
                                "frac_of_8tbs": r["step_hbm"]["frac_of_8tbs"],
                                "frac_of_measured": r["step_hbm"]["frac_of_measured"],
                                "stage_ms": r["stage_ms"],
                                "dominant": {"kernel": rf["kernel"], "ms_per_launch": rf["ms_per_launch"],
                                             "achieved_gbs": rf["achieved"], "frac_of_measured": rf["frac"]},
                                "gpu_launches": r["gpu_launches"], "clocks": r["clocks"]}
            except Exception as exc:                               # e.g. the device is too small for C5
                others[name] = {"error": str(exc)[:200]}
                torch.cuda.empty_cache()

    cpu = None
    if rank == 0 and not args.no_cpu_baseline:
        frac, sample_steps = SAMPLE[w.name]
        dt, ws = oracle_sample(w, frac, sample_steps)
        cpu = {"value": frac / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
               "host_cores": os.cpu_count(),
               "sample": "first %g of the coordinates (d=%d, same recipe, n=%d), %d steps; "
                         "seconds per step scaled by 1/%g" % (frac, ws.d, ws.n, sample_steps, frac)}

    if rank == 0:
        line = {"metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": head["workload"] + ("" if args.scale == 1.0 else " (scaled by %g)" % args.scale)
                           + {"markov": "", "ef": " [error-feedback mode]", "naive": " [naive-compression mode]"}[args.mode]
                           + ("" if args.grads == "f32" else " [bf16 gradients]"),
                           "replicas": world, "l2": head["l2"]},
                "repeats": head["repeats"],
                "params_per_s": head["value"] * w.d,
                "step_hbm": head["step_hbm"], "stage_ms": head["stage_ms"],
                "roofline": head["roofline"], "cpu_baseline": cpu, "e2e": head["e2e"],
                "gpu_launches": head["gpu_launches"], "clocks": head["clocks"],
                "other_workloads": others}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
