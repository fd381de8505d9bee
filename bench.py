#!/usr/bin/env python
"""Benchmark of the five streaming kernels (copy, scale, add, triad, dot) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl ours|reference]

One step = one pass of all five kernels over the three arrays of the workload, in the STREAM
dataflow (c <- a; b <- s*c; c <- a+b; a <- b+s*c; dot(a, b)). The line printed by rank 0 reports
the whole-job algorithmic GB/s of the step, the GB/s of each kernel from CUDA events recorded
around every launch inside the timed region, the end-to-end figure through the host-buffer
entry point, and the CPU oracle timed on the host cores beside it.

With N > 1 (launched by torchrun, one rank per GPU) every rank runs its own replica of the
workload: the kernels are independent per index, so the path shards with no data-path
collective; the only communication is the barrier and the MAX/SUM of the timings.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "HBM GB/s over the five stream ops (copy/scale/add/triad/dot), algorithmic bytes"
UNIT = "GB/s"

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel from
# an ncu capture, keyed by (workload, op, tuning signature); absent = not captured for this build.
NCU_TRAFFIC_BYTES: dict = {
    # profiles/ncu_chain_dram_c2_fp64.md (L2 state kept between kernels, as in the timed loop):
    # add reads 465.9 MB + writes 272.9 MB; triad reads 464.1 MB + writes 266.6 MB per launch
    ("c2", "add", '{"blocks_per_sm": 0, "chunk_bytes": 16384, "compensated": 0, "contiguous": 0, "keep_mib": 112, "kind": 0, "pdl": 1, '
                  '"policy": 7, "reverse": 2, "stages": 4, "threads": 128, "two_pass": 0, "unroll": 2, "vec_bytes": 32}'): 738_800_000,
    ("c2", "triad", '{"blocks_per_sm": 0, "chunk_bytes": 16384, "compensated": 0, "contiguous": 0, "keep_mib": 112, "kind": 0, "pdl": 1, '
                    '"policy": 7, "reverse": 2, "stages": 4, "threads": 128, "two_pass": 0, "unroll": 2, "vec_bytes": 32}'): 730_700_000,
}


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=200)
    p.add_argument("--warmup", type=int, default=10)
    p.add_argument("--workload", default="c2", choices=["c1", "c2", "c3", "c4"])
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--e2e-steps", type=int, default=5)
    p.add_argument("--tuning", default="",
                   help='JSON overrides of the launch tuning for A/B runs, e.g. \'{"ew": {"policy": 5}, "dot": {"two_pass": 1}}\' '
                        '("ew" = copy, scale, add, triad; "all" = the five ops)')
    p.add_argument("--no-shmem", action="store_true", help="skip the shared-memory microkernel line")
    p.add_argument("--cpu-seconds", type=float, default=12.0,
                   help="CPU time budget of the oracle baseline leg (0 = skip)")
    return p.parse_args()


def tuning_signature(so, dtype):
    return {op: so.get_tuning(op, dtype).as_dict() for op in so.OPS}


# ------------------------------------------------------------------------------- oracle legs
def time_oracle(w, seconds: float, nthreads: int):
    """Times the CPU oracle, as it stands, on passes of all five kernels over the workload's
    arrays (full length) until `seconds` of wall time are used. Returns (GB/s all-threads form,
    GB/s single thread, passes, description)."""
    import oracle
    from paper_2510_00932_b200 import harness, inputs
    a, b, c = inputs.make_arrays(w)
    nbytes = harness.step_bytes(w.n, w.itemsize)

    def one_pass(nt):
        t0 = time.perf_counter()
        if nt == 1:
            oracle.chain(a, b, c, w.scalar)
        else:
            cc = oracle.run_mt("copy", a, None, 0.0, nt)
            bb = oracle.run_mt("scale", cc, None, w.scalar, nt)
            cc = oracle.run_mt("add", a, bb, 0.0, nt)
            aa = oracle.run_mt("triad", bb, cc, w.scalar, nt)
            oracle.run_mt("dot", aa, bb, 0.0, nt)
        return time.perf_counter() - t0

    one_pass(nthreads)                                   # page in, warm up
    mt, t_end = [], time.perf_counter() + seconds * 0.6
    while not mt or time.perf_counter() < t_end:
        mt.append(one_pass(nthreads))
    st, t_end = [], time.perf_counter() + seconds * 0.4
    while not st or time.perf_counter() < t_end:
        st.append(one_pass(1))
    desc = (f"{len(mt)} all-thread + {len(st)} single-thread passes of the five kernels over the "
            f"full {w.name} arrays ({w.dtype}, n={w.n})")
    return nbytes / statistics.median(mt) / 1e9, nbytes / statistics.median(st) / 1e9, len(mt), desc


def run_reference(args):
    """The reference arm: the CPU oracle on the host cores, same metric and workload."""
    from paper_2510_00932_b200 import harness, inputs
    rank, _, world = harness.dist_env()
    if rank != 0:
        return 0
    import oracle
    w = inputs.WORKLOADS[args.workload]
    nthreads = len(os.sched_getaffinity(0))
    # a bounded sample: shrink n until steps+warmup passes fit in about two minutes
    n = w.n
    a, b, c = inputs.make_arrays(w, n)
    t0 = time.perf_counter(); oracle.chain(a, b, c, w.scalar); t1 = time.perf_counter() - t0
    budget = 120.0
    while n > (1 << 16) and t1 * (n / w.n) * (args.steps + args.warmup) > budget * nthreads * 0.5:
        n //= 2
    if n != w.n:
        a, b, c = inputs.make_arrays(w, n)

    def step():
        cc = oracle.run_mt("copy", a, None, 0.0, nthreads)
        bb = oracle.run_mt("scale", cc, None, w.scalar, nthreads)
        cc = oracle.run_mt("add", a, bb, 0.0, nthreads)
        aa = oracle.run_mt("triad", bb, cc, w.scalar, nthreads)
        oracle.run_mt("dot", aa, bb, 0.0, nthreads)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    elapsed = time.perf_counter() - t0
    ms = elapsed / args.steps * 1e3
    gbs = harness.step_bytes(n, w.itemsize) / (ms * 1e-3) / 1e9
    sample = f"each step = the five kernels over n={n} of {w.name}'s {w.n} elements, all-threads oracle"
    line = {
        "impl": "reference", "metric": METRIC, "value": round(gbs, 3), "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms, 4), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "n": w.n, "sample_n": n, "dist": w.dist, "seed": w.seed, "scalar": w.scalar},
        "cpu_baseline": {"value": round(gbs, 3), "unit": UNIT, "cores": nthreads, "kind": "oracle", "sample": sample},
        "e2e": {"value": round(gbs, 3), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# ------------------------------------------------------------------------------- the CUDA arm
def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2510_00932_b200 import harness, inputs
    from paper_2510_00932_b200 import streamops as so

    rank, local_rank, world = harness.dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    so.lib()                                             # fail loudly if the library is not built
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    so.init(local_rank)

    w = inputs.WORKLOADS[args.workload]
    for key, fields in (json.loads(args.tuning) if args.tuning else {}).items():
        for op in {"ew": so.OPS[:4], "all": so.OPS}.get(key, (key,)):
            so.set_tuning(op, w.dtype, **fields)
    # every rank works on its own replica of the workload (same recipe, rank-specific seed)
    wr = inputs.Workload(w.name, w.dtype, w.n, w.dist, w.seed + 1000 * rank, w.scalar, w.iterations)
    a, b, c = inputs.make_arrays(wr)
    pinned = [torch.from_numpy(v).pin_memory() for v in (a, b, c)]
    da, db, dc = (p.to(device, non_blocking=False) for p in pinned)
    dd = torch.zeros(1, dtype=da.dtype, device=device)
    stream = torch.cuda.current_stream(device)
    n, itemsize = w.n, w.itemsize
    calls = [("copy", lambda: so.copy(da, dc)), ("scale", lambda: so.scale(dc, db, w.scalar)),
             ("add", lambda: so.add(da, db, dc)), ("triad", lambda: so.triad(db, dc, da, w.scalar)),
             ("dot", lambda: so.dot(da, db, dd))]

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(device)

    # fp32 with s = 3.0 grows a by 15x per chain step and overflows after ~33 steps: bound the
    # chained steps per region and start every region from the seeded arrays
    chain_cap = 25 if (w.dtype == "f32" and abs(w.scalar) > 1.0) else None

    def reseed():
        if chain_cap is not None:
            for dst, src in zip((da, db, dc), pinned):
                dst.copy_(src, non_blocking=False)

    warm = max(args.warmup, 3) if chain_cap is None else 3
    for _ in range(warm):
        for _, f in calls:
            f()
    reseed()
    barrier()

    # timed region 1: K chain steps back to back, one event pair around all of them -> `value`
    sampler = harness.ClockSampler(gpu_index=local_rank).start() if rank == 0 else None
    time.sleep(0.3 if sampler else 0.0)
    K = args.steps if chain_cap is None else min(args.steps, chain_cap)
    launches0 = so.launch_count()
    e_begin, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    first = sampler.mark() if sampler else 0
    e_begin.record(stream)
    for k in range(K):
        for _, f in calls:
            f()
    e_end.record(stream)
    barrier()
    elapsed_ms = e_begin.elapsed_time(e_end)
    launches = so.launch_count() - launches0             # kernels launched inside region 1

    reseed()
    barrier()
    # timed region 2: K more chain steps with an event before every launch -> per-kernel durations
    # in chain order (the extra events cost ~2 us per launch, which is why region 1 has none)
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(len(calls) + 1)] for _ in range(K)]
    for k in range(K):
        for i, (_, f) in enumerate(calls):
            events[k][i].record(stream)
            f()
        events[k][-1].record(stream)
    barrier()
    last = sampler.mark() if sampler else 0
    so.check()
    op_ms = {name: statistics.fmean(events[k][i].elapsed_time(events[k][i + 1]) for k in range(K))
             for i, (name, _) in enumerate(calls)}
    op_ms_best = {name: min(events[k][i].elapsed_time(events[k][i + 1]) for k in range(K))
                  for i, (name, _) in enumerate(calls)}
    # sustained clocks: keep sampling through a short extra burst if the regions were too brief
    if sampler and last - first < 3:
        t_end = time.perf_counter() + 0.6
        while time.perf_counter() < t_end:
            for _, f in calls:
                f()
        torch.cuda.synchronize(device)
        last = sampler.mark()
    clocks = sampler.summary(first, last) if sampler else None
    if sampler:
        sampler.stop()

    value, max_ms = harness.whole_job_gbs(harness.step_bytes(n, itemsize) * K, elapsed_ms, device)
    ms_per_step = max_ms / K

    reseed()
    # timed region 3, op-major: each kernel K times back to back, so that every launch pays
    # for its own write-backs and none inherits cached or dirty lines from a different kernel
    iso_ms = {}
    for name, f in calls:
        for _ in range(3):
            f()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize(device)
        e0.record(stream)
        for _ in range(K):
            f()
        e1.record(stream)
        torch.cuda.synchronize(device)
        iso_ms[name] = harness.max_over_ranks(e0.elapsed_time(e1) / K, device)
    launches_all = so.launch_count() - launches0

    # end to end: host buffers in, host buffers out, through the library's host entry point
    ha, hb, hc = (p.numpy() for p in pinned)              # last use of the pinned arrays: updated in place
    e2e_steps = args.e2e_steps if chain_cap is None else min(args.e2e_steps, 8)
    e2e_value = None                                      # --e2e-steps 0 (profiling runs) skips this leg
    if e2e_steps > 0:
        so.chain_host(ha, hb, hc, w.scalar)               # allocates the library's device buffers
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            so.chain_host(ha, hb, hc, w.scalar)
        torch.cuda.synchronize(device)
        e2e_ms = (time.perf_counter() - t0) * 1e3
        e2e_value, _ = harness.whole_job_gbs(harness.step_bytes(n, itemsize) * e2e_steps, e2e_ms, device)

    # the shared-memory exchange microkernel, at the paper's default repetition count (own line, not part of `value`)
    shmem = None
    if rank == 0 and world == 1 and not args.no_shmem:
        from paper_2510_00932_b200 import shmembench
        s2 = harness.ClockSampler(gpu_index=local_rank).start()
        shmem = shmembench.measure(1 << 26, 600, 16, iters=20, device=device)
        c2 = s2.summary(); s2.stop()
        mhz = c2["sm_mhz"] or c2["sm_max_mhz"] or 1965.0
        sms = torch.cuda.get_device_properties(device).multi_processor_count
        shmem.update({"bound": "shared memory", "peak_gbs": round(shmembench.smem_peak_gbs(sms, mhz), 1),
                      "peak_source": f"derived: 128 B/clk/SM x {sms} SMs x {mhz:.0f} MHz sampled during the launches",
                      "frac": round(shmem["smem_gbs"] / shmembench.smem_peak_gbs(sms, mhz), 4), "sm_mhz": mhz})
        if args.cpu_seconds > 0:
            import oracle
            nthreads = len(os.sched_getaffinity(0))
            words = inputs.make_words(1 << 22)
            oracle.shmem_mix(words, 8, nthreads)
            t0 = time.perf_counter(); oracle.shmem_mix(words, 600, nthreads); dt = time.perf_counter() - t0
            shmem["cpu_baseline"] = {"value": round(shmembench.smem_bytes(words.size, 600) / dt / 1e9, 2), "unit": "GB/s",
                                     "cores": nthreads, "kind": "oracle",
                                     "sample": "one all-threads pass over n=2^22 words, 600 rounds, same byte accounting"}

    peak, peak_src = harness.measured_peak()
    per_op = harness.per_op_report(op_ms, n, itemsize, peak)
    for name in per_op:
        per_op[name]["best_gbs"] = round(harness.op_bytes(name, n, itemsize) / (op_ms_best[name] * 1e-3) / 1e9, 1)
    per_op_isolated = harness.per_op_report(iso_ms, n, itemsize, peak)
    dominant = max(op_ms, key=lambda k: op_ms[k])
    sig = tuning_signature(so, w.dtype)
    traffic = NCU_TRAFFIC_BYTES.get((w.name, dominant, json.dumps(sig[dominant], sort_keys=True)))
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": per_op[dominant]["gbs"], "peak": peak,
                "peak_source": f"of {peak_src}", "unit": "GB/s",
                "frac": round(per_op[dominant]["gbs"] / peak, 4), "traffic": traffic,
                "region": "chain-order steps with per-launch events; per_op_isolated = same kernels op-major"}

    cpu_baseline = None
    if rank == 0 and world == 1 and args.cpu_seconds > 0:
        nthreads = len(os.sched_getaffinity(0))
        mt_gbs, st_gbs, _, desc = time_oracle(w, args.cpu_seconds, nthreads)
        cpu_baseline = {"value": round(mt_gbs, 3), "unit": UNIT, "cores": nthreads, "kind": "oracle",
                        "sample": desc, "single_thread_value": round(st_gbs, 3)}

    if rank == 0:
        line = {
            "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": warm, "ms_per_step": round(ms_per_step, 5), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
            "config": {"workload": w.name, "n": n, "dist": w.dist, "seed": w.seed, "scalar": w.scalar,
                       "arrays": 3, "array_bytes": n * itemsize, "order": "chain (copy, scale, add, triad, dot per step)",
                       "l2": "no flush: each array is larger than the 126 MB L2", "parallelism": f"replicas x{world}"},
            "clocks": clocks, "shmem_mix": shmem, "per_op": per_op, "per_op_isolated": per_op_isolated, "roofline": roofline, "cpu_baseline": cpu_baseline,
            "e2e": {"value": None if e2e_value is None else round(e2e_value, 2), "unit": UNIT, "h2d_bytes_per_step": 3 * n * itemsize,
                    "d2h_bytes_per_step": 3 * n * itemsize + itemsize, "steps": e2e_steps},
            "gpu_launches": int(launches), "gpu_launches_all_regions": int(launches_all), "frac_nominal_8tbs": round(value / world / harness.NOMINAL_HBM_GBS, 4),
            "tuning": sig,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    args = parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
