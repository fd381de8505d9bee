#!/usr/bin/env python
"""Benchmark of the five streaming kernels (copy, scale, add, triad, dot) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl ours|reference]

One step = one pass of all five kernels over the three arrays of the workload, in the STREAM
dataflow (c <- a; b <- s*c; c <- a+b; a <- b+s*c; dot(a, b)). The line printed by rank 0 reports

  value            whole-job algorithmic GB/s of K steps back to back. Consecutive kernels of a step
                   hand data to each other through L2, so this is NOT a DRAM rate (see value_note);
  per_op_isolated  each kernel launched K times in a row (op-major): no kernel inherits cached lines
                   from a different kernel, so these are the per-kernel HBM figures, and `roofline`
                   is taken from the slowest of them relative to its bytes;
  per_op           the same kernels in chain order with an event before every launch;
  parity           the arrays and the dot product after the K timed steps, compared with the CPU
                   oracle applied K times to the same seeded inputs (bit-exact / 1e-12, 1e-5);
  e2e              the same pass through the host-buffer entry point, copies inside the timed region;
  cpu_baseline     the CPU oracle timed on the host cores beside it.

With N > 1 every rank runs its own replica of the workload (one process per GPU): the kernels are
independent per index, so the path shards with no data-path collective; the only communication is
the barrier and the MAX/SUM of the timings. `python bench.py --gpus N` starts the N ranks itself
(torch.distributed.run on 127.0.0.1) unless it already runs under one.
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
DOT_TOL = {"f64": 1e-12, "f32": 1e-5}


def parse_args(argv=None):
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=200)
    p.add_argument("--warmup", type=int, default=10)
    p.add_argument("--workload", default="c2", choices=["c1", "c2", "c3", "c4"])
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--e2e-steps", type=int, default=20)
    p.add_argument("--tuning", default="",
                   help='JSON overrides of the launch tuning for A/B runs, e.g. \'{"ew": {"policy": 5}, "dot": {"two_pass": 1}}\' '
                        '("ew" = copy, scale, add, triad; "all" = the five ops)')
    p.add_argument("--no-shmem", action="store_true", help="skip the shared-memory microkernel line")
    p.add_argument("--no-parity", action="store_true", help="skip the oracle comparison of the timed arrays")
    p.add_argument("--extra", default="c3,c4",
                   help="other workloads to time op-major after the main one (N = 1 only; '' = none)")
    p.add_argument("--cpu-seconds", type=float, default=12.0,
                   help="CPU time budget of the oracle baseline leg (0 = skip)")
    return p.parse_args(argv)


def tuning_signature(so, dtype):
    return {op: so.get_tuning(op, dtype).as_dict() for op in so.OPS}


# ------------------------------------------------------------------------------- oracle legs
def oracle_chain_mt(oracle, a, b, c, scalar, nthreads):
    """One pass of the five kernels by the all-threads form of the oracle; returns (a, b, c, dot)."""
    cc = oracle.run_mt("copy", a, None, 0.0, nthreads)
    bb = oracle.run_mt("scale", cc, None, scalar, nthreads)
    cc = oracle.run_mt("add", a, bb, 0.0, nthreads)
    aa = oracle.run_mt("triad", bb, cc, scalar, nthreads)
    return aa, bb, cc, oracle.run_mt("dot", aa, bb, 0.0, nthreads)


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
            oracle_chain_mt(oracle, a, b, c, w.scalar, nt)
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
    for _ in range(args.warmup):
        oracle_chain_mt(oracle, a, b, c, w.scalar, nthreads)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_chain_mt(oracle, a, b, c, w.scalar, nthreads)
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
def make_calls(so, w, da, db, dc, dd):
    return [("copy", lambda: so.copy(da, dc)), ("scale", lambda: so.scale(dc, db, w.scalar)),
            ("add", lambda: so.add(da, db, dc)), ("triad", lambda: so.triad(db, dc, da, w.scalar)),
            ("dot", lambda: so.dot(da, db, dd))]


def time_op_major(torch, calls, K, device, stream, harness):
    """Each kernel K times back to back (after 3 untimed launches), one event pair around the K:
    every launch pays for its own write-backs and none inherits cached lines from another kernel."""
    out = {}
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
        out[name] = harness.max_over_ranks(e0.elapsed_time(e1) / K, device)
    return out


def check_parity(oracle, w, seeded, device_arrays, device_dot, steps, nthreads):
    """The CPU oracle applied `steps` times to the seeded inputs against what the device holds:
    arrays bit for bit (raw words), dot product within the tolerance of its precision."""
    import numpy as np
    a, b, c = seeded
    d = 0.0
    for _ in range(steps):
        a, b, c, d = oracle_chain_mt(oracle, a, b, c, w.scalar, nthreads)
    word = np.uint64 if w.itemsize == 8 else np.uint32
    mismatches = {name: int((got.view(word) != want.view(word)).sum())
                  for name, got, want in zip("abc", device_arrays, (a, b, c))}
    mags = oracle.dot_abs(a, b)
    rel = abs(float(device_dot) - d) / abs(d) if d != 0 else abs(float(device_dot)) / max(mags, 1e-300)
    ok = not any(mismatches.values()) and rel <= DOT_TOL[w.dtype]
    return {"verdict": "ok" if ok else "FAILED", "steps_checked": steps, "array_word_mismatches": mismatches,
            "dot": float(device_dot), "dot_oracle": d, "dot_rel_err": rel, "dot_tol": DOT_TOL[w.dtype],
            "dot_condition_number": mags / abs(d) if d != 0 else None}


def host_link_ceiling(torch, device, up_bytes: int, down_bytes: int, reps: int = 5):
    """What the host link itself delivers for pinned memory, to hold the end-to-end figure against:
    GB/s of a host-to-device copy alone, of a device-to-host copy alone, and the time one step's bytes
    take when its upload and its download run at the same time on two streams (plain cudaMemcpyAsync
    through torch; no kernel involved)."""
    nu, nd = up_bytes // 8, down_bytes // 8
    h_in, h_out = torch.empty(nu, dtype=torch.float64).pin_memory(), torch.empty(nd, dtype=torch.float64).pin_memory()
    d_in, d_out = torch.empty(nu, dtype=torch.float64, device=device), torch.zeros(nd, dtype=torch.float64, device=device)
    s_up, s_down = torch.cuda.Stream(device), torch.cuda.Stream(device)

    def timed(up: bool, down: bool):
        best = float("inf")
        for _ in range(reps):
            torch.cuda.synchronize(device)
            t0 = time.perf_counter()
            if up:
                with torch.cuda.stream(s_up):
                    d_in.copy_(h_in, non_blocking=True)
            if down:
                with torch.cuda.stream(s_down):
                    h_out.copy_(d_out, non_blocking=True)
            torch.cuda.synchronize(device)
            best = min(best, time.perf_counter() - t0)
        return best

    return {"h2d_alone_gbs": round(up_bytes / timed(True, False) / 1e9, 1),
            "d2h_alone_gbs": round(down_bytes / timed(False, True) / 1e9, 1),
            "one_step_both_ways_ms": round(timed(True, True) * 1e3, 3), "up_bytes": up_bytes, "down_bytes": down_bytes}


def versions(torch):
    import subprocess
    import numpy as np
    try:
        drv = subprocess.run(["nvidia-smi", "--query-gpu=driver_version,name", "--format=csv,noheader"],
                             capture_output=True, text=True, timeout=20).stdout.strip().splitlines()[0]
    except (OSError, subprocess.SubprocessError, IndexError):
        drv = None
    return {"numpy": np.__version__, "torch": torch.__version__, "cuda_runtime": torch.version.cuda,
            "driver_and_gpu": drv, "python": sys.version.split()[0]}


def run_extra(torch, so, harness, inputs, name, K, device, stream, peak, pin_gbs=None):
    """Op-major timing of another named workload (few launches), so that the record carries the
    single-precision and the 2 GiB-per-array figures beside the headline one."""
    w = inputs.WORKLOADS[name]
    need = 3 * w.n * w.itemsize
    if torch.cuda.mem_get_info(device)[0] < need + (2 << 30):
        return {"skipped": "not enough free device memory"}
    da, db, dc = (torch.from_numpy(v).to(device) for v in inputs.make_arrays(w))
    dd = torch.zeros(1, dtype=da.dtype, device=device)
    ms = time_op_major(torch, make_calls(so, w, da, db, dc, dd), K, device, stream, harness)
    so.check()
    rep = harness.per_op_report(ms, w.n, w.itemsize, peak, pin_gbs)
    return {"dtype": w.dtype, "n": w.n, "dist": w.dist, "launches_per_op": K, "order": "op-major", "per_op_isolated": rep}


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
    checksums = [inputs.checksum(v) for v in (a, b, c)]
    pinned = [torch.from_numpy(v).pin_memory() for v in (a, b, c)]
    da, db, dc = (p.to(device, non_blocking=False) for p in pinned)
    dd = torch.zeros(1, dtype=da.dtype, device=device)
    stream = torch.cuda.current_stream(device)
    n, itemsize = w.n, w.itemsize
    calls = make_calls(so, w, da, db, dc, dd)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(device)

    def reseed():
        for dst, src in zip((da, db, dc), pinned):
            dst.copy_(src, non_blocking=False)

    # fp32 with s = 3.0 grows a by 15x per chain step and overflows after ~33 steps: bound the
    # chained steps per region
    chain_cap = 25 if (w.dtype == "f32" and abs(w.scalar) > 1.0) else None
    warm = max(args.warmup, 3) if chain_cap is None else 3
    for _ in range(warm):
        for _, f in calls:
            f()
    reseed()                                             # every timed region starts from the seeded arrays
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
    so.check()

    # what region 1 left on the device, for the parity check further down (rank 0, one GPU)
    parity_wanted = rank == 0 and world == 1 and not args.no_parity
    timed_arrays = [t.cpu().numpy() for t in (da, db, dc)] if parity_wanted else None
    timed_dot = dd.cpu().numpy()[0] if parity_wanted else None

    reseed()
    barrier()
    # timed region 2: K more chain steps with an event before every launch -> per-kernel durations
    # in chain order (the extra events cost a few us per launch, which is why region 1 has none)
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

    value, max_ms = harness.whole_job_gbs(harness.step_bytes(n, itemsize) * K, elapsed_ms, device)
    ms_per_step = max_ms / K

    reseed()
    # timed region 3, op-major
    iso_ms = time_op_major(torch, calls, K, device, stream, harness)
    # sustained clocks: keep sampling through a short extra burst if the regions were too brief
    last = sampler.mark() if sampler else 0
    if sampler and last - first < 3:
        t_end = time.perf_counter() + 0.6
        while time.perf_counter() < t_end:
            for _, f in calls[:4]:
                f()
        torch.cuda.synchronize(device)
        last = sampler.mark()
    clocks = sampler.summary(first, last) if sampler else None
    if sampler:
        sampler.stop()
    launches_all = so.launch_count() - launches0
    so.check()

    # end to end: host buffers in, host buffers out, through the library's host entry point
    ha, hb, hc = (p.numpy() for p in pinned)              # the pinned arrays are updated in place from here on
    e2e_steps = args.e2e_steps if chain_cap is None else min(args.e2e_steps, 8)
    e2e_value, e2e_dot, e2e_link = None, None, None       # --e2e-steps 0 (profiling runs) skips this leg
    if e2e_steps > 0:
        warm_e2e = [v[:1 << 22].copy() for v in (ha, hb, hc)]
        so.chain_host(*warm_e2e, w.scalar)                # creates the library's device ring; leaves the arrays alone
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_dot = so.chain_host(ha, hb, hc, w.scalar)
        torch.cuda.synchronize(device)
        e2e_ms = (time.perf_counter() - t0) * 1e3
        e2e_value, _ = harness.whole_job_gbs(harness.step_bytes(n, itemsize) * e2e_steps, e2e_ms, device)
        if rank == 0 and world == 1:
            # the link's own ceiling: a step moves one array up (a; b and c are outputs only) and three down
            e2e_link = host_link_ceiling(torch, device, n * itemsize, 3 * n * itemsize)
            ceiling = harness.step_bytes(n, itemsize) / (e2e_link["one_step_both_ways_ms"] * 1e-3) / 1e9
            e2e_link.update({"e2e_ceiling_gbs": round(ceiling, 1), "e2e_frac_of_ceiling": round(e2e_value / ceiling, 4)})

    peak, peak_src = harness.measured_peak()
    # what the memory pins could carry: data rate x bus width, both read from the device at run time
    props = torch.cuda.get_device_properties(device)
    pin_gbs = None
    if getattr(props, "memory_clock_rate", 0) and getattr(props, "memory_bus_width", 0):
        pin_gbs = harness.pin_bandwidth_gbs(props.memory_clock_rate, props.memory_bus_width)
    extra = {}
    if rank == 0 and world == 1:
        del calls, da, db, dc
        torch.cuda.empty_cache()
        for name in [x for x in args.extra.split(",") if x and x != w.name]:
            extra[name] = run_extra(torch, so, harness, inputs, name, max(5, min(K, 20)), device, stream, peak, pin_gbs)
            torch.cuda.empty_cache()

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

    per_op = harness.per_op_report(op_ms, n, itemsize, peak, pin_gbs)
    for name in per_op:
        per_op[name]["best_gbs"] = round(harness.op_bytes(name, n, itemsize) / (op_ms_best[name] * 1e-3) / 1e9, 1)
    per_op_isolated = harness.per_op_report(iso_ms, n, itemsize, peak, pin_gbs)
    # the kernel that takes the largest share of the op-major time is the one the roofline entry describes
    dominant = max(iso_ms, key=lambda k: iso_ms[k])
    sig = tuning_signature(so, w.dtype)
    traffic = harness.captured_traffic(w.name, dominant, sig[dominant])
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": per_op_isolated[dominant]["gbs"], "peak": peak,
                "peak_source": f"of {peak_src}", "unit": "GB/s",
                "frac": round(per_op_isolated[dominant]["gbs"] / peak, 4),
                "frac_nominal_8tbs": per_op_isolated[dominant]["frac_nominal_8tbs"], "traffic": traffic,
                "pin_bandwidth_gbs": None if pin_gbs is None else round(pin_gbs, 1),
                "pin_bandwidth_source": "2 x memory clock x bus width as the device reports them "
                                        f"({props.memory_clock_rate / 1e3:.0f} MHz, {props.memory_bus_width} bits)",
                "frac_of_pin_bandwidth": None if pin_gbs is None else round(per_op_isolated[dominant]["gbs"] / pin_gbs, 4),
                "region": "op-major: the kernel launched K times in a row, one CUDA-event pair around the K; "
                          "no cached lines inherited from other kernels. The peak is a plain 1:1 copy; a 2:1 read-heavy "
                          "kernel can read a little above it"}

    parity = None
    cpu_baseline = None
    if rank == 0 and world == 1:
        import oracle
        nthreads = len(os.sched_getaffinity(0))
        if parity_wanted:
            parity = check_parity(oracle, w, (a, b, c), timed_arrays, timed_dot, K, nthreads)
            parity["input_checksums"] = checksums
            if e2e_steps > 0:
                # the host-buffer leg applied e2e_steps passes to the pinned copies of the same seeded arrays
                e = check_parity(oracle, w, (a, b, c), (ha, hb, hc), e2e_dot, e2e_steps, nthreads)
                parity["e2e"] = {k: e[k] for k in ("verdict", "steps_checked", "array_word_mismatches", "dot_rel_err")}
                if e["verdict"] != "ok":
                    parity["verdict"] = "FAILED"
        if args.cpu_seconds > 0:
            mt_gbs, st_gbs, _, desc = time_oracle(w, args.cpu_seconds, nthreads)
            cpu_baseline = {"value": round(mt_gbs, 3), "unit": UNIT, "cores": nthreads, "kind": "oracle",
                            "sample": desc, "single_thread_value": round(st_gbs, 3)}

    if rank == 0:
        line = {
            "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": warm, "ms_per_step": round(ms_per_step, 5), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
            "value_note": "algorithmic bytes of the five kernels in chain order; includes inter-kernel L2 reuse "
                          "(each kernel reads part of what its producer just wrote from L2), so it is not a DRAM rate: "
                          "per_op_isolated holds the per-kernel HBM figures",
            "config": {"workload": w.name, "n": n, "dist": w.dist, "seed": w.seed, "scalar": w.scalar,
                       "arrays": 3, "array_bytes": n * itemsize, "order": "chain (copy, scale, add, triad, dot per step)",
                       "l2": "no flush: each array is larger than the 126 MB L2", "parallelism": f"replicas x{world}"},
            "clocks": clocks, "parity": parity, "per_op_isolated": per_op_isolated, "per_op": per_op, "roofline": roofline,
            "cpu_baseline": cpu_baseline,
            "e2e": {"value": None if e2e_value is None else round(e2e_value, 2), "unit": UNIT, "h2d_bytes_per_step": n * itemsize,
                    "d2h_bytes_per_step": 3 * n * itemsize + itemsize, "steps": e2e_steps,
                    "note": "the pass reads only a of the three host arrays (it overwrites c and b before reading them), "
                            "so one array goes up and three come down",
                    "host_link": e2e_link},
            "gpu_launches": int(launches), "gpu_launches_all_regions": int(launches_all),
            "frac_nominal_8tbs": round(value / world / harness.NOMINAL_HBM_GBS, 4),
            "other_workloads": extra, "shmem_mix": shmem, "versions": versions(torch), "tuning": sig,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 0 if (parity is None or parity["verdict"] == "ok") else 1


def main(argv=None):
    args = parse_args(argv)
    from paper_2510_00932_b200 import harness
    if args.impl == "reference":
        return run_reference(args)                       # rank 0 alone works, under a launcher or not
    _, _, world = harness.dist_env()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started by hand: become the launcher of N ranks of this same command
        import torch
        have = torch.cuda.device_count()
        if have < args.gpus:
            raise SystemExit(f"bench.py --gpus {args.gpus}: only {have} CUDA device(s) are visible; "
                             "there is no CPU fallback and ranks never share a GPU")
        return harness.launch_ranks(os.path.abspath(__file__), sys.argv[1:] if argv is None else list(argv), args.gpus)
    if world != args.gpus:
        raise SystemExit(f"bench.py --gpus {args.gpus} was started with WORLD_SIZE={world}")
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
