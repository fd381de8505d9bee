"""Host-side benchmark logic, on CPU: byte accounting, clock-log parsing, and the N > 1 aggregation
(whole-job GB/s = all ranks' bytes / slowest rank's time) over a 2-rank gloo group."""
import os
import socket

import pytest

from paper_2510_00932_b200 import harness


def test_byte_accounting_is_the_standard_stream_count():
    n = 1 << 25
    assert harness.op_bytes("copy", n, 8) == 536_870_912
    assert harness.op_bytes("scale", n, 8) == 536_870_912
    assert harness.op_bytes("add", n, 8) == 805_306_368
    assert harness.op_bytes("triad", n, 8) == 805_306_368
    assert harness.op_bytes("dot", n, 8) == 536_870_912
    assert harness.step_bytes(n, 8) == 12 * n * 8
    assert harness.step_bytes(1 << 26, 4) == harness.step_bytes(n, 8)


def test_per_op_report_fractions():
    rep = harness.per_op_report({"triad": 0.1}, 1 << 25, 8, 6548.2)
    assert rep["triad"]["gbs"] == pytest.approx(8053.1, abs=0.1)
    assert rep["triad"]["frac_nominal_8tbs"] == pytest.approx(1.0066, abs=1e-3)
    assert rep["triad"]["frac_measured_peak"] == pytest.approx(8053.06 / 6548.2, abs=1e-3)


def test_clock_log_summary():
    lines = [
        "0, 1965, 1965, 612.1, 0x0000000000000004, Not Active, Not Active, Not Active, Active",
        "0, 1800, 1965, 998.0, 0x0000000000000004, Not Active, Not Active, Not Active, Active",
        "0, 1700, 1965, 990.0, 0x0000000000000000, Not Active, Not Active, Not Active, Not Active",
        "garbage",
    ]
    s = harness.summarize_clock_lines(lines)
    assert s == {"sm_mhz": 1800.0, "sm_max_mhz": 1965.0, "reasons": ["sw_power_cap"], "samples": 3}
    hot = harness.summarize_clock_lines(["0, 900, 1965, 500, 0x40, Active, Active, Not Active, Not Active"])
    assert hot["reasons"] == ["hw_slowdown", "hw_thermal_slowdown"]
    assert harness.summarize_clock_lines([])["sm_mhz"] is None


def test_single_process_aggregation_is_identity():
    gbs, ms = harness.whole_job_gbs(3.2e9, 0.5)
    assert ms == 0.5 and gbs == pytest.approx(6400.0)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert harness.dist_env() == (rank, rank, world)
        # rank 1 is the slow one: the job's time is its time, the job's bytes are the sum
        elapsed = 10.0 if rank == 0 else 16.0
        gbs, ms = harness.whole_job_gbs(4.0e9, elapsed)
        assert ms == 16.0 and abs(gbs - 8.0e9 / 16e-3 / 1e9) < 1e-9
        assert harness.max_over_ranks(rank + 1.0) == 2.0 and harness.sum_over_ranks(rank + 1.0) == 3.0
        out.put((rank, gbs))
    finally:
        dist.destroy_process_group()


def test_two_rank_gloo_aggregation():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out, port = ctx.Queue(), _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    got = sorted(out.get(timeout=5) for _ in range(2))
    assert got[0][1] == got[1][1] == pytest.approx(500.0)


def test_reference_arm_prints_one_json_line():
    import json, subprocess, sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--workload", "c1",
                        "--steps", "3", "--warmup", "1"], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "GB/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["config"]["workload"] == "c1"
    # under torchrun only rank 0 works
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--workload", "c1",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=60, env=env)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_launcher_starts_the_ranks_and_rank_zero_prints_one_line(capfd):
    """The path `bench.py --gpus N` takes when it is started by hand: harness.launch_ranks runs
    torch.distributed.run with N processes on 127.0.0.1; here N = 2 gloo ranks of a stub."""
    import json
    here = os.path.dirname(os.path.abspath(__file__))
    rc = harness.launch_ranks(os.path.join(here, "rank_stub.py"), ["--steps", "2"], 2)
    out = capfd.readouterr().out
    assert rc == 0
    lines = [l for l in out.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["argv"] == ["--steps", "2"]
    assert d["ms"] == 15.0 and d["value"] == pytest.approx(3.0e9 / 15e-3 / 1e9)


def test_bench_refuses_more_gpus_than_are_visible_and_the_reference_arm_needs_none():
    import json, subprocess, sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    import torch
    if torch.cuda.device_count() < 2:
        r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--steps", "1", "--warmup", "1"],
                           capture_output=True, text=True, timeout=300, env=env)
        assert r.returncode != 0 and "CUDA device" in r.stderr and "--gpus 2" in r.stderr and r.stdout.strip() == ""
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--impl", "reference", "--workload", "c1",
                        "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0, r.stderr
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1 and json.loads(lines[0])["n_gpus"] == 2
    # a world size that contradicts --gpus is an error, not a silently mislabelled line
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "4", "--steps", "1"],
                       capture_output=True, text=True, timeout=300, env=dict(env, WORLD_SIZE="2", RANK="0", LOCAL_RANK="0"))
    assert r.returncode != 0 and "WORLD_SIZE=2" in r.stderr


def test_traffic_summary_round_trip(tmp_path, monkeypatch):
    """ncu launch list -> per-kernel DRAM bytes of the op-major runs -> what bench.py reads; a
    capture taken under another tuning is not used."""
    from paper_2510_00932_b200 import build, ncu_summary
    build.build()
    hdr = '"ID","Process ID","Process Name","Host Name","Kernel Name","Context","Stream","Block Size","Grid Size","Device","CC","Section Name","Metric Name","Metric Unit","Metric Value"'
    add = "void streamops::ew_vec_kernel<double, (int)2, (int)32, (int)2, (int)7>(const T1 *, const T1 *, T1 *, T1, unsigned long, int, int, unsigned long)"
    cpy = "void streamops::ew_vec_kernel<unsigned long long, (int)0, (int)32, (int)2, (int)7>(const T1 *, const T1 *, T1 *, T1, unsigned long, int, int, unsigned long)"
    rows, i = [hdr], 0

    def launch(kernel, rd, wr, ns):
        nonlocal i
        for m, u, v in (("dram__bytes_read.sum", "Mbyte", rd), ("dram__bytes_write.sum", "Mbyte", wr), ("gpu__time_duration.sum", "ns", ns)):
            rows.append(f'"{i}","1","python","h","{kernel}","1","7","(128, 1, 1)","(100, 1, 1)","0","10.0","Command line profiler metrics","{m}","{u}","{v}"')
        i += 1

    for k in (add, cpy, add, cpy):                        # chain-order launches: runs of one, ignored
        launch(k, 100.0, 100.0, "50,000")
    for v in (300.0, 536.9, 537.1, 536.8, 537.0):         # op-major run of add (first launch differs)
        launch(add, v, 268.4, "118,000")
    for v in (268.4, 268.5, 268.3, 268.4):
        launch(cpy, v, 268.4, "79,900")
    p = tmp_path / "l.csv"
    p.write_text("==PROF== Connected\n" + "\n".join(rows) + "\n")
    out = tmp_path / "t.txt"
    assert ncu_summary.main([str(p), "--workload", "c2", "--command", "ncu ...", "--out", str(out)]) == 0
    data = harness.read_traffic_file(str(out))
    assert data["kernels"]["add"]["dram_read_bytes"] == 536_950_000 and data["kernels"]["add"]["launch_us"] == 118.0
    assert data["kernels"]["copy"]["dram_write_bytes"] == 268_400_000 and "dot" not in data["kernels"]
    monkeypatch.setattr(harness, "traffic_file", lambda w: str(out))
    from paper_2510_00932_b200 import streamops as so
    so.reset_tuning()
    t = so.get_tuning("add", "f64").as_dict()
    assert harness.captured_traffic("c2", "add", t) == 536_950_000 + 268_400_000
    assert harness.captured_traffic("c2", "add", dict(t, unroll=4)) is None
    assert harness.captured_traffic("c2", "dot", so.get_tuning("dot", "f64").as_dict()) is None


def test_pin_bandwidth_from_device_attributes():
    assert harness.pin_bandwidth_gbs(3996000, 7680) == pytest.approx(7672.3, abs=0.1)
    assert harness.pin_bandwidth_gbs(3996000, 8192) == pytest.approx(8183.8, abs=0.1)
    rep = harness.per_op_report({"dot": 0.0731}, 1 << 25, 8, 6548.8, 7672.3)
    assert rep["dot"]["frac_pin_bandwidth"] == pytest.approx(536870912 / 0.0731e-3 / 1e9 / 7672.3, abs=1e-3)
