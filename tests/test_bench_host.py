"""Host-side logic of bench.py: the multi-rank aggregation (world size 2, gloo, CPU) and the
reference arm (the CPU oracle timed on the host cores)."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import bench
    r, w, _ = bench.dist_setup("gloo")
    bench.barrier()
    units, ms = bench.aggregate(100.0 * (rank + 1), 10.0 + 5.0 * rank)
    out.put((r, w, units, ms))
    bench.barrier()


def test_aggregate_sums_units_and_takes_the_slowest_rank():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[:2] for g in got] == [(0, 2), (1, 2)]
    for _, _, units, ms in got:
        assert units == 300.0 and ms == 15.0


def test_reference_arm_prints_one_json_line():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1",
           "--steps", "3", "--warmup", "1"]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert res.returncode == 0, res.stderr
    lines = [l for l in res.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["steps"] == 3 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["config"]["workload"] == "mlp_p4_dense"


def test_captured_traffic_is_tied_to_the_kernel_sources(monkeypatch):
    """`roofline.traffic` comes from an ncu capture: it is reported only while the sources of the
    kernels the configuration launches are the ones the capture was taken with, and says so
    otherwise instead of going silently null."""
    import types

    import bench
    dense = types.SimpleNamespace(topk=None, P=16, N=11173962)
    small = types.SimpleNamespace(topk=None, P=8, N=269722)
    sparse = types.SimpleNamespace(topk=(1, 100), P=8, N=11173962)
    assert bench.kernel_sources(dense) == bench.DENSE_SOURCES
    assert "eg_step_small.cuh" in bench.kernel_sources(small) and "eg_topk.cuh" in bench.kernel_sources(sparse)
    now = bench.kernel_source_hash(bench.DENSE_SOURCES)
    monkeypatch.setitem(bench.FUSED_TRAFFIC, "dense", {now: (2.0e9, "profiles/somewhere.md")})
    got = bench.fused_traffic(dense, 2 * bench.FUSED_TRAFFIC_ELEMENTS, None)
    assert got["traffic"] == 4.0e9 and got["traffic_from"] == "profiles/somewhere.md"
    monkeypatch.setitem(bench.FUSED_TRAFFIC, "dense", {"0" * 12: (2.0e9, "profiles/somewhere.md")})
    stale = bench.fused_traffic(dense, bench.FUSED_TRAFFIC_ELEMENTS, None)
    assert stale["traffic"] is None and "0" * 12 in stale["traffic_stale_since"] and now in stale["traffic_stale_since"]
    for wl in (small, sparse):
        other = bench.fused_traffic(wl, 1000, None)
        assert other["traffic"] is None and "traffic_note" in other
    assert bench.fused_traffic(dense, 1000, 0.9)["traffic"] is None
