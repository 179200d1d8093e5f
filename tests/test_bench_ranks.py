"""Host-side plumbing of bench.py for N > 1 ranks, on CPU with the gloo backend (world size 2):
the max-over-ranks reduction, the whole-job (replicas) aggregate, and the reference arm under
torchrun (rank 0 alone works and prints one JSON line)."""
import json
import os
import socket
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    import workloads as wl
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    per_rank_seconds = 1.0e-3 * (1 + rank)            # rank 1 is the slow one
    worst = bench.max_over_ranks(per_rank_seconds)
    w = wl.configs()["c2"]
    out.put((rank, worst, bench.whole_job_value(w, worst, world)))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value_gloo():
    port = free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [2.0e-3, 2.0e-3]     # every rank sees the slowest rank's time
    flops = 2.0 * 8192 ** 3
    assert abs(res[0][2] - 2 * flops / 2.0e-3 / 1e12) < 1e-6 and res[0][2] == res[1][2]


def test_single_process_helpers_need_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(0.25) == 0.25


def test_reference_arm_under_torchrun_prints_one_line_from_rank0():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(free_port()), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--steps", "2", "--warmup", "1", "--config", "c1", "--ref-step-seconds", "0.2"]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["steps"] == 2 and d["gpu_launches"] == 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"] > 0
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["unit"] == "TFLOP/s" and d["higher_is_better"] is True and d["config"]["workload"].startswith("c1")


def test_shape_specifications_of_the_sweep_mode():
    import pytest
    import bench
    import workloads as wl
    w = bench.parse_shape("28672x8x8192:beta=1:cd=f32:epi=bias_silu:rowbias=1")
    assert (w.M, w.N, w.K, w.beta, w.c_dtype, w.epilogue, w.bias_per_row) == (28672, 8, 8192, 1.0, wl.F32, wl.EPI_BIAS_SILU, True)
    w = bench.parse_shape("256x128x512:ab=e4m3:tri=upper:batch=3:ta=0:tb=1:lda=520")
    assert (w.ab_dtype, w.a_tri, w.batch, w.lda, w.c_dtype) == (wl.FP8_E4M3, 2, 3, 520, wl.BF16)
    assert w.min_bytes == 3 * (256 * 512 + 512 * 128) * 1 + 3 * 256 * 128 * 2       # 8-bit operands, 16-bit output
    w = bench.parse_shape("4096x4096x512:dtri=lower")
    assert w.d_tri == 1 and w.flops == 2.0 * (4096 * 4097 // 2) * 512
    with pytest.raises(SystemExit):
        bench.parse_shape("8x8x8:nonsense=1")
    # an 8-bit problem is held against the measured bf16 peak times the nominal fp8 : bf16 ratio
    peaks = {"bf16_tflops": 1000.0, "bf16_tflops_sustained": 900.0, "hbm_gbs": 6000.0}
    r = bench.roofline_for(bench.parse_shape("8192x8192x8192:ab=e4m3"), "x", 1e-3, peaks, "measured")
    assert r["bound"] == "tensor" and r["peak"] == 2000.0 and abs(r["frac"] - 2 * 8192 ** 3 / 1e-3 / 1e12 / 2000.0) < 1e-3
