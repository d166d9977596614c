"""Host-side parts of bench.py: the reference (oracle) arm and the max-over-ranks
reduction used for multi-rank timing (two gloo ranks on CPU)."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                          "--warmup", "1", "--reference-columns", "3000"], capture_output=True, text=True, check=True)
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["metric"] == "replica_params_synchronised_per_sec"
    assert rec["value"] > 0 and rec["steps"] == 2 and rec["warmup"] == 1 and rec["higher_is_better"] is True
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["cpu_baseline"]["cores"] == 1
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["e2e"]["d2h_bytes_per_step"] == 0
    assert rec["e2e"]["value"] == rec["value"]


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, check=True, env=env)
    assert out.stdout.strip() == ""


def _rank_main(rank, world, port, results):
    sys.path.insert(0, ROOT)
    import bench

    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        bench.barrier()
        got = bench.max_over_ranks(10.0 + 5.0 * rank)
        results.put((rank, got))
        bench.barrier()
    finally:
        dist.destroy_process_group()


def test_max_over_ranks_with_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    results = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, results)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(results.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert got == {0: 15.0, 1: 15.0}


def _shard_rank_main(rank, world, port, results):
    sys.path.insert(0, ROOT)
    from paper_1810_07766_b200 import binding

    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        d = 4_000_037
        mine = torch.tensor(binding.shard_columns(d, world, rank), dtype=torch.int64)
        everyone = [torch.zeros(2, dtype=torch.int64) for _ in range(world)]
        dist.all_gather(everyone, mine)
        results.put((rank, [tuple(int(v) for v in e) for e in everyone]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_column_shards_of_two_gloo_ranks_tile_the_model():
    """Every rank derives its own column range from (d, world, rank) alone; together they cover the model once."""
    ctx = mp.get_context("spawn")
    results = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_shard_rank_main, args=(r, 2, port, results)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(results.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert got[0] == got[1]
    (b0, c0), (b1, c1) = got[0]
    assert b0 == 0 and b1 == c0 and b1 % 64 == 0 and c0 + c1 == 4_000_037 and abs(c0 - c1) < 128


def test_shard_ranges_cover_the_model_once():
    sys.path.insert(0, ROOT)
    from paper_1810_07766_b200 import binding

    for d in (1, 63, 64, 65, 1000, 4_000_037, 11_173_962):
        for world in (1, 2, 3, 8, 64):
            ranges = [binding.shard_columns(d, world, r) for r in range(world)]
            at = 0
            for begin, cols in ranges:
                if cols:
                    assert begin == at and begin % 64 == 0
                    at += cols
            assert at == d
            sizes = [c for _, c in ranges if c]
            assert max(sizes) - min(sizes) < 128


def test_max_over_ranks_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(3.5) == 3.5


def test_bench_refuses_to_run_the_product_arm_without_a_gpu():
    if torch.cuda.is_available():
        return
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "1"], capture_output=True, text=True)
    assert out.returncode != 0 and "CUDA" in (out.stderr + out.stdout)


def test_default_suite_and_kernel_names():
    """The default run times every configuration with the largest fp32 model (d >= 11M) as the headline, and names the
    kernel the library picks for each (the names are what the profiler's launch list shows)."""
    sys.path.insert(0, ROOT)
    import argparse

    import bench
    from paper_1810_07766_b200 import workloads as wl

    assert bench.DEFAULT_SUITE[0] == bench.HEADLINE == "cfg3"
    assert set(bench.DEFAULT_SUITE) == {"cfg2", "cfg3", "cfg4", "cfg5"}
    head = wl.WORKLOADS[bench.HEADLINE]
    assert head.dtype == "f32" and head.d >= 11_000_000
    assert all(wl.WORKLOADS[c].n * wl.WORKLOADS[c].d <= head.n * head.d for c in bench.DEFAULT_SUITE if wl.WORKLOADS[c].dtype == "f32")
    args = argparse.Namespace(kernel=0, average_gradients=False, track=False, workers_per_lane=0, consumer_warps=0,
                              copy_mode=0, slice_bytes=0, d=None, sigma=None, n=None)
    names = {c: bench.fused_kernel_name(args, wl.WORKLOADS[c]) for c in ("cfg1", "cfg2", "cfg3", "cfg4", "cfg5")}
    assert names == {"cfg1": "rps_fused_direct_kernel", "cfg2": "rps_fused_staged_kernel", "cfg3": "rps_fused_staged_kernel",
                     "cfg4": "rps_fused_staged_kernel", "cfg5": "rps_fused_stream_kernel"}
    from dataclasses import replace
    assert bench.fused_kernel_name(args, replace(wl.WORKLOADS["cfg5"], n=32)) == "rps_fused_ring_kernel"
    args.track = True
    assert bench.fused_kernel_name(args, replace(wl.WORKLOADS["cfg5"], n=32)) == "rps_fused_stream_kernel"
    args.track, args.average_gradients = False, True
    assert bench.fused_kernel_name(args, wl.WORKLOADS["cfg5"]) == "rps_fused_ring_kernel"
    assert bench.fused_kernel_name(args, replace(wl.WORKLOADS["cfg5"], n=48)) == "rps_fused_stream_kernel"
    assert bench.fused_kernel_name(args, replace(wl.WORKLOADS["cfg5"], n=56)) == "rps_fused_ring_kernel"
    args.average_gradients = False
    # between two powers of two the streamed kernel serves both types
    assert bench.fused_kernel_name(args, replace(wl.WORKLOADS["cfg5"], n=24)) == "rps_fused_stream_kernel"
    assert bench.fused_kernel_name(args, replace(wl.WORKLOADS["cfg4"], n=24)) == "rps_fused_stream_kernel"
    assert bench.fused_kernel_name(args, replace(wl.WORKLOADS["cfg5"], n=16)) == "rps_fused_ring_kernel"
    assert bench.fused_kernel_name(args, replace(wl.WORKLOADS["cfg5"], n=4)) == "rps_fused_stream_kernel"
    w = bench.resolve_workload(argparse.Namespace(d=1000, sigma=0.0, n=6), "cfg2", p=0.3)
    assert (w.n, w.d, w.p, w.sigma, w.gamma, w.seed) == (6, 1000, 0.3, 0.0, 0.05, 1)
