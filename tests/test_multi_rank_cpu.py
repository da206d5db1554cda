"""The multi-rank path of the benchmark on CPU: two gloo ranks.

The hot path shards by whole, independent problems (every rank runs the full
workload on its own GPU; no collective touches the data), so what has to be
right across ranks is only the timing reduction -- the slowest rank's time --
and the whole-job aggregate built from it.
"""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench

    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # rank r pretends its step took (10 + 5 r) ms and its retrieves (2 + r) ms
        red = bench.max_over_ranks([10.0 + 5.0 * rank, 2.0 + rank], world)
        total_bytes = 1.5e9
        value = bench.aggregate_value(total_bytes, red[0], world)
        dist.barrier()
        out[rank] = (red, value)
    finally:
        dist.destroy_process_group()


def test_two_ranks_report_slowest_time_and_whole_job_throughput():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_rank_main, args=(world, _free_port(), out), nprocs=world, join=True)
    assert len(out) == world
    for rank in range(world):
        red, value = out[rank]
        assert red == [15.0, 3.0]                       # maximum over ranks, on every rank
        assert value == pytest.approx(2 * 1.5e9 / 15e-3 / 1e9)   # both ranks' bytes over the slowest time


def test_single_rank_is_identity():
    import bench

    assert bench.max_over_ranks([3.0, 4.0], 1) == [3.0, 4.0]
    assert bench.aggregate_value(2e9, 1.0, 1) == pytest.approx(2000.0)


def test_row_sliced_job_counts_the_model_once():
    """--shard rows: the slices of all ranks add up to the model, and the job's value is the model's bytes over the
    slowest rank's time."""
    import bench
    from paper_2505_11204_b200 import workloads as wl

    w = wl.vit_b32()
    for parts in (2, 3, 8):
        slices = [wl.row_slice(w, r, parts)[0] for r in range(parts)]
        assert sum(s.n_params for s in slices) == w.n_params
        assert sum(bench.step_bytes(s, 5)[1] for s in slices) == bench.step_bytes(w, 5)[1]
    assert bench.aggregate_value_sliced(3e9, 2.0) == pytest.approx(1500.0)
    assert bench.parse_args(["--shard", "rows"]).shard == "rows" and bench.parse_args([]).shard == "replicas"


def test_step_bytes_match_the_per_parameter_figures():
    import bench
    from paper_2505_11204_b200 import workloads as wl

    w = wl.vit_l14()
    b, total = bench.step_bytes(w, 5)
    P = w.n_params
    assert P == 303_966_208
    assert b["compress"] == 88 * P and b["retrieve"] == 12 * P and b["add"] == 16 * P == b["remove"]
    assert total == (88 + 20 * 12 + 10 * 16) * P
    wb = w.with_storage(wl.BF16)
    b, _ = bench.step_bytes(wb, 5, out_bytes=2)
    assert b["compress"] == 46 * P and b["retrieve"] == 8 * P and b["add"] == 12 * P


def test_workload_parameter_counts():
    from paper_2505_11204_b200 import workloads as wl

    want = {0: (1_575_936, 12, 2), 1: (87_849_216, 152, 20), 2: (124_439_808, 148, 16), 3: (247_577_856, 282, 29),
            4: (303_966_208, 296, 20)}
    for k, (P, L, G) in want.items():
        w = wl.CONFIGS[k]()
        assert (w.n_params, w.n_layers, len(w.gflags)) == (P, L, G), w.name
    assert len(wl.flan_t5_lora_targets(wl.flan_t5_base())) == 72


def test_context_switch_of_the_benchmark_swaps_the_flip_for_the_gaussian_diagonal():
    """--context gauss: every group that flips signs carries the Gaussian-like context instead, nothing else changes,
    and the line's config says so (the same dict from both arms)."""
    import bench
    from paper_2505_11204_b200 import workloads as wl

    plain = bench.make_workload(bench.parse_args(["--workload", "vit_b32"]))
    args = bench.parse_args(["--workload", "vit_b32", "--context", "gauss"])
    rd = bench.make_workload(args)
    assert rd.name.endswith(":rd") and (rd.rows, rd.cols, rd.group) == (plain.rows, plain.cols, plain.group)
    assert any(f & wl.FLIP for f in plain.gflags)
    for f0, f1 in zip(plain.gflags, rd.gflags):
        assert f1 == ((f0 & ~wl.FLIP) | wl.GAUSS if f0 & wl.FLIP else f0)
    assert "context" in bench.config_dict(rd, args) and "context" not in bench.config_dict(plain, bench.parse_args(["--workload", "vit_b32"]))
    assert bench.step_bytes(rd, 5) == bench.step_bytes(plain, 5)


def test_row_slices_of_every_layer_are_independent_problems():
    """Sharding by row slices needs no collective: the oracle on each slice equals the slice of the oracle."""
    import numpy as np

    from oracle import randes_oracle as ro
    from paper_2505_11204_b200 import workloads as wl

    w = wl.subset(wl.toy(n_tasks=3, width=40, n_blocks=5), list(range(10)))
    w.rows = [7 if r > 1 else 1 for r in w.rows]           # odd row counts: uneven slices, vectors stay whole on part 0
    base, tasks = wl.model_set(w)
    M = ro.compress(w.spec, w.storage, w.task_ids, w.seeds, base, tasks)
    out = ro.retrieve(w.spec, w.storage, wl.F32, 1, w.seeds[1], 0.3, base, M)
    parts = 3
    for part in range(parts):
        ws, bounds = wl.row_slice(w, part, parts)
        cut = lambda model: [np.ascontiguousarray(a[lo:hi]) for a, (lo, hi) in zip(model, bounds)]
        Ms = ro.compress(ws.spec, ws.storage, ws.task_ids, ws.seeds, cut(base), [cut(t) for t in tasks])
        outs = ro.retrieve(ws.spec, ws.storage, wl.F32, 1, ws.seeds[1], 0.3, cut(base), Ms)
        for l, (lo, hi) in enumerate(bounds):
            assert np.array_equal(Ms[l], M[l][lo:hi]) and np.array_equal(outs[l], out[l][lo:hi])


def _bench(*argv, env=None, timeout=240):
    import subprocess

    e = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    e.update(env or {})
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + list(argv), capture_output=True, text=True,
                          env=e, timeout=timeout)


def test_gpus_flag_starts_its_own_ranks_and_counts_them():
    """`python bench.py --gpus 2` without a launcher starts two ranks itself; --check-ranks stops after the
    rendezvous (gloo here, where there is no GPU), so the launcher can be checked without a kernel."""
    import json

    r = _bench("--gpus", "2", "--check-ranks")
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads([l for l in r.stdout.splitlines() if l.startswith("{")][-1])
    assert line["n_gpus"] == 2 and line["ranks_joined"] == 2


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the refusal on a machine without a GPU")
def test_gpus_flag_never_falls_back_to_one_silent_rank():
    """On a machine without GPUs the two ranks refuse to run (no CPU fallback) and the launcher passes the failure
    on: what must not happen is a line that reports n_gpus 1."""
    r = _bench("--gpus", "2", "--steps", "1", "--no-e2e", "--no-cpu-baseline")
    assert r.returncode != 0
    assert "needs a CUDA device" in r.stderr
    assert '"n_gpus"' not in r.stdout


def test_world_size_that_contradicts_gpus_is_an_error():
    import bench

    args = bench.parse_args(["--gpus", "4"])
    old = {k: os.environ.get(k) for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    try:
        os.environ.update(WORLD_SIZE="2", RANK="1", LOCAL_RANK="1")
        with pytest.raises(SystemExit) as e:
            bench.rank_env(args)
        assert "WORLD_SIZE=2" in str(e.value)
        os.environ["WORLD_SIZE"] = "4"
        assert bench.rank_env(args) == (1, 4, 1)
        del os.environ["WORLD_SIZE"]
        with pytest.raises(SystemExit):
            bench.rank_env(args)                      # --gpus 4 and nobody started ranks
        assert bench.rank_env(bench.parse_args([])) == (0, 1, 0)
    finally:
        for k, v in old.items():
            if v is None:
                os.environ.pop(k, None)
            else:
                os.environ[k] = v


def test_reference_arm_times_the_whole_workload_with_the_requested_steps():
    """--impl reference: the oracle on every layer of the workload, the warm-up and step counts that were asked
    for (fewer timed steps only when the budget runs out, and then the line says so)."""
    import json

    r = _bench("--impl", "reference", "--workload", "toy", "--steps", "3", "--warmup", "2", "--gpus", "2",
               env={"RANK": "0", "WORLD_SIZE": "2"})
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["steps"] == 3 and line["warmup"] == 2 and line["steps_timed"] == 3
    assert line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert "all 12 layers" in line["cpu_baseline"]["sample"] and "2 warm-up + 3 timed" in line["cpu_baseline"]["sample"]
    assert line["e2e"]["value"] == line["value"] and line["e2e"]["h2d_bytes_per_step"] == 0
    # the other ranks of the same launch do no work and print nothing
    r1 = _bench("--impl", "reference", "--workload", "toy", "--gpus", "2", env={"RANK": "1", "WORLD_SIZE": "2"})
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    # a budget too small for the request: one step is still timed, and the note says what happened
    r2 = _bench("--impl", "reference", "--workload", "toy", "--steps", "50", "--warmup", "1", "--reference-budget-s", "0")
    line2 = json.loads(r2.stdout.strip().splitlines()[-1])
    assert line2["steps"] == 50 and 1 <= line2["steps_timed"] < 50 and "budget" in line2["note"]
