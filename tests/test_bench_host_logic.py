"""Host-side logic of the benchmark that needs no GPU: the byte accounting, and the multi-rank
aggregation (slowest rank's time, whole-job value) over a world-size-2 gloo group on CPU."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_algorithmic_bytes_match_the_format():
    n, nnz = 1 << 20, 1 << 19
    comp = n // 8 + 4 * nnz + 8 * (n // 4096)
    assert bench.algorithmic_bytes("bt_compress", n, nnz, 4) == 4 * n + comp
    assert bench.algorithmic_bytes("bt_decompress", n, nnz, 4) == 4 * n + comp
    assert bench.algorithmic_bytes("bt_relu_fwd_compress", n, nnz, 2, with_y=True) == 2 * n + 2 * n + n // 8 + 2 * nnz + 8 * (n // 4096)
    assert bench.algorithmic_bytes("bt_relu_bwd_from_bitmap", n, 0, 2) == 4 * n + n // 8
    # 6.127 bytes per fp32 element at half zeros
    assert abs(bench.algorithmic_bytes("bt_compress", n, nnz, 4) / n - 6.127) < 1e-3


def test_whole_job_value_is_the_sum_over_ranks():
    one = bench.whole_job_value(10 ** 9, 1, 1.0)
    assert one == pytest.approx(1000.0)
    assert bench.whole_job_value(10 ** 9, 8, 1.0) == pytest.approx(8 * one)


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    my_ms = 3.0 if rank == 0 else 5.0                      # rank 1 is the slow one
    ms = bench.max_over_ranks(my_ms, world, torch.device("cpu"))
    dist.barrier()
    out.put((rank, ms, bench.whole_job_value(10 ** 9, world, ms)))
    dist.destroy_process_group()


def test_max_over_ranks_gloo_world_size_2():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in got:
        assert ms == pytest.approx(5.0)                    # both ranks agree on the slowest time
        assert value == pytest.approx(2 * 10 ** 9 / 5e-3 / 1e9)


def test_reference_arm_prints_one_json_line(capsys):
    import json
    args = type("A", (), dict(gpus=1, steps=2, warmup=1, impl="reference", reference_budget_s=1.5))()
    bench.run_reference(args)
    line = json.loads(capsys.readouterr().out.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0 and line["metric"] == bench.METRIC
    # the same workload, step count and warm-up as the other arm is asked for
    assert line["config"] == bench.workload_config() and line["steps"] == 2 and line["warmup"] == 1
    assert line["config"]["workload"] == bench.WORKLOAD and line["cpu_baseline"]["value"] == line["value"]


def test_default_arguments():
    a = bench.parse_args([])
    assert (a.gpus, a.steps, a.warmup, a.impl) == (1, 20, 5, "ours") and a.case is None
    c = bench.parse_args(["--case", "bf16", "relu", "--log2n", "27"])
    assert c.case == ["bf16", "relu"] and c.log2n == 27
