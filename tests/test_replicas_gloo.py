"""The N > 1 path is "replicas only": no data-path collective, just a barrier and a max over
ranks of the device time.  Exercised here with two gloo ranks on CPU."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        dist.barrier()
        ms = bench.replica_max_ms(torch, dist, 10.0 + 5.0 * rank, torch.device("cpu"))
        local = {"value": 0.0, "unit": "TFLOP/s", "ms_per_step": 40.0 + 10.0 * rank, "h2d_bytes_per_step": 1000,
                 "d2h_bytes_per_step": 10}
        e2e = bench.replica_e2e(torch, dist, local, world, 1e12, torch.device("cpu"))
        out[rank] = (ms, bench.replica_throughput(world, 1e12, ms), e2e)
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_slowest_time_and_summed_work():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29731, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, tflops, e2e = res[0]
    assert ms == 15.0
    assert tflops == pytest.approx(2 * 1e12 / 15e-3 / 1e12)
    # the end-to-end record of the job: slowest rank's time, both replicas' work and bytes
    assert e2e["ms_per_step"] == 50.0 and e2e["h2d_bytes_per_step"] == 2000 and e2e["d2h_bytes_per_step"] == 20
    assert e2e["value"] == pytest.approx(2 * 1e12 / 50e-3 / 1e12, rel=1e-3)


def test_reference_arm_runs_on_rank0_only(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import argparse

    import bench

    args = argparse.Namespace(workload="c1_single_512", warmup=0, steps=1, gpus=2)
    bench.run_reference(args, rank=1)
    assert capsys.readouterr().out == ""
    bench.run_reference(args, rank=0)
    line = capsys.readouterr().out.strip()
    import json

    d = json.loads(line)
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
