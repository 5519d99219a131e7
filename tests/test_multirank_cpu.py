"""The multi-GPU run shards flows across ranks with no data-path collective; the only
communication is the max of the elapsed times.  Exercised here with two gloo ranks on CPU:
per-rank inputs differ and are reproducible, the slowest rank sets the job's time, and the
whole-job figure counts every rank's flows.  The oracle stands in for the per-rank work."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close()
    return p


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import flowgen
    import oracle
    cfg = flowgen.get_config(1)
    n = 512
    wide = flowgen.gen_packets(bench.rank_data_seed(cfg, rank), n, cfg.P, cfg.H)
    feat = oracle.extract_features(flowgen.fast_view(wide, cfg.N), cfg.N, cfg.F)
    ms_local = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    ms = bench.max_over_ranks(ms_local, dist, torch.device("cpu"))
    value = bench.whole_job_flows_per_s(world, n, 4, ms)
    # every rank's digest, gathered only to check the sharding in this test
    dig = torch.tensor([float(feat.astype(np.float64).sum())], dtype=torch.float64)
    all_d = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(all_d, dig)
    if rank == 0:
        out.put({"ms": ms, "value": value, "digests": [float(x) for x in all_d]})
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_flows_and_take_the_slowest_time():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res["ms"] == 15.0
    assert res["value"] == pytest.approx(2 * 512 * 4 / 0.015)
    assert res["digests"][0] != res["digests"][1]              # different shards
    import bench, flowgen, oracle
    cfg = flowgen.get_config(1)
    w0 = flowgen.gen_packets(bench.rank_data_seed(cfg, 0), 512, cfg.P, cfg.H)
    f0 = oracle.extract_features(flowgen.fast_view(w0, cfg.N), cfg.N, cfg.F)
    assert res["digests"][0] == float(f0.astype(np.float64).sum())     # reproducible per rank


def test_reference_arm_runs_on_rank0_only(tmp_path):
    import subprocess
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""            # other ranks exit 0 without work
    env = dict(os.environ, RANK="0", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1", "--steps", "1",
                        "--warmup", "0", "--ref-flows", "256"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0
    import json
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["unit"] == "flows/s"
