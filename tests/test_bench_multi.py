"""The N > 1 path of bench.py is "replicas only": every rank runs the whole job, the step time is the maximum over
ranks and the value the sum of the replicas' work.  Checked here with two gloo ranks on the CPU."""
import json
import os
import socket
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world)        # rank 1 is the slow one
    with open(os.path.join(out, "rank%d.json" % rank), "w") as fh:
        json.dump([ms, bench.job_value(20, world, ms)], fh)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_agree_on_the_slowest_time_and_sum_the_work(tmp_path):
    world = 2
    mp.spawn(_rank, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    got = [json.load(open(tmp_path / ("rank%d.json" % r))) for r in range(world)]
    assert got[0] == got[1]
    ms, value = got[0]
    assert ms == 15.0
    assert abs(value - 2 * 20 / 15e-3) < 1e-9


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.job_value(10, 1, 5.0) == 2000.0


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0", "--workload", "tiny"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_reference_arm_prints_the_contract_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2", "--warmup", "1",
                        "--workload", "tiny"], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "epochs/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": "epochs/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


def test_oracle_sample_is_sized_from_a_pilot_and_never_times_the_whole_workload():
    """With a step budget far below one epoch the reference arm takes the leading core rows of subgraph 0 as a block of
    their own and scales by their share of the store rows; with a generous budget it runs whole epochs."""
    import numpy as np
    sys.path.insert(0, ROOT)
    import bench
    from gad_synth import make_workload, glorot_params
    w = make_workload("c2", scale=0.2)
    theta = glorot_params(w.dims, np.random.default_rng(0))
    m, frac, sample = bench.oracle_sample(w, theta, 1e-4)
    rows_all = sum(len(c) + len(h) for c, h in zip(w.core, w.halo))
    assert 0.0 < frac < 1.0 and "pilot" in sample
    assert m.store.K == 1 and m.store.n_prime == round(frac * rows_all) and m.store.n_prime >= 2000
    assert np.all(np.isfinite(m.train_epoch()))
    m.close()
    m, frac, sample = bench.oracle_sample(w, theta, 1e9)
    assert frac == 1.0 and m.store.K == w.K
    m.close()
