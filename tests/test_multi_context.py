"""The subgraphs of Algorithm 2 spread over several contexts, checked on the CPU: the orchestration classes of the
package driven by oracle-backed engines.  Two gloo ranks with half of the subgraphs each must reach the model of one
oracle run over all of them (the weighted consensus of Section 3.4.2 is a sum over subgraphs, so it splits over
ranks); rounds must hand the model on from one to the next."""
import json
import os
import socket
import sys

import numpy as np
import torch.multiprocessing as mp

from conftest import small_random_case, flat, rel_err
from gad_synth import glorot_params

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
DIMS, LR, STEPS = (7, 6, 3), 0.3, 3


def _inputs(case, seed=5):
    n = case[0]
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((n, DIMS[0])).astype(np.float32)
    y = rng.integers(0, DIMS[-1], size=n).astype(np.int32)
    split = rng.integers(0, 3, size=n).astype(np.uint8)
    return X, y, split, glorot_params(DIMS, rng, bias_scale=0.2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank, world, port, out, weighted):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import torch.distributed as dist
    from oracle_engine import OracleEngine
    from paper_2110_02987_b200.multi import ShardedEpoch, shard_subgraphs
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    case = small_random_case(11, n=60, K=4)
    X, y, split, theta = _inputs(case)
    eng = OracleEngine(case, shard_subgraphs(4, world, rank), X, y, split, DIMS, theta, LR, weighted=weighted)
    sh = ShardedEpoch(eng, weighted=weighted)
    losses = [sh.step() for _ in range(STEPS)]
    with open(os.path.join(out, "rank%d.json" % rank), "w") as fh:
        json.dump({"loss": losses, "params": eng.model.get_params(0).tolist()}, fh)
    dist.barrier()
    dist.destroy_process_group()


def _whole(weighted, seed=11):
    from oracle import gad_oracle as orc
    case = small_random_case(seed, n=60, K=4)
    n, rowptr, col, w, core, halo = case
    X, y, split, theta = _inputs(case)
    st = orc.Store(n, rowptr, col, *flat(core), *flat(halo), weights=w)
    m = orc.Model(st, X, y, split, DIMS, theta, lr=LR, weighted=weighted)
    losses = [float(m.train_epoch()[-1]) for _ in range(STEPS)]
    return losses, m.get_params(0)


def _check_two_ranks(tmp_path, weighted):
    world = 2
    mp.spawn(_rank, args=(world, _free_port(), str(tmp_path), weighted), nprocs=world, join=True)
    got = [json.load(open(tmp_path / ("rank%d.json" % r))) for r in range(world)]
    losses, params = _whole(weighted)
    for g in got:
        assert np.max(np.abs(np.array(g["loss"]) - np.array(losses))) <= 1e-12
        assert rel_err(np.array(g["params"]), params) <= 1e-12
    assert got[0]["params"] == got[1]["params"]      # one all-reduce: bit-identical models on both ranks


def test_two_ranks_reach_the_model_of_one_run_over_all_subgraphs(tmp_path):
    _check_two_ranks(tmp_path, True)


def test_two_ranks_plain_average(tmp_path):
    _check_two_ranks(tmp_path, False)


def test_one_rank_needs_no_process_group():
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from oracle_engine import OracleEngine
    from paper_2110_02987_b200.multi import ShardedEpoch
    case = small_random_case(11, n=60, K=4)
    X, y, split, theta = _inputs(case)
    eng = OracleEngine(case, [0, 1, 2, 3], X, y, split, DIMS, theta, LR)
    sh = ShardedEpoch(eng)
    losses = [sh.step() for _ in range(STEPS)]
    want, params = _whole(True)
    assert np.max(np.abs(np.array(losses) - np.array(want))) <= 1e-12
    assert rel_err(eng.model.get_params(2), params) <= 1e-12


def test_rounds_hand_the_model_from_one_to_the_next():
    """z = 2 rounds of two subgraphs: round 1 must start from round 0's consensus, and the next epoch's round 0 from
    round 1's.  The expected run is written out with two oracle models and explicit parameter copies."""
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from oracle_engine import OracleEngine
    from paper_2110_02987_b200.multi import RoundsEpoch
    case = small_random_case(12, n=60, K=4)
    X, y, split, theta = _inputs(case)
    engines = [OracleEngine(case, [0, 1], X, y, split, DIMS, theta, LR), OracleEngine(case, [2, 3], X, y, split, DIMS, theta, LR)]
    rounds = RoundsEpoch(engines)
    a = OracleEngine(case, [0, 1], X, y, split, DIMS, theta, LR).model
    b = OracleEngine(case, [2, 3], X, y, split, DIMS, theta, LR).model
    for _ in range(2):
        got = rounds.step()
        la = a.train_epoch()
        for k in range(2):
            b.set_params(k, a.get_params(0))
        lb = b.train_epoch()
        for k in range(2):
            a.set_params(k, b.get_params(0))
        assert np.array_equal(got[0], la) and np.array_equal(got[1], lb)
    assert np.array_equal(engines[0].model.get_params(1), a.get_params(1))
    assert np.array_equal(engines[1].model.get_params(0), b.get_params(0))
    # the two rounds really differ from one epoch over all four subgraphs at once
    assert rel_err(engines[0].model.get_params(0), _whole(True, seed=12)[1]) > 1e-6
