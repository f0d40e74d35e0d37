"""Frozen oracle values (regression pin) and the multi-rank plumbing of the benchmark on CPU."""
import importlib.util
import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _load(path, name):
    spec = importlib.util.spec_from_file_location(name, path)
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_oracle_matches_frozen_values(oracle):
    """tests/golden/oracle_cfg0.txt was written by make_golden.py from the oracle alone; a change of
    the oracle's arithmetic must show up here."""
    mk = _load(os.path.join(ROOT, "tests", "golden", "make_golden.py"), "make_golden")
    now = mk.compute()
    stored = {}
    for line in open(os.path.join(ROOT, "tests", "golden", "oracle_cfg0.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, *vals = line.split()
        stored[name] = np.array([float(x) for x in vals])
    assert set(stored) == set(now)
    for name, vals in now.items():
        np.testing.assert_allclose(np.asarray(vals, np.float64), stored[name], rtol=1e-12, atol=0, err_msg=name)


def _rank_main(rank, world, port, out):
    import torch
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    bench = _load(os.path.join(ROOT, "bench.py"), "bench_mod")
    bench.barrier(world)
    # every rank times its own replica; the job's time is the slowest rank's
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, torch.device("cpu"))
    slots = bench.algorithmic_work(bench.inputs.CONFIGS[1])[0]
    out[rank] = (ms, world * slots / (ms * 1e-3) / 1e9)
    bench.barrier(world)
    dist.destroy_process_group()


def test_two_rank_replica_timing_on_gloo():
    """N > 1 runs N independent replicas (units never exchange data): the only cross-rank steps are
    the barrier and the max over ranks of the step time.  Checked with two gloo ranks on CPU."""
    import torch.multiprocessing as mp
    world = 2
    port = 29500 + (os.getpid() % 2000)
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 15.0                       # max over ranks, seen by both
    slots = 65536
    assert res[0][1] == pytest.approx(world * slots / 15.0e-3 / 1e9)
