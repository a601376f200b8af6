"""Multi-process CPU test (gloo, world size 2) of the replica bookkeeping that bench.py uses for
runs on several GPUs: independent seeds per rank, barrier, maximum over ranks of the measured
time, and the whole-job metric. Also checks that two replicas' synthetic inputs differ and that the
same rank's inputs are reproducible, since replicas must be independent (no exchange on the path).
"""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    if ROOT not in sys.path:
        sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    from paper_2609_35629_b200 import replicas, synth
    assert replicas.env_rank_world() == (rank, world, rank)
    assert replicas.init_replicas("gloo") == world
    seed = replicas.replica_seed(1234, rank)
    spec = synth.spec_tiny(seed=seed)
    data = synth.make_layer(spec, layer=0)
    digest = int(np.asarray(data.k_prompt, dtype=np.uint64).sum())
    replicas.barrier()
    # each rank "measures" a different time; the job's time is the slowest rank's
    ms_local = 10.0 + 5.0 * rank
    ms = replicas.max_over_ranks(ms_local)
    value = replicas.us_per_layer_step(ms, steps=4, layers=2, world=world)
    replicas.barrier()
    torch.save({"rank": rank, "seed": seed, "digest": digest, "ms": ms, "value": value},
               os.path.join(out_dir, f"r{rank}.pt"))
    torch.distributed.destroy_process_group()


@pytest.mark.timeout(180)
def test_two_replicas_over_gloo(tmp_path):
    world = 2
    port = _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = [torch.load(os.path.join(str(tmp_path), f"r{r}.pt")) for r in range(world)]
    assert [r["seed"] for r in res] == [1234, 1235]
    assert res[0]["digest"] != res[1]["digest"]                       # replicas own different sequences
    assert all(r["ms"] == 15.0 for r in res)                          # max over ranks, on every rank
    # 2 ranks x 4 steps x 2 layers = 16 layer-steps in 15 ms
    assert all(abs(r["value"] - 15.0e3 / 16) < 1e-9 for r in res)


def test_single_process_is_a_no_op():
    if ROOT not in sys.path:
        sys.path.insert(0, ROOT)
    from paper_2609_35629_b200 import replicas
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    assert replicas.env_rank_world() == (0, 1, 0)
    assert replicas.init_replicas("gloo") == 1
    replicas.barrier()
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.us_per_layer_step(2.0, steps=4, layers=5, world=1) == 100.0


def test_replica_inputs_reproducible():
    from paper_2609_35629_b200 import replicas, synth
    a = synth.make_layer(synth.spec_tiny(seed=replicas.replica_seed(7, 1)), layer=0)
    b = synth.make_layer(synth.spec_tiny(seed=replicas.replica_seed(7, 1)), layer=0)
    assert np.array_equal(a.k_prompt, b.k_prompt) and np.array_equal(a.v_prompt, b.v_prompt)
