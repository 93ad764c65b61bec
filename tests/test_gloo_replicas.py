"""The evaluation step does not shard across GPUs with an exchange: candidates are independent,
so several GPUs run replicas over disjoint candidates.  This checks, with two CPU processes over
gloo, that splitting a population by candidate id and gathering the per-rank results gives the
same records and verdicts as one pass (records are computed by the oracle here: no GPU)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import workloads


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out_dir):
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    pop = workloads.config5("cpu", n_cand=24, log2_min=4.0, log2_max=12.0, trials=4)
    mine = workloads.shard_by_candidate(pop, rank, world)
    res = np.zeros(len(mine), dtype=oracle.RESULT_DTYPE)
    for j, i in enumerate(mine):
        t = pop.tensors[i]
        res[j] = oracle.validate(workloads.to_host_bits(t.cand), workloads.to_host_bits(pop.refs[t.ref_index]),
                                 t.dtype, pop.atol, pop.rtol)
    gathered = [None] * world
    dist.all_gather_object(gathered, (mine, res.tobytes()))
    if rank == 0:
        full = np.zeros(len(pop.tensors), dtype=oracle.RESULT_DTYPE)
        seen = []
        for idx, raw in gathered:
            full[idx] = np.frombuffer(raw, dtype=oracle.RESULT_DTYPE)
            seen += idx
        assert sorted(seen) == list(range(len(pop.tensors)))
        np.save(os.path.join(out_dir, "sharded.npy"), full)
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_cover_the_population(tmp_path):
    import oracle
    from parity import oracle_population
    port = _free_port()
    mp.start_processes(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True, start_method="spawn")
    full = np.load(os.path.join(str(tmp_path), "sharded.npy"))
    pop = workloads.config5("cpu", n_cand=24, log2_min=4.0, log2_max=12.0, trials=4)
    want, _ = oracle_population(pop)
    assert full.tobytes() == want.tobytes()
