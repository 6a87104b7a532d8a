"""The N > 1 path on CPU: two gloo ranks each verify their shard of a batch (with the oracle standing
in for the device path) and the pieces must tile the unsharded result exactly; the timing reduction
must return the slowest rank's time on every rank."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2601_09212_b200 import sharding
from paper_2601_09212_b200 import workloads as W


def test_shard_bounds_tile_the_batch():
    for n in (0, 1, 7, 64, 65, 256):
        for world in (1, 2, 3, 8):
            cuts = [sharding.shard_bounds(n, world, r) for r in range(world)]
            assert cuts[0][0] == 0 and cuts[-1][1] == n
            assert all(cuts[i][1] == cuts[i + 1][0] for i in range(world - 1))
            sizes = [e - b for b, e in cuts]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.shard_bounds(4, 2, 2)
    assert sharding.job_throughput(512, 8, 0.5) == 8192.0


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    oracle.build()
    oracle.set_num_threads(1)
    B, L, V = 9, 4, 512
    sched = oracle.make_schedule(1, 1.1, 0.7, L).astype(np.float32)
    w = W.make("t", B=B, gamma=L, V=V, rho=0.9, bonus_row=True, schedule=sched, seed=3, device="cpu")
    h = w.host_arrays()
    b0, b1 = sharding.shard_bounds(B, world, rank)
    ref = oracle.verify(h["target_logits"][b0:b1], h["draft_logits"][b0:b1], h["draft_tokens"][b0:b1],
                        h["uniforms"][b0:b1], h["relax_schedule"], dtype=w.dtype, want_G=False)
    np.save(os.path.join(out_dir, f"tok{rank}.npy"), ref.tokens)
    np.save(os.path.join(out_dir, f"tau{rank}.npy"), ref.accept_len)
    slowest = sharding.max_over_ranks(0.25 * (rank + 1))
    np.save(os.path.join(out_dir, f"t{rank}.npy"), np.array([slowest]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_tile_the_unsharded_result(tmp_path, oracle):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    B, L, V = 9, 4, 512
    sched = oracle.make_schedule(1, 1.1, 0.7, L).astype(np.float32)
    w = W.make("t", B=B, gamma=L, V=V, rho=0.9, bonus_row=True, schedule=sched, seed=3, device="cpu")
    h = w.host_arrays()
    full = oracle.verify(h["target_logits"], h["draft_logits"], h["draft_tokens"], h["uniforms"],
                         h["relax_schedule"], dtype=w.dtype, want_G=False)
    tok = np.concatenate([np.load(tmp_path / f"tok{r}.npy") for r in range(world)])
    tau = np.concatenate([np.load(tmp_path / f"tau{r}.npy") for r in range(world)])
    assert np.array_equal(tok, full.tokens) and np.array_equal(tau, full.accept_len)
    for r in range(world):
        assert np.load(tmp_path / f"t{r}.npy")[0] == 0.5
