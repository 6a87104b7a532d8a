"""The exchange wiring of the vocabulary-sharded round over torch.distributed (gloo, two ranks, CPU): the
three all-gathers must deliver every rank's block in rank order to every rank.  The library calls need a
GPU, so a stand-in with the ShardedRound interface takes their place here: its four methods tag what they
produce with the rank and check what they receive; csd_verify_sharded itself is the code under test."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


class FakeRound:
    def __init__(self, rank, n, B=3, rows=7):
        self.rank, self.n, self.B, self.rows = rank, n, B, rows
        self.emitted = None

    def stats(self):
        return torch.full((self.rows, 4), float(self.rank), dtype=torch.float32)

    def partial(self, records_all, dbg_p=None, dbg_q=None, dbg_f=None):
        assert records_all.shape == (self.n, self.rows, 4)
        for r in range(self.n):
            assert torch.all(records_all[r] == float(r))
        return torch.full((self.B, 2), 10.0 + self.rank, dtype=torch.float64)

    def pick(self, totals_all):
        assert totals_all.shape == (self.n, self.B, 2) and totals_all.dtype == torch.float64
        for r in range(self.n):
            assert torch.all(totals_all[r] == 10.0 + r)
        return torch.full((self.B, 2), 100 + self.rank, dtype=torch.int32)

    def emit(self, cand_all, out_tokens, out_accept_len, out_status=None):
        assert cand_all.shape == (self.n, self.B, 2) and cand_all.dtype == torch.int32
        for r in range(self.n):
            assert torch.all(cand_all[r] == 100 + r)
        out_tokens.fill_(int(cand_all.max()))
        out_accept_len.fill_(self.n)
        self.emitted = True


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2601_09212_b200.vocab_sharded import csd_verify_sharded
        rd = FakeRound(rank, world)
        out_t = torch.zeros(3, 5, dtype=torch.int32)
        out_l = torch.zeros(3, dtype=torch.int32)
        csd_verify_sharded(rd, out_t, out_l)
        q.put((rank, bool(rd.emitted), int(out_t[0, 0]), int(out_l[0])))
    finally:
        dist.destroy_process_group()


def test_three_all_gathers_deliver_rank_major_blocks():
    world = 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == [(0, True, 101, 2), (1, True, 101, 2)]
