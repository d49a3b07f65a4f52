"""The multi-rank paths on CPU: two gloo ranks exercise the exchange of the batch-wide Alloc-T (all-gather of the
score rows, identical selection on every rank, slicing) and the max-over-ranks timing reduce.  The selection itself
is the library's kernel on a GPU; here a stand-in written from the oracle takes its place, so what is tested is the
plumbing around it."""
import os

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import alloc_moe_oracle as orc
from paper_2604_08133_b200 import dist as D
from paper_2604_08133_b200 import synth


def _oracle_select(pool, K_base, budget):
    return torch.from_numpy(orc.n_sel_from_mask(orc.alloc_t_select(pool.numpy(), K_base, budget)).astype(np.int32))


def _worker(rank, world, port, T, K, K_base, budget, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        full = synth.score_rows(world * T, K, 99, ties=True)          # the whole batch, same on every rank
        mine = full[rank * T:(rank + 1) * T].clone()
        n_sel, b_local = D.alloc_t_select_global(mine, K_base, budget, select=_oracle_select)
        slow = D.max_over_ranks(10.0 + rank)                          # rank 1 is "slower"
        q.put((rank, n_sel.numpy(), int(b_local), slow))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("T,K,K_base,mult", [(64, 6, 1, 3.0), (33, 4, 0, 1.5)])
def test_global_selection_over_two_gloo_ranks(T, K, K_base, mult):
    world = 2
    budget = int(mult * world * T)
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, world, port, T, K, K_base, budget, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    got.sort(key=lambda g: g[0])
    full = synth.score_rows(world * T, K, 99, ties=True).numpy()
    want = orc.n_sel_from_mask(orc.alloc_t_select(full, K_base, budget))
    # every rank holds exactly its slice of the one batch-wide selection; the shares add up to the budget
    for r, n_sel, b_local, slow in got:
        assert np.array_equal(n_sel, want[r * T:(r + 1) * T])
        assert b_local == int(want[r * T:(r + 1) * T].sum())
        assert slow == 11.0
    assert sum(g[2] for g in got) == budget
    # and it differs from two independent selections with the budget split evenly (the ranks' scores differ)
    indep = np.concatenate([orc.n_sel_from_mask(orc.alloc_t_select(full[r * T:(r + 1) * T], K_base, budget // world))
                            for r in range(world)])
    assert not np.array_equal(indep, want)


def test_single_process_is_the_identity():
    s = synth.score_rows(16, 3, 5)
    n_sel, b = D.alloc_t_select_global(s, 1, 30, select=_oracle_select)
    assert int(b) == 30 and np.array_equal(n_sel.numpy(), orc.n_sel_from_mask(orc.alloc_t_select(s.numpy(), 1, 30)))
    assert D.max_over_ranks(3.5) == 3.5
