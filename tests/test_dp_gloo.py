"""The multi-rank host logic on gloo ranks (CPU): disjoint micro-batch ownership and the max-over-ranks
time that defines whole-job throughput; the two exchanges of the vocabulary-parallel form (all-gather of
per-row statistics in rank order, all-reduce of the dH parts), with the oracle standing in for the
kernels on each rank."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2602_05885_b200 import dp
from benchlib import synth


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rb = synth.rollout_batch(4, 8, 3, 16, 128, seed=11)
    plans = synth.pack_first_fit(rb, 700)
    owned = dp.assign_microbatches([p.used for p in plans], world)
    mine = owned[rank]
    tokens = sum(plans[i].used for i in mine)
    t_rank = 1.0 + rank            # pretend rank 1 is slower
    t_job = dp.max_over_ranks(t_rank)
    total = dp.sum_over_ranks(tokens)
    # gradient exchange by vocabulary slices, in the order in which the backward finishes them
    dW = torch.full((1000, 4), float(rank + 1))
    n_slices = dp.all_reduce_dw_slices(dW, 256)
    assert n_slices == 4 and dp.chunk_slices(1000, 256)[-1] == (768, 1000)
    assert torch.equal(dW, torch.full((1000, 4), 3.0))          # 1 + 2 on every element, every slice covered once
    # the same exchange as a reduce-scatter: every rank keeps its rows of each slice only (ragged slice ends and
    # a last slice of 232 rows included); together the ranks hold every row of the sum exactly once
    V, vc = 1001, 256
    g = torch.Generator().manual_seed(100)
    parts = [torch.randn((V, 4), generator=g) for _ in range(world)]
    mine_rows = dp.dw_shard_rows(V, vc, world, rank)
    shard = torch.empty((sum(b - a for a, b in mine_rows), 4))
    assert dp.reduce_scatter_dw_slices(parts[rank].clone(), vc, shard) == 4
    want = torch.cat([(parts[0] + parts[1])[a:b] for a, b in mine_rows])
    assert torch.allclose(shard, want, atol=1e-6)
    covered = sorted(r for k in range(world) for r in dp.dw_shard_rows(V, vc, world, k))
    assert covered[0][0] == 0 and covered[-1][1] == V and all(x[1] == y[0] for x, y in zip(covered, covered[1:]))
    # partial sums of dH never cross the ranks in 16 bits
    try:
        dp.all_reduce_dh(torch.zeros(4, dtype=torch.bfloat16))
        raise AssertionError("bf16 partial sums must be refused")
    except ValueError:
        pass
    out.put((rank, mine, tokens, t_job, total, len(plans), sum(p.used for p in plans)))
    dist.destroy_process_group()


def test_two_rank_sharding_and_timing():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, a, ta, ja, tot_a, n, all_tokens), (_, b, tb, jb, tot_b, _, _) = res
    assert sorted(a + b) == list(range(n)) and not set(a) & set(b)     # every micro-batch exactly once
    assert ja == jb == 2.0                                             # job time = slowest rank
    assert tot_a == tot_b == all_tokens == ta + tb
    assert abs(ta - tb) <= 700                                         # balanced within one micro-batch


def test_assignment_balances_and_covers():
    loads = [700, 10, 650, 640, 30, 500, 20]
    owned = dp.assign_microbatches(loads, 3)
    assert sorted(i for o in owned for i in o) == list(range(7))
    tot = [sum(loads[i] for i in o) for o in owned]
    assert max(tot) - min(tot) <= 700
    assert dp.max_over_ranks(3.5) == 3.5 and dp.sum_over_ranks(2.0) == 2.0   # no process group: identity


def _vocab_worker(rank, world, port, out):
    from oracle import drk_oracle as O
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rng = np.random.default_rng(5)                       # the same micro-batch on every rank
    T, H, V = 12, 8, 700
    hidden, W = rng.normal(size=(T, H)), rng.normal(size=(V, H))
    ids = rng.integers(0, V, size=T)
    coeff = rng.normal(size=T)
    a, b = dp.vocab_shards(V, world)[rank]
    s = O.logits(hidden, W)
    stats = torch.from_numpy(O.shard_stats(s, ids, a, b))
    stats_all = dp.all_gather_stats(stats)
    assert stats_all.shape == (world, T, 4) and torch.equal(stats_all[rank], stats)
    logp, lse, ent = O.merge_shard_stats(stats_all.numpy())
    dH_part, dW_rows = O.shard_gradients(hidden, W, s, lse, ids, coeff, a, b)
    dH = dp.all_reduce_dh(torch.from_numpy(dH_part.copy()))
    out.put((rank, (a, b), logp, lse, dH.numpy(), dW_rows))
    dist.destroy_process_group()


def test_vocabulary_parallel_exchanges_on_three_ranks():
    from oracle import drk_oracle as O
    world = 3
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_vocab_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=120) for _ in procs), key=lambda r: r[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    rng = np.random.default_rng(5)
    T, H, V = 12, 8, 700
    hidden, W = rng.normal(size=(T, H)), rng.normal(size=(V, H))
    ids = rng.integers(0, V, size=T)
    coeff = rng.normal(size=T)
    s = O.logits(hidden, W)
    logp, lse = O.token_logprob(s, ids)
    dH, dW = O.gradients(hidden, W, s, lse, ids, coeff)
    ranges = [r[1] for r in res]
    assert ranges == [(0, 256), (256, 512), (512, 700)]          # tiles of 256 rows, the last rank takes the rest
    for _, _, lp, z, dh, _ in res:                                # identical, complete results on every rank
        assert np.abs(lp - logp).max() < 1e-12 and np.abs(z - lse).max() < 1e-12
        assert np.abs(dh - dH).max() < 1e-12
    assert np.abs(np.concatenate([r[5] for r in res]) - dW).max() < 1e-12


def test_vocab_shards_cover_the_vocabulary():
    import pytest
    for V, world, align in ((151936, 8, 256), (151936, 2, 256), (151936, 1, 256), (4096, 3, 256), (300, 2, 256),
                            (300, 4, 32)):
        sh = dp.vocab_shards(V, world, align)
        assert len(sh) == world and sh[0][0] == 0 and sh[-1][1] == V
        assert all(a[1] == b[0] for a, b in zip(sh, sh[1:])) and all(b > a for a, b in sh)
        assert all(a % align == 0 for a, _ in sh)
    # more ranks than vocabulary tiles: a clear error instead of an empty range that the library would reject
    with pytest.raises(ValueError, match="without rows"):
        dp.vocab_shards(300, 4)


def test_reduce_scatter_without_a_process_group_keeps_every_row():
    dW = torch.arange(40, dtype=torch.float32).reshape(10, 4)
    rows = dp.dw_shard_rows(10, 4, 1, 0)
    assert rows == [(0, 4), (4, 8), (8, 10)]
    shard = torch.empty((10, 4))
    assert dp.reduce_scatter_dw_slices(dW, 4, shard) == 3 and torch.equal(shard, dW)
