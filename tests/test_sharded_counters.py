"""The sharded (one pool per GPU) form of the predictor update, on CPU with gloo.

Each rank owns its entries and sees only its own events; the 16 Beta pairs are
shared, so ranks sum their 32 per-epoch (pair, hit) counters before forming the
posterior -- the exchange bench.py does with one 256-byte NCCL all-reduce
between kv_epoch_events and kv_epoch_update.  Checked here against the oracle:
the all-reduced counters give exactly the posterior a single pool seeing all
events would compute.
"""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import kv_oracle as O


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _pool(blocks, pairs):
    part = dict(model=O.model(variant=O.GQA, n_layers=1, n_q_heads=8, n_kv_heads=2, head_dim=8),
                block_tokens=4, blocks_per_layer=blocks, ring_slots=8)
    p = O.OraclePool([part], n_tags=4 * blocks, payload=False)
    p.admit(0, 0.9, pairs, None)
    return p


def _events(rank, epoch, n_entries, n):
    r = np.random.default_rng([rank, epoch])
    return r.integers(0, n_entries, n).astype(np.uint32), (r.random(n) < 0.3 + 0.4 * rank).astype(np.uint8)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    blocks = 50 + 10 * rank
    pairs = np.random.default_rng(100 + rank).integers(0, 16, 2 * blocks, dtype=np.uint8)
    hits = np.zeros(16, np.int64)
    misses = np.zeros(16, np.int64)
    P = None
    for epoch in range(3):
        ev, hit = _events(rank, epoch, 2 * blocks, 400 + 50 * rank)
        counts = np.zeros(32, np.int64)                  # index 2*pair + hit, as the library lays them out
        np.add.at(counts, 2 * pairs[ev].astype(np.int64) + hit, 1)
        t = torch.from_numpy(counts)
        dist.all_reduce(t)
        hits += t.numpy()[1::2]
        misses += t.numpy()[0::2]
        a = np.float32(1.0) + hits.astype(np.float32)
        b = np.float32(1.0) + misses.astype(np.float32)
        P = a / (a + b)
    out[rank] = (hits.copy(), misses.copy(), P.copy())
    dist.destroy_process_group()


def test_all_reduced_pair_counters_equal_single_pool_oracle():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Manager().dict()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    # one oracle pool holding both ranks' entries, fed both ranks' events
    blocks = [50, 60]
    pairs = [np.random.default_rng(100 + r).integers(0, 16, 2 * blocks[r], dtype=np.uint8) for r in range(world)]
    big = _pool(sum(blocks), np.concatenate(pairs))
    base = [0, 2 * blocks[0]]
    for epoch in range(3):
        evs, hs = [], []
        for r in range(world):
            ev, hit = _events(r, epoch, 2 * blocks[r], 400 + 50 * r)
            evs.append(ev + base[r])
            hs.append(hit)
        assert big.epoch_score(epoch, np.concatenate(evs), np.concatenate(hs)) == O.OK
    for r in range(world):
        hits, misses, P = out[r]
        assert np.array_equal(hits.astype(np.uint64), big.hits)
        assert np.array_equal(misses.astype(np.uint64), big.misses)
        assert np.array_equal(P.view(np.uint32), big.P.view(np.uint32))
