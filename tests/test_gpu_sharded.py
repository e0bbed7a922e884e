"""The sharded form of kv_epoch_score on one GPU.

Two pools stand for two ranks.  Each reduces its own events (kv_epoch_events);
the 32 epoch counters of the two pools are summed and written back to both (what
the NCCL all-reduce does across GPUs); each then runs kv_epoch_update.  Nothing
here waits on another kernel: the pools run one after the other on one stream.
The result must equal ONE oracle pool that holds both ranks' entries and sees
all events: same posteriors, and the same EMA and scores per entry.
"""
import numpy as np
import pytest

from oracle import kv_oracle as O
from paper_2604_26968_b200 import binding as B
from paper_2604_26968_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_two_pools_with_summed_pair_counters_equal_one_oracle_pool():
    import torch
    from paper_2604_26968_b200.harness import EpochRunner, INITIAL_EPOCH_KEY
    blocks = [700, 1100]
    ws = [W.Workload("rank%d" % r, [W.gqa(2, 8, 2, 8, 4, blocks[r], 64, "entry")], 0.05, 0.0, seed=20 + r)
          for r in range(2)]
    runners = [EpochRunner(w, batch_bytes=1 << 20) for w in ws]
    # the oracle: one pool with both ranks' entries (two partitions), same pair ids
    parts = [dict(model=O.Model(p.variant, p.n_layers, p.n_q_heads, p.n_kv_heads, p.head_dim, p.d_latent,
                                p.d_rope, p.dtype_bits),
                  block_tokens=p.block_tokens, blocks_per_layer=p.blocks_per_layer, ring_slots=p.ring_slots)
             for p in (ws[0].parts[0], ws[1].parts[0])]
    ora = O.OraclePool(parts, n_tags=1 << 16, payload=False)
    pairs = [w.new_pairs(INITIAL_EPOCH_KEY, w.N) for w in ws]
    assert ora.admit(0, ws[0].decay, np.concatenate(pairs), None) == ws[0].N + ws[1].N
    base = [0, ws[0].N]
    for r in range(2):
        assert np.array_equal(runners[r].host_array("pair"), pairs[r])
    for epoch in range(5):
        evs = []
        for r, run in enumerate(runners):
            ev_entry, ev_hit = ws[r].events(epoch, pairs[r])
            evs.append((ev_entry, ev_hit))
            d_e, d_h, n = run.stage_events(ev_entry, ev_hit)
            run.check(run.pool.kv_epoch_events(d_e, d_h, n), "kv_epoch_events")
        # "all-reduce": sum the two pools' epoch counters and give every pool the sum
        for run in runners:
            run.pool.sync()
        total = runners[0].pool.kv_epoch_counts().clone() + runners[1].pool.kv_epoch_counts()
        for run in runners:
            run.pool.kv_epoch_counts().copy_(total)
        torch.cuda.synchronize()
        for run in runners:
            run.check(run.pool.kv_epoch_update(epoch), "kv_epoch_update")
        all_e = np.concatenate([evs[r][0].astype(np.int64) + base[r] for r in range(2)]).astype(np.uint32)
        all_h = np.concatenate([evs[r][1] for r in range(2)])
        assert ora.epoch_score(epoch, all_e, all_h) == O.OK
        for r, run in enumerate(runners):
            lo, hi = base[r], base[r] + ws[r].N
            assert np.array_equal(run.host_array("hits"), ora.hits)
            assert np.array_equal(run.host_array("misses"), ora.misses)
            assert np.array_equal(run.host_array("P").view(np.uint32), ora.P.view(np.uint32))
            assert np.array_equal(run.host_array("ema").view(np.uint32), ora.ema[lo:hi].view(np.uint32))
            assert np.array_equal(run.host_array("score").view(np.uint32), ora.score[lo:hi].view(np.uint32))
            assert run.pool.kv_device_status() == 0
    for run in runners:
        run.close()
