"""Deferred packing: the demotion's later chunks are enqueued interleaved with the
promotion's chunks.  Results must be exactly those of the plain order (and of
the oracle), in particular the payload bytes of promoted blocks that land in
slots the same epoch's demotion freed."""
import numpy as np
import pytest

from paper_2604_26968_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg,scale,batch_kb,epochs", [
    (1, 1.0, 16, 20),        # 4 entries per chunk: 51 demote chunks, 20 promote chunks per epoch
    (1, 1.0, 256, 10),
    (2, 1 / 64, 512, 6),
    (3, 1 / 192, 1024, 4),   # promotes 10 %, demotes 15 %
    (4, 1 / 128, 2048, 5),   # 72 KB MLA entries
    (5, 1 / 128, 1024, 5),   # four partitions, promotions per partition
])
def test_deferred_packing_matches_the_oracle(cfg, scale, batch_kb, epochs):
    from lockstep import Lockstep
    w = W.config(cfg, scale=scale)
    if cfg == 5:
        for p in w.parts:
            p.ring_slots = w.k + 64
    ls = Lockstep(w, payload=True, batch_bytes=batch_kb << 10, deferred=True)
    for e in range(epochs):
        r = ls.epoch(e)
        assert r["promoted"] > 0
    ls.close()


def test_deferred_packing_with_promotions_of_just_demoted_slots_and_block_mode():
    from lockstep import Lockstep
    # "recent" promote lists name slots that the same epoch's demotion writes: the demotion must be
    # fully enqueued before the promotion's copies wait for it
    w = W.Workload("recent", [W.gqa(2, 8, 4, 16, 8, 300, 900, "entry")], 0.2, 0.1, seed=13, promote_style="recent")
    ls = Lockstep(w, payload=True, batch_bytes=8 << 10, deferred=True)
    for e in range(8):
        ls.epoch(e)
    for e in range(8, 12):
        ls.epoch(e, k_blocks=40)
    ls.close()


@pytest.mark.parametrize("cfg,scale,batch_kb,pieces", [
    (1, 1.0, 16, 3),         # 81 promotions in calls of 27: the later calls land beyond the first victims
    (2, 1 / 64, 256, 4),
    (5, 1 / 128, 512, 2),
])
def test_deferred_packing_with_several_promotions_per_partition(cfg, scale, batch_kb, pieces):
    """A promote list longer than max_promote has to be split by the caller, so several
    kv_promote calls on one partition between a demotion and the next draining call are
    normal.  Every later call scatters into freed slots further up the victim list, whose
    payload must have been packed by then: ring bytes of those victims and slab bytes of
    the promoted blocks are compared in full."""
    from lockstep import Lockstep
    w = W.config(cfg, scale=scale)
    if cfg == 5:
        for p in w.parts:
            p.ring_slots = w.k + 64
    ls = Lockstep(w, payload=True, batch_bytes=batch_kb << 10, deferred=True, split_promote=pieces)
    for e in range(6):
        r = ls.epoch(e)
        assert r["promoted"] > 0
    ls.close()
