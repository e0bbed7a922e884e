"""Pools of several partitions without a host wait inside the library.

Ring slots are assigned on the host, so a demotion has to know how many of its victims
fall in each partition.  kv_demote finds out by itself and waits for the answer; every
selection call also leaves the counts in pinned host memory (kv_victim_counts), and a
caller that passes them to kv_demote_counted never makes the library block.  Both ways
must give the oracle's result, and kv_stats.host_waits tells them apart."""
import numpy as np
import pytest

from paper_2604_26968_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _pool5(scale=1 / 128):
    w = W.config(5, scale=scale)
    for p in w.parts:
        p.ring_slots = w.k + 64
    return w


@pytest.mark.parametrize("fused,variant,deferred", [(True, 1, False), (False, 1, True), (False, 0, False)])
def test_counted_demotion_never_waits(fused, variant, deferred):
    from lockstep import Lockstep
    ls = Lockstep(_pool5(), payload=True, batch_bytes=1 << 20, fused=fused, counted=True,
                  select_variant=variant, deferred=deferred)
    for e in range(5):
        r = ls.epoch(e)
        assert r["promoted"] > 0
    for e in range(5, 7):      # whole paged blocks, their number of entries never read back by the call
        ls.epoch(e, k_blocks=60)
    assert ls.gpu.pool.kv_get_stats()["host_waits"] == 0
    ls.close()


def test_plain_demotion_of_several_partitions_counts_its_wait():
    from lockstep import Lockstep
    ls = Lockstep(_pool5(), payload=False, batch_bytes=1 << 20)
    for e in range(2):
        ls.epoch(e)
    assert ls.gpu.pool.kv_get_stats()["host_waits"] == 2      # one per kv_demote
    ls.close()


def test_counts_that_do_not_add_up_are_refused_before_anything_changes():
    from lockstep import Lockstep
    from paper_2604_26968_b200 import binding as B
    ls = Lockstep(_pool5(), payload=False, batch_bytes=1 << 20, counted=True)
    g, o, w = ls.gpu, ls.ora, ls.w
    ev_entry, ev_hit = w.events(0, o.pair, ls.fresh)
    d_e, d_h, n = g.stage_events(ev_entry, ev_hit)
    assert o.epoch_score(0, ev_entry, ev_hit) == 0
    g.check(g.pool.kv_epoch_score_select(0, d_e, d_h, n, w.k, g.victims), "kv_epoch_score_select")
    g.pool.sync()
    counts = g.pool.kv_victim_counts()
    bad = list(counts)
    bad[0] += 1
    assert g.pool.kv_demote_counted(g.victims, w.k, bad, g.batch_bytes) == B.KV_ERR_INVALID_ARG
    ls.compare_state("refused demotion")
    g.check(g.pool.kv_demote_counted(g.victims, w.k, counts, g.batch_bytes), "kv_demote_counted")
    rc, v = o.select_victims(w.k)
    assert o.demote(v) == 0
    ls.compare_state("demotion", scores=False)
    ls.close()


def test_counts_over_several_rows_of_chunks():
    """1.2 M entries: every CTA of the persistent selection holds two chunks, the victims per
    partition come from the pool-wide chunk table (metadata only: no block bytes move)."""
    from lockstep import Lockstep
    ls = Lockstep(_pool5(scale=1 / 16), payload=False, batch_bytes=8 << 20, fused=True, counted=True)
    for e in range(4):
        ls.epoch(e)
    assert ls.gpu.pool.kv_get_stats()["host_waits"] == 0
    ls.close()


@pytest.mark.parametrize("fused", [False, True])
def test_partition_boundaries_on_chunk_boundaries(fused):
    """Partitions of exactly 4,096 and 8,192 entries: the boundaries between them coincide with
    the chunks of the persistent selection (no chunk is split between two partitions)."""
    from lockstep import Lockstep
    parts = [W.gqa(2, 8, 4, 8, 4, 512, 3000, "entry"),      # 2 * 512 * 4 = 4,096 entries
             W.mha(2, 8, 8, 4, 512, 6000, "entry"),         # 2 * 512 * 8 = 8,192
             W.mla(3, 24, 8, 2, 333, 1000, "entry")]        # 999, ragged
    w = W.Workload("aligned_parts", parts, 0.2, 0.1, seed=5, promote_style="recent", epochs=8)
    ls = Lockstep(w, payload=False, batch_bytes=1 << 20, fused=fused, counted=True)
    for e in range(6):
        ls.epoch(e)
    assert ls.gpu.pool.kv_get_stats()["host_waits"] == 0
    ls.close()
