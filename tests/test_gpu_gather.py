"""Promotion of position-ordered (fragmented) lists.

The long-context pool's prefetch list names, for every block of a sequence's next
window, its layers one after the other; a host ring filled in (layer, block, head) order
holds only a block's heads side by side, so the list breaks into runs of `heads` slots.
kv_promote fetches such lists with its gather kernel (through the device's view of the
pinned ring) instead of one DMA transfer per run.  Both ways must leave exactly the
oracle's state and bytes."""
import numpy as np
import pytest

from paper_2604_26968_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_position_ordered_lists_are_runs_of_one_blocks_heads():
    w = W.config(3, scale=1 / 64)
    p = w.parts[0]
    live = np.ones(p.ring_slots, np.uint8)
    lst = w.promote_list(2, 0, w.m, 777, live, just_written=w.k).astype(np.int64)
    assert lst.size == w.m and np.unique(lst).size == lst.size
    runs = np.flatnonzero(np.diff(lst) != 1).size + 1
    assert lst.size / runs == p.heads          # every run is one (block, layer): its KV heads


@pytest.mark.parametrize("threshold,deferred,pieces", [(None, False, 1), (None, True, 2), (0, True, 1)])
def test_long_context_pool_with_position_ordered_promotion(threshold, deferred, pieces):
    from lockstep import Lockstep
    w = W.config(3, scale=1 / 192)
    ls = Lockstep(w, payload=True, batch_bytes=1 << 20, deferred=deferred, split_promote=pieces, fused=True)
    if threshold is not None:
        assert ls.gpu.pool.kv_set_gather_threshold(threshold) == 0
    for e in range(5):
        r = ls.epoch(e)
        assert r["promoted"] > 0
    gathered = ls.gpu.pool.kv_get_stats()["gathered"]
    assert (gathered == 0) if threshold == 0 else (gathered > 0)
    ls.close()


def test_gather_kernel_on_large_single_chunk_entries_and_four_partitions():
    from lockstep import Lockstep
    w = W.config(5, scale=1 / 128)              # MLA entries of 18 KB next to 8 KB K/V entries
    for p in w.parts:
        p.ring_slots = w.k + 64
    ls = Lockstep(w, payload=True, batch_bytes=1 << 20, deferred=True, counted=True)
    assert ls.gpu.pool.kv_set_gather_threshold(1 << 40) == 0     # every list goes through the gather kernel
    for e in range(4):
        ls.epoch(e)
    st = ls.gpu.pool.kv_get_stats()
    assert st["gathered"] == st["promoted"] > 0
    ls.close()
