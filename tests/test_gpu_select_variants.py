"""The selection as one launch per phase (kv_set_select_variant(pool, 0)).

That form runs where a device cannot co-schedule the persistent kernel or a pool has more
entries per SM than its bitmaps hold, and under the entry point with built-in scratch; it
must give the oracle's victims like the default form: heavy ties, pools whose size is not
a multiple of any tile, k = every resident entry, several partitions."""
import numpy as np
import pytest

from paper_2604_26968_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg,scale,epochs", [(1, 1.0, 12), (2, 1 / 64, 5), (5, 1 / 128, 5)])
def test_phase_by_phase_selection_matches_the_oracle(cfg, scale, epochs):
    from lockstep import Lockstep
    w = W.config(cfg, scale=scale)
    if cfg == 5:
        for p in w.parts:
            p.ring_slots = w.k + 64
    ls = Lockstep(w, payload=False, batch_bytes=1 << 20, select_variant=0)
    for e in range(epochs):
        ls.epoch(e)
    ls.close()


@pytest.mark.parametrize("variant", [0, 1])
def test_ties_ragged_sizes_and_k_equal_to_the_resident_count(variant):
    from lockstep import Lockstep
    # 3 x 347 x 3 = 3,123 entries: no multiple of a vector, a tile or a chunk; epoch 0 scores are
    # all equal (every EMA is the same one touch or none), so every k cuts through a tie
    w = W.Workload("ragged", [W.gqa(3, 6, 3, 16, 8, 347, 4096, "entry")], 0.1, 0.05, seed=21,
                   promote_style="recent")
    ls = Lockstep(w, payload=False, batch_bytes=1 << 18, select_variant=variant)
    N = w.N
    for e, k in enumerate([1, 2, N // 3, N - 1, N, 0, 17, N // 2]):
        ls.epoch(e, k=k)
    ls.close()
