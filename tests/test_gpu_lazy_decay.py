"""Lazy decay of promoted entries (kv_set_lazy_decay) against the oracle: whole
epochs in lock step on pools whose promote lists reach back several epochs, and
a directed case with a known number of missed scoring passes."""
import numpy as np
import pytest

from oracle import kv_oracle as O
from paper_2604_26968_b200 import binding as B
from paper_2604_26968_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg,scale,epochs,fused", [
    (1, 1.0, 20, False),
    (2, 1 / 64, 8, True),      # promote lists start at seeded older slots: several passes missed
    (2, 1 / 64, 6, False),
    (4, 1 / 128, 6, True),     # MLA
    (5, 1 / 128, 6, True),     # four partitions
])
def test_lazy_decay_epochs_match_the_oracle(cfg, scale, epochs, fused):
    from lockstep import Lockstep
    w = W.config(cfg, scale=scale)
    ls = Lockstep(w, payload=False, batch_bytes=512 << 10, fused=fused, lazy=True)
    missed = 0
    for e in range(epochs):
        before = [ls.ora.part_array(q, "r_depoch").copy() for q in range(len(w.parts))]
        live = [ls.ora.part_array(q, "r_live").copy() for q in range(len(w.parts))]
        ls.epoch(e)
        for q in range(len(w.parts)):   # slots that were live before the epoch and are dead now were promoted
            gone = (live[q] != 0) & (ls.ora.part_array(q, "r_live") == 0)
            missed += int((e - before[q][gone].astype(np.int64)).clip(min=0).sum())
    ls.close()
    if cfg != 1:
        assert missed > 0, "no promotion reached back past its own epoch: the catch-up was not exercised"


@pytest.mark.parametrize("gap", [0, 1, 5, 300])
def test_directed_gap(gap):
    """Demote a few warmed entries, run `gap` scoring passes without them, promote:
    the EMA must equal the oracle's (which equals a resident untouched twin's)."""
    from lockstep import Lockstep
    w = W.Workload("gap", [W.gqa(2, 8, 4, 16, 8, 64, 256, "entry")], 0.05, 0.05, seed=5, promote_style="recent")
    ls = Lockstep(w, payload=True, batch_bytes=64 << 10, lazy=True)
    g, o = ls.gpu, ls.ora
    for e in range(3):
        ls.epoch(e)
    e = 3
    ev_entry, ev_hit = w.events(e, o.pair, ls.fresh)
    d_e, d_h, n = g.stage_events(ev_entry, ev_hit)
    assert o.epoch_score(e, ev_entry, ev_hit) == O.OK
    g.check(g.pool.kv_epoch_score(e, d_e, d_h, n), "kv_epoch_score")
    rc, v = o.select_victims(12)
    g.check(g.pool.kv_select_victims(12, g.victims), "kv_select_victims")
    assert o.demote(v) == O.OK
    g.check(g.pool.kv_demote(g.victims, 12, g.batch_bytes), "kv_demote")
    ls.compare_ring("demote")
    cur = o.info(0)["cursor"]
    slots = np.array([(cur - 12 + j) % w.parts[0].ring_slots for j in range(12)], np.uint64)
    none_e, none_h = np.zeros(0, np.uint32), np.zeros(0, np.uint8)
    d0_e, d0_h, _ = g.stage_events(none_e, none_h)
    for s in range(gap):
        assert o.epoch_score(e + 1 + s, none_e, none_h) == O.OK
        g.check(g.pool.kv_epoch_score(e + 1 + s, d0_e, d0_h, 0), "kv_epoch_score")
    before = o.part_array(0, "r_ema")[slots.astype(np.int64)].copy()
    assert o.promote(0, slots) == O.OK
    g.check(g.pool.kv_promote(0, slots, g.batch_bytes), "kv_promote")
    ls.compare_state("promote after %d passes" % gap, scores=False)
    ls.compare_payload("promote after %d passes" % gap)
    got = g.host_array("ema")[v.astype(np.int64)]        # j-th listed slot -> j-th lowest FREE id = v[j]
    want = before.astype(np.float64) * float(np.float32(w.decay)) ** gap
    assert np.allclose(got, want, rtol=1e-4, atol=1e-30)
    ls.close()
