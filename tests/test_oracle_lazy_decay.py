"""Pins for the oracle's lazy decay of promoted entries.

The paper does not say what happens to a block's importance while the block
sits in a lower tier; the reading taken is that promotion first applies the EMA
steps the block missed, one per scoring pass, each the untouched step
ema <- decay*ema.  What can be pinned is that reading's own claim: a promoted
block ends with exactly the EMA of a twin that stayed resident and untouched,
and that value is decay^missed * ema within binary32 rounding.
"""
import numpy as np
import pytest

from oracle import kv_oracle as O


def _pool(decay, lazy, blocks=16):
    part = dict(model=O.model(variant=O.GQA, n_layers=1, n_q_heads=4, n_kv_heads=2, head_dim=8),
                block_tokens=4, blocks_per_layer=blocks, ring_slots=64)
    p = O.OraclePool([part], n_tags=4096, payload=False)
    p.admit(0, decay, np.zeros(p.N, np.uint8), None)
    assert p.set_lazy_decay(lazy) == O.OK
    return p


def _warm(p, epochs=3):
    """Entries 0 and 1 receive identical touches, so they carry identical EMAs."""
    for e in range(1, epochs + 1):
        ev = np.array([0, 1, 0, 1, 0, 1], np.uint32)
        assert p.epoch_score(e, ev, np.ones(ev.size, np.uint8)) == O.OK
    assert p.ema[0] == p.ema[1] and p.ema[0] > 0
    return epochs


@pytest.mark.parametrize("decay", [0.1, 0.3, 0.5, 0.7, 0.9])
@pytest.mark.parametrize("missed", [0, 1, 2, 7, 40])
def test_promoted_entry_equals_untouched_resident_twin(decay, missed):
    p = _pool(decay, True)
    e = _warm(p)
    s0 = float(p.ema[0])
    assert p.demote(np.array([0], np.uint32)) == O.OK        # demoted in epoch e; twin 1 stays
    none = np.zeros(0, np.uint32), np.zeros(0, np.uint8)
    for _ in range(missed):
        e += 1
        assert p.epoch_score(e, *none) == O.OK
    slot = int(p.loc[0] & 0x7FFFFFFF)
    assert p.promote(0, np.array([slot], np.uint64)) == O.OK
    f = int(p.loc[0])
    assert f == 0 and p.state[0] == O.RESIDENT
    assert p.ema[f].tobytes() == p.ema[1].tobytes()          # bit for bit the twin's value
    want = (float(np.float32(decay)) ** missed) * s0         # closed form in binary64
    assert p.ema[f] == pytest.approx(want, rel=1e-5, abs=1e-30)
    assert p.decay[f] == np.float32(decay)


def test_off_restores_verbatim_and_same_epoch_round_trip_is_identity():
    for lazy in (False, True):
        p = _pool(0.9, lazy)
        e = _warm(p)
        s0 = p.ema[0].tobytes()
        assert p.demote(np.array([0], np.uint32)) == O.OK
        if not lazy:
            for _ in range(5):
                e += 1
                p.epoch_score(e, np.zeros(0, np.uint32), np.zeros(0, np.uint8))
        slot = int(p.loc[0] & 0x7FFFFFFF)
        assert p.promote(0, np.array([slot], np.uint64)) == O.OK
        assert p.ema[int(p.loc[0])].tobytes() == s0           # off: verbatim; on with 0 missed passes: verbatim


def test_decay_one_keeps_and_decay_zero_clears():
    for decay, keep in ((1.0, True), (0.0, False)):
        p = _pool(decay, True)
        p.ema[0] = np.float32(2.5)                            # set directly: with these decays touches cannot build it
        p.epoch_score(1, np.zeros(0, np.uint32), np.zeros(0, np.uint8))
        s0 = float(p.ema[0])
        assert p.demote(np.array([0], np.uint32)) == O.OK
        for e in (2, 3, 4):
            p.epoch_score(e, np.zeros(0, np.uint32), np.zeros(0, np.uint8))
        slot = int(p.loc[0] & 0x7FFFFFFF)
        assert p.promote(0, np.array([slot], np.uint64)) == O.OK
        assert float(p.ema[int(p.loc[0])]) == (s0 if keep else 0.0)


def test_demotion_epoch_is_recorded_per_slot():
    p = _pool(0.5, True)
    _warm(p, epochs=4)
    assert p.demote(np.array([2, 3], np.uint32)) == O.OK
    p.epoch_score(5, np.zeros(0, np.uint32), np.zeros(0, np.uint8))
    assert p.demote(np.array([4], np.uint32)) == O.OK
    dep = p.part_array(0, "r_depoch")
    assert dep[:3].tolist() == [4, 4, 5]
