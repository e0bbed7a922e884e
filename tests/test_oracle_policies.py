"""Pins for the oracle's policy variants and its confidence-weighted blend.

LRU and EMA-only are the two policies the paper compares the Bayesian one with
(its table of cache hit rates); the blend follows the paragraph on confidence
scores in the Bayesian reuse section, whose formula the paper withholds: the
tests pin the properties that paragraph states and the arithmetic of the
reading taken (c = n/(n+kappa); estimate = c*P + (1-c)*f_window).
"""
from fractions import Fraction

import numpy as np
import pytest

from oracle import kv_oracle as O


def _pool(blocks=32, **kw):
    part = dict(model=O.model(variant=O.GQA, n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=8),
                block_tokens=4, blocks_per_layer=blocks, ring_slots=64)
    p = O.OraclePool([part], n_tags=4096, payload=False, **kw)
    r = np.random.default_rng(0)
    p.admit(0, 0.5, r.integers(0, 16, p.N, dtype=np.uint8), None)
    return p


def test_lru_evicts_least_recently_touched_then_lowest_id():
    p = _pool()
    assert p.set_policy(2) == O.OK
    r = np.random.default_rng(1)
    for epoch in range(1, 9):
        ev = r.choice(p.N, size=p.N // 3, replace=False).astype(np.uint32)
        assert p.epoch_score(epoch, ev, np.ones(ev.size, np.uint8)) == O.OK
    assert np.array_equal(p.score, p.last_epoch.astype(np.float32))
    rc, v = p.select_victims(20)
    brute = sorted(sorted(range(p.N), key=lambda i: (int(p.last_epoch[i]), i))[:20])
    assert rc == O.OK and v.tolist() == brute


def test_ema_only_ignores_the_posterior():
    p = _pool()
    assert p.set_policy(1) == O.OK
    r = np.random.default_rng(2)
    for epoch in range(1, 5):
        ev = r.integers(0, p.N, 200).astype(np.uint32)
        p.epoch_score(epoch, ev, (r.random(200) < 0.3).astype(np.uint8))
    assert np.array_equal(p.score, p.ema)
    assert len(set(np.round(p.P, 6))) > 4           # the posteriors did move; the score ignores them
    assert p.set_policy(3) == O.ERR_INVALID_ARG


def test_blend_off_is_the_plain_posterior_and_bad_arguments_are_refused():
    p = _pool()
    p.epoch_score(1, np.arange(50, dtype=np.uint32), np.ones(50, np.uint8))
    assert np.array_equal(p.estimate, p.P)
    assert p.set_confidence_blend(0.0, 4) == O.ERR_INVALID_ARG
    assert p.set_confidence_blend(8.0, 65) == O.ERR_INVALID_ARG
    assert p.set_confidence_blend(8.0, 0) == O.OK


def test_blend_exact_rational_values_and_limits():
    kappa, W = 10.0, 3
    p = _pool()
    p.pair[:] = 0
    assert p.set_confidence_blend(kappa, W) == O.OK
    # epochs of (hits, misses) on pair 0; pair 5 is never observed
    seq = [(3, 1), (0, 4), (2, 2), (10, 0), (0, 0), (1, 7)]
    H = M = 0
    for e, (h, m) in enumerate(seq, start=1):
        ev = np.zeros(h + m, np.uint32)
        hit = np.array([1] * h + [0] * m, np.uint8)
        assert p.epoch_score(e, ev, hit) == O.OK
        H, M = H + h, M + m
        wh = sum(x for x, _ in seq[max(0, e - W):e])
        wm = sum(y for _, y in seq[max(0, e - W):e])
        P = Fraction(1 + H, 2 + H + M)
        c = Fraction(H + M) / (Fraction(H + M) + Fraction(int(kappa)))
        f = Fraction(wh, wh + wm) if wh + wm else P
        exact = c * P + (1 - c) * f
        assert abs(float(p.estimate[0]) - float(exact)) <= 4e-7, (e, float(exact))
        # an unobserved pair has confidence 0 and an empty window: estimate = prior mean
        assert p.estimate[5] == np.float32(0.5)
    # confidence saturates toward 1: after many observations the estimate is the posterior
    ev = np.zeros(200000, np.uint32)
    p.epoch_score(99, ev, np.ones(ev.size, np.uint8))
    assert abs(float(p.estimate[0]) - float(p.P[0])) < 1e-4


def test_blend_reacts_to_a_shift_faster_than_the_posterior():
    # 400 epochs of hits establish a high posterior; then the pair turns to misses.  A young-confidence
    # setting (large kappa) follows the recent window, the plain posterior lags: the adaptation the
    # paragraph on distribution shifts describes.
    p = _pool()
    p.pair[:] = 3
    p.set_confidence_blend(2000.0, 4)
    for e in range(1, 41):
        p.epoch_score(e, np.zeros(10, np.uint32), np.ones(10, np.uint8))
    for e in range(41, 45):
        p.epoch_score(e, np.zeros(10, np.uint32), np.zeros(10, np.uint8))
    assert p.P[3] > 0.85 and p.estimate[3] < 0.3
    assert np.array_equal(p.score[:8], (p.estimate[p.pair[:8]] * p.ema[:8]).astype(np.float32))


def test_block_level_selection_equals_brute_force_with_architecture_weights():
    # three partitions: MHA (w = 1, 3 heads), GQA (w = 4, 2 heads), MLA (w = 16, 1 entry per block)
    parts = [dict(model=O.model(variant=O.MHA, n_layers=2, n_q_heads=3, n_kv_heads=3, head_dim=8),
                  block_tokens=4, blocks_per_layer=7, ring_slots=64),
             dict(model=O.model(variant=O.GQA, n_layers=1, n_q_heads=8, n_kv_heads=2, head_dim=8),
                  block_tokens=4, blocks_per_layer=9, ring_slots=64),
             dict(model=O.model(n_layers=2, n_q_heads=16, n_kv_heads=16, head_dim=8, d_latent=12, d_rope=4),
                  block_tokens=4, blocks_per_layer=5, ring_slots=64)]
    p = O.OraclePool(parts, n_tags=4096, payload=False)
    r = np.random.default_rng(4)
    p.admit(0, 0.5, r.integers(0, 16, p.N, dtype=np.uint8), None)
    for epoch in range(1, 4):
        ev = r.integers(0, p.N, 60).astype(np.uint32)
        p.epoch_score(epoch, ev, np.ones(60, np.uint8))
    assert p.demote(np.array([4, 44], np.uint32)) == O.OK      # two blocks lose a head: no longer candidates
    p.epoch_score(4, [], [])
    H = [3, 2, 1]
    w = [np.float32(1), np.float32(4), np.float32(16)]
    blocks = []
    for q in range(3):
        inf = p.info(q)
        for lb in range(inf["n"] // H[q]):
            first = inf["base"] + lb * H[q]
            if not all(p.state[first + h] == O.RESIDENT for h in range(H[q])):
                continue
            s = np.float32(0)
            for h in range(H[q]):
                s = np.float32(s + p.score[first + h])
            blocks.append((float(np.float32(w[q] * s)), first, H[q]))
    order = sorted(range(len(blocks)), key=lambda j: (blocks[j][0], blocks[j][1]))
    for k in (0, 1, 5, len(blocks) // 2, len(blocks)):
        rc, v = p.select_victim_blocks(k)
        expect = sorted(i for j in order[:k] for i in range(blocks[j][1], blocks[j][1] + blocks[j][2]))
        assert rc == O.OK and v.tolist() == expect, k
    rc, _ = p.select_victim_blocks(len(blocks) + 1)
    assert rc == O.ERR_K_TOO_LARGE
    assert len(blocks) == 2 * 7 + 9 + 2 * 5 - 2
    # all-zero scores: aggregates tie, lowest (partition, layer, block) first, whole blocks come out
    q = O.OraclePool(parts, n_tags=4096, payload=False)
    q.admit(0, 0.5, np.zeros(q.N, np.uint8), None)
    q.epoch_score(1, [], [])
    rc, v = q.select_victim_blocks(3)
    assert rc == O.OK and v.tolist() == list(range(9))
