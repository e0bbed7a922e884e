"""Pins for the oracle's head-granular importance weighting (head-granular
eviction section: a [layer][head] importance matrix kept as an EMA, the group
maximum as a GQA KV head's score, a [layer][1] matrix for MLA, per-head
multipliers at task transitions).  The paper prints no formula for it, so the
tests pin what the section states in words and the arithmetic of the reading:
    M <- d*M + (1-d)*x;  W[l][h] = max over the group of M[l][.] * mult[l][h];
    score = policy score * W[layer][head].
"""
import numpy as np
import pytest

from oracle import kv_oracle as O


def _pool(variant=O.GQA, layers=3, hq=8, hkv=2, blocks=16, parts=None, **mk):
    if parts is None:
        m = O.model(variant=variant, n_layers=layers, n_q_heads=hq, n_kv_heads=hkv, head_dim=8, **mk)
        parts = [dict(model=m, block_tokens=4, blocks_per_layer=blocks, ring_slots=64)]
    p = O.OraclePool(parts, n_tags=1 << 14, payload=False)
    r = np.random.default_rng(0)
    p.admit(0, 0.5, r.integers(0, 16, p.N, dtype=np.uint8), None)
    return p


def _run_epoch(p, epoch, seed):
    r = np.random.default_rng(seed)
    ev = r.integers(0, p.N, p.N).astype(np.uint32)
    assert p.epoch_score(epoch, ev, (r.random(ev.size) < 0.5).astype(np.uint8)) == O.OK


def test_untouched_pool_is_unweighted_and_unit_matrix_is_the_identity():
    a, b = _pool(), _pool()
    x = np.ones(3 * 8, np.float32)          # M stays 1 whatever the decay: d*1 + (1-d)*1
    assert b.head_importance_update(0, x, 0.25) == O.OK
    assert np.array_equal(b.head_array(0, "weights"), np.ones(3 * 2, np.float32))
    for e in range(1, 4):
        _run_epoch(a, e, e)
        _run_epoch(b, e, e)
        assert np.array_equal(a.score.view(np.uint32), b.score.view(np.uint32))
    assert np.array_equal(a.head_array(0, "importance"), np.ones(24, np.float32))


def test_matrix_recurrence_closed_forms():
    p = _pool()
    d = np.float32(0.9)
    x = np.full(24, 3.0, np.float32)
    m = np.float64(1.0)
    for t in range(1, 30):
        assert p.head_importance_update(0, x, float(d)) == O.OK
        m = float(d) * m + (1.0 - float(d)) * 3.0        # = 3 - 2 d^t in exact arithmetic
        got = p.head_array(0, "importance")
        assert np.all(got == got[0])
        assert abs(float(got[0]) - (3.0 - 2.0 * float(d) ** t)) < 1e-5
    q = _pool()
    assert q.head_importance_update(0, np.arange(24, dtype=np.float32), 0.0) == O.OK     # d = 0: M = x
    assert np.array_equal(q.head_array(0, "importance"), np.arange(24, dtype=np.float32))
    assert q.head_importance_update(0, np.zeros(24, np.float32), 1.0) == O.OK            # d = 1: unchanged
    assert np.array_equal(q.head_array(0, "importance"), np.arange(24, dtype=np.float32))


@pytest.mark.parametrize("variant,hq,hkv", [(O.GQA, 8, 2), (O.GQA, 12, 4), (O.MHA, 4, 4), (O.MQA, 6, 1)])
def test_kv_head_weight_is_the_group_maximum_times_the_multiplier(variant, hq, hkv):
    p = _pool(variant=variant, hq=hq, hkv=hkv, layers=3)
    r = np.random.default_rng(5)
    x = r.random((3, hq)).astype(np.float32) * 4
    assert p.head_importance_update(0, x, 0.0) == O.OK
    g = hq // hkv
    brute = x.reshape(3, hkv, g).max(axis=2)        # contiguous groups of g query heads per KV head
    assert np.array_equal(p.head_array(0, "weights").reshape(3, hkv), brute)
    mult = r.choice(np.array([0.5, 1.0, 2.0], np.float32), size=(3, hkv))
    assert p.set_head_multipliers(0, mult) == O.OK
    assert np.array_equal(p.head_array(0, "weights").reshape(3, hkv), brute * mult)
    assert p.set_head_multipliers(0, None) == O.OK
    assert np.array_equal(p.head_array(0, "weights").reshape(3, hkv), brute)


def test_mla_matrix_is_layer_by_one():
    m = O.model(n_layers=4, n_q_heads=16, d_latent=32, d_rope=8)
    p = _pool(parts=[dict(model=m, block_tokens=4, blocks_per_layer=8, ring_slots=16)])
    x = np.array([0.5, 1.0, 2.0, 4.0], np.float32)
    assert p.head_importance_update(0, x, 0.0) == O.OK
    assert np.array_equal(p.head_array(0, "weights"), x)
    _run_epoch(p, 1, 1)
    w = np.repeat(x, 8)                              # entries of layer l: 8 blocks x 1 head
    assert np.array_equal(p.score, (p.estimate[p.pair] * p.ema) * w)


@pytest.mark.parametrize("policy", [0, 1, 2])
def test_score_is_the_policy_score_times_the_weight_of_layer_and_head(policy):
    p, ref = _pool(), _pool()
    assert p.set_policy(policy) == O.OK and ref.set_policy(policy) == O.OK
    r = np.random.default_rng(9)
    x = (r.random(24) * 3).astype(np.float32)
    assert p.head_importance_update(0, x, 0.5) == O.OK
    for e in range(1, 4):
        _run_epoch(p, e, e)
        _run_epoch(ref, e, e)
    w = p.head_array(0, "weights").reshape(3, 2)
    ids = np.arange(p.N)
    layer, head = ids // (16 * 2), ids % 2          # id = (layer*NB + block)*H + head
    if policy == 2:      # recency only: the matrix plays no part
        assert np.array_equal(p.score, ref.score)
    else:                # one more binary32 multiply; the product of two floats is exact in double
        want = (ref.score.astype(np.float64) * w[layer, head].astype(np.float64)).astype(np.float32)
        assert np.array_equal(p.score.view(np.uint32), want.view(np.uint32))
        assert not np.array_equal(p.score, ref.score)


def test_low_weight_heads_are_evicted_first():
    """Bias stated by the section: entries of a head with a small weight go before equally
    used entries of other heads."""
    p = _pool(layers=1, hq=4, hkv=2, blocks=32)
    ev = np.arange(p.N, dtype=np.uint32)             # every entry touched once, all hits
    assert p.head_importance_update(0, np.array([1, 1, 0.25, 0.125], np.float32), 0.0) == O.OK
    assert p.set_policy(1) == O.OK                   # EMA only: isolates the weight
    assert p.epoch_score(1, ev, np.ones(ev.size, np.uint8)) == O.OK
    rc, v = p.select_victims(32)
    assert rc == O.OK and np.all(v % 2 == 1)         # all 32 victims are entries of KV head 1 (weight 0.25)


def test_partitions_have_their_own_matrices():
    parts = [dict(model=O.model(variant=O.MHA, n_layers=2, n_q_heads=2, n_kv_heads=2, head_dim=8),
                  block_tokens=4, blocks_per_layer=4, ring_slots=8),
             dict(model=O.model(variant=O.GQA, n_layers=1, n_q_heads=4, n_kv_heads=2, head_dim=8),
                  block_tokens=4, blocks_per_layer=4, ring_slots=8)]
    p, ref = _pool(parts=parts), _pool(parts=parts)
    assert p.head_importance_update(1, np.array([2, 1, 1, 4], np.float32), 0.0) == O.OK
    _run_epoch(p, 1, 3)
    _run_epoch(ref, 1, 3)
    n0 = 2 * 4 * 2
    assert np.array_equal(p.score[:n0], ref.score[:n0])                       # partition 0 untouched
    w1 = np.tile(np.array([2, 4], np.float32), 4)
    assert np.array_equal(p.score[n0:], ref.score[n0:] * w1)


def test_bad_arguments_change_nothing():
    p = _pool()
    before = p.head_array(0, "importance").copy()
    bad = np.ones(24, np.float32)
    for v in (-1.0, np.nan, np.inf):
        bad[5] = v
        assert p.head_importance_update(0, bad, 0.5) == O.ERR_INVALID_ARG
    assert p.head_importance_update(0, np.ones(24, np.float32), 1.5) == O.ERR_INVALID_ARG
    assert p.head_importance_update(1, np.ones(24, np.float32), 0.5) == O.ERR_INVALID_ARG
    m = np.ones(6, np.float32)
    m[0] = -2
    assert p.set_head_multipliers(0, m) == O.ERR_INVALID_ARG
    assert np.array_equal(p.head_array(0, "importance"), before)
    assert np.array_equal(p.head_array(0, "weights"), np.ones(6, np.float32))
