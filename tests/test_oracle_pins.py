"""Pins the CPU oracle to what the paper prints and to what mathematics fixes.

Each test is chosen so that a plausible slip in the oracle (a dropped factor, a
swapped operand, an off-by-one in an index or a tie rule) makes it fail.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import kv_oracle as O
from paper_2604_26968_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows():
    rows = []
    with open(os.path.join(GOLDEN, "sizing.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, fields, _what, expected, _cite = [c.strip() for c in line.split("|")]
            rows.append((key, [int(x) for x in fields.split()], int(expected)))
    return rows


@pytest.mark.parametrize("key,fields,expected", _rows())
def test_sizing_matches_values_printed_in_the_paper(key, fields, expected):
    m = O.Model(*fields)
    if key == "per_token_layer":
        got = O.size_bytes(m, 1, per_layer=True)
    elif key == "sequence_total":
        got = O.size_bytes(m, 128000, per_layer=False)
    elif key == "max_batch_mha":
        got = O.max_batch(m, 8 * 30 * 10**9, 4096)
    elif key == "max_batch_arch":
        got = O.max_batch(m, 30 * 10**9, 4096)
    elif key == "ckpt_1000_tokens":
        got = O.size_bytes(m, 1000, per_layer=False)
    else:
        raise AssertionError(key)
    assert got == expected


def test_sizing_mla_bytes_per_token_closed_form():
    # (d_latent + d_rope) x layers x dtype bytes
    m = O.model(n_layers=61, n_q_heads=128, n_kv_heads=128, head_dim=128, d_latent=512, d_rope=64)
    assert O.size_bytes(m, 1, per_layer=False) == (512 + 64) * 61 * 2 == 70272


def test_sizing_variant_inference_and_precision():
    assert O.infer_variant(O.model(n_q_heads=32, n_kv_heads=32, head_dim=128)) == O.MHA
    assert O.infer_variant(O.model(n_q_heads=32, n_kv_heads=1, head_dim=128)) == O.MQA
    assert O.infer_variant(O.model(n_q_heads=32, n_kv_heads=8, head_dim=128)) == O.GQA
    assert O.infer_variant(O.model(n_q_heads=32, n_kv_heads=8, head_dim=128, d_latent=512,
                                   d_rope=64)) == O.MLA
    assert O.infer_variant(O.model(n_q_heads=8, n_kv_heads=32, head_dim=128)) == O.ERR_UNSUPPORTED_VARIANT
    # INT4 (p = 0.5) is half of INT8, a quarter of BF16
    g = dict(n_q_heads=64, n_kv_heads=8, head_dim=128)
    b16 = O.size_bytes(O.model(dtype_bits=16, **g), 100)
    b8 = O.size_bytes(O.model(dtype_bits=8, **g), 100)
    b4 = O.size_bytes(O.model(dtype_bits=4, **g), 100)
    assert (b16, b8, b4) == (409600, 204800, 102400)
    # sizes that are not whole bytes, and inconsistent fields, are errors
    assert O.size_bytes(O.model(variant=O.MLA, d_latent=3, d_rope=0, dtype_bits=4), 1) == O.ERR_INVALID_ARG
    assert O.size_bytes(O.model(variant=O.MLA, n_q_heads=8, n_kv_heads=8, head_dim=64), 1) == O.ERR_INVALID_ARG
    assert O.size_bytes(O.model(variant=O.MQA, n_q_heads=8, n_kv_heads=2, head_dim=64), 1) == O.ERR_INVALID_ARG
    # linear in n; MQA equals GQA with one KV head
    assert O.size_bytes(O.model(variant=O.MQA, n_q_heads=8, n_kv_heads=1, head_dim=64), 7) == \
        O.size_bytes(O.model(variant=O.GQA, n_q_heads=8, n_kv_heads=1, head_dim=64), 7) == 7 * 2 * 64 * 2


def _tiny_pool(layers=2, heads=4, blocks=8, ring=16, payload=True, n_tags=4096, **kw):
    part = dict(model=O.model(variant=O.GQA, n_layers=layers, n_q_heads=4 * heads, n_kv_heads=heads,
                              head_dim=8),
                block_tokens=4, blocks_per_layer=blocks, ring_slots=ring)
    return O.OraclePool([part], n_tags=n_tags, payload=payload, **kw)


def _fill(pool, epoch=0, decay=0.9, seed=0, pairs=None):
    n_free = int((pool.state == O.FREE).sum())
    r = np.random.default_rng(seed)
    if pairs is None:
        pairs = r.integers(0, 16, n_free, dtype=np.uint8)
    first = pool.next_tag
    payload = None
    if pool.payload:
        # partitions admit in id order; build the images partition by partition
        imgs = []
        t = first
        for q in range(pool.n_parts):
            inf = pool.info(q)
            nf = int((pool.state[inf["base"]:inf["base"] + inf["n"]] == O.FREE).sum())
            imgs.append(W.pattern_bytes(np.arange(t, t + nf), inf["entry_bytes"]).reshape(-1))
            t += nf
        payload = np.concatenate(imgs) if imgs else None
    got = pool.admit(epoch, decay, pairs, payload)
    assert got == n_free
    return pairs


def test_posterior_hand_sequences_rule_of_succession():
    # prior Beta(1,1): no events -> 1/2; H,H,M -> 3/5; 500 hits -> 501/502 (> 0.97)
    pool = _tiny_pool()
    _fill(pool, pairs=np.full(pool.N, 3, np.uint8))
    pool.pair[5] = 7
    pool.pair[6] = 9
    assert pool.epoch_score(0, [], []) == O.OK
    assert np.all(pool.P == np.float32(0.5))
    ev = np.array([5, 5, 5], np.uint32)
    assert pool.epoch_score(1, ev, [1, 1, 0]) == O.OK
    assert pool.P[7] == np.float32(3.0) / np.float32(5.0)
    assert abs(float(pool.P[7]) - 0.6) < 1e-7
    assert pool.P[3] == np.float32(0.5) and pool.P[9] == np.float32(0.5)
    assert pool.epoch_score(2, np.full(500, 6, np.uint32), np.ones(500, np.uint8)) == O.OK
    assert abs(float(pool.P[9]) - 501.0 / 502.0) < 1e-7 and pool.P[9] > 0.97
    assert pool.hits[9] == 500 and pool.misses[9] == 0 and pool.hits[7] == 2 and pool.misses[7] == 1
    # a miss raises beta, not alpha: all-miss sequence tends to 0
    pool.pair[0] = 1
    assert pool.epoch_score(3, np.zeros(9, np.uint32), np.zeros(9, np.uint8)) == O.OK
    assert abs(float(pool.P[1]) - 1.0 / 11.0) < 1e-8


def test_posterior_counters_equal_histogram_of_events_and_priors_shift():
    r = np.random.default_rng(5)
    pool = _tiny_pool(alpha0=2.0, beta0=0.5)
    _fill(pool, seed=1)
    tot_h = np.zeros(16, np.int64)
    tot_m = np.zeros(16, np.int64)
    for epoch in range(4):
        ev = r.integers(0, pool.N, 300).astype(np.uint32)
        hit = r.integers(0, 2, 300).astype(np.uint8)
        pr = pool.pair[ev]
        tot_h += np.bincount(pr[hit == 1], minlength=16)
        tot_m += np.bincount(pr[hit == 0], minlength=16)
        assert pool.epoch_score(epoch, ev, hit) == O.OK
        assert np.array_equal(pool.hits.astype(np.int64), tot_h)
        assert np.array_equal(pool.misses.astype(np.int64), tot_m)
    for p in range(16):
        exact = Fraction(2 + int(tot_h[p])) / (Fraction(2 + int(tot_h[p])) + Fraction(1, 2) + int(tot_m[p]))
        assert abs(float(pool.P[p]) - float(exact)) <= 2e-7 * float(exact)


def test_posterior_priors_wash_out_within_100_observations():
    # three symmetric priors, same 100 Bernoulli(0.8) observations: estimates agree closely
    r = np.random.default_rng(11)
    obs = (r.random(100) < 0.8).astype(np.uint8)
    est = []
    for a0 in (0.5, 1.0, 2.0):
        pool = _tiny_pool(alpha0=a0, beta0=a0)
        _fill(pool, pairs=np.zeros(pool.N, np.uint8))
        pool.epoch_score(0, np.zeros(100, np.uint32), obs)
        est.append(float(pool.P[0]))
    assert max(est) - min(est) < 0.02
    assert abs(est[1] - (1 + obs.sum()) / 102.0) < 1e-6


@pytest.mark.parametrize("d", [0.1, 0.3, 0.5, 0.7, 0.9])
def test_ema_closed_forms(d):
    pool = _tiny_pool()
    _fill(pool, decay=d, pairs=np.zeros(pool.N, np.uint8))
    d32 = float(np.float32(d))
    # entry 0 touched once per epoch from 0: s_t = 1 - d^t ; entry 1 touched 3x per epoch: 3(1-d^t)
    # entry 2 never touched after one initial touch of 5: s_t = (1-d)*5*d^(t-1)
    for t in range(1, 41):
        ev = [0, 1, 1, 1] + ([2] * 5 if t == 1 else [])
        assert pool.epoch_score(t, np.array(ev, np.uint32), np.ones(len(ev), np.uint8)) == O.OK
        assert abs(float(pool.ema[0]) - (1 - d32 ** t)) <= 1e-6 * (1 - d32 ** t)
        assert abs(float(pool.ema[1]) - 3 * (1 - d32 ** t)) <= 1e-6 * 3 * (1 - d32 ** t)
        ref2 = (1 - d32) * 5 * d32 ** (t - 1)
        assert abs(float(pool.ema[2]) - ref2) <= 2e-6 * ref2
        assert pool.ema[3] == 0.0
        assert pool.last_epoch[0] == t and pool.last_epoch[2] == 1 and pool.last_epoch[3] == 0
        assert not pool.touch.any()


def test_ema_degenerate_decays_and_free_entries_untouched():
    pool = _tiny_pool()
    _fill(pool, pairs=np.zeros(pool.N, np.uint8))
    pool.decay[0] = 0.0     # no memory: s = x
    pool.decay[1] = 1.0     # frozen: s unchanged
    pool.ema[1] = 0.375
    pool.epoch_score(1, np.array([0, 0, 1], np.uint32), np.ones(3, np.uint8))
    assert pool.ema[0] == 2.0 and pool.ema[1] == np.float32(0.375)
    pool.epoch_score(2, np.array([1], np.uint32), np.ones(1, np.uint8))
    assert pool.ema[0] == 0.0 and pool.ema[1] == np.float32(0.375)
    # a demoted (FREE) slot keeps its arrays and is skipped by the update
    assert pool.demote(np.array([4], np.uint32)) == O.OK
    before = float(pool.ema[4])
    pool.ema[4] = 0.25
    pool.epoch_score(3, [], [])
    assert pool.ema[4] == np.float32(0.25) and np.isinf(pool.score[4]) and before == 0.0
    # events on a non-resident entry are an input error and change nothing
    h = pool.hits.copy()
    assert pool.epoch_score(4, np.array([4], np.uint32), np.ones(1, np.uint8)) == O.ERR_INVALID_ARG
    assert np.array_equal(h, pool.hits)


def test_score_is_one_correctly_rounded_product():
    r = np.random.default_rng(3)
    pool = _tiny_pool(blocks=64)
    _fill(pool, seed=2)
    for epoch in range(6):
        ev = r.integers(0, pool.N, 700).astype(np.uint32)
        pool.epoch_score(epoch, ev, (r.random(700) < 0.6).astype(np.uint8))
    # float x float is exact in double, so the binary32 result is that product rounded once
    expect = (pool.P[pool.pair].astype(np.float64) * pool.ema.astype(np.float64)).astype(np.float32)
    assert np.array_equal(expect, pool.score)
    assert (pool.score >= 0).all() and not np.signbit(pool.score).any()


def _brute_select(score, state, k):
    ids = [i for i in range(len(score)) if state[i] == O.RESIDENT]
    ids.sort(key=lambda i: (float(score[i]), i))
    return sorted(ids[:k])


def test_selection_equals_brute_force_for_every_k_with_heavy_ties():
    r = np.random.default_rng(9)
    pool = _tiny_pool(layers=1, heads=3, blocks=9, ring=64)
    _fill(pool, seed=4)
    ev = r.integers(0, pool.N, 20).astype(np.uint32)
    pool.epoch_score(0, ev, np.ones(20, np.uint8))      # most scores are exactly 0: ties
    pool.demote(np.array([2, 11], np.uint32))            # two FREE holes
    pool.epoch_score(1, [], [])
    n_res = int((pool.state == O.RESIDENT).sum())
    for k in range(n_res + 1):
        rc, v = pool.select_victims(k)
        assert rc == O.OK
        assert v.tolist() == _brute_select(pool.score, pool.state, k)
    rc, _ = pool.select_victims(n_res + 1)
    assert rc == O.ERR_K_TOO_LARGE


def test_selection_all_equal_scores_takes_lowest_ids_and_invariants_hold():
    pool = _tiny_pool(blocks=16)
    _fill(pool)
    pool.epoch_score(0, [], [])
    rc, v = pool.select_victims(10)
    assert rc == O.OK and v.tolist() == list(range(10))
    r = np.random.default_rng(2)
    for epoch in range(1, 5):
        ev = r.integers(0, pool.N, 60).astype(np.uint32)
        pool.epoch_score(epoch, ev, np.ones(60, np.uint8))
        k = 37
        rc, v = pool.select_victims(k)
        assert rc == O.OK and len(v) == k and np.all(np.diff(v.astype(np.int64)) > 0)
        chosen = np.zeros(pool.N, bool)
        chosen[v] = True
        key = lambda i: (float(pool.score[i]), i)
        worst_in = max(key(i) for i in v)
        best_out = min(key(i) for i in range(pool.N) if not chosen[i])
        assert worst_in < best_out


def _check_conservation(pool, issued):
    """Every issued tag is in exactly one of HBM / host / dropped and the maps invert."""
    loc = pool.loc
    in_hbm = {}
    for i in np.flatnonzero(pool.state == O.RESIDENT):
        t = int(pool.tag[i])
        assert t not in in_hbm
        in_hbm[t] = int(i)
        assert loc[t] == i
    on_host = {}
    for q in range(pool.n_parts):
        live = pool.part_array(q, "r_live")
        rt = pool.part_array(q, "r_tag")
        for s in np.flatnonzero(live):
            t = int(rt[s])
            assert t not in on_host and t not in in_hbm
            on_host[t] = (q, int(s))
            assert loc[t] == (O.HOST_BIT | int(s))
    for t in range(issued):
        if t not in in_hbm and t not in on_host:
            assert loc[t] == O.NONE
    assert np.all(pool.tag[pool.state == O.FREE] == O.NONE)
    return in_hbm, on_host


def _check_payload(pool, in_hbm, on_host):
    for q in range(pool.n_parts):
        inf = pool.info(q)
        slab = pool.part_array(q, "slab")
        ring = pool.part_array(q, "ring").reshape(inf["R"], inf["entry_bytes"])
        H, cb = inf["H"], inf["chunk_bytes"]
        for t, i in in_hbm.items():
            if not (inf["base"] <= i < inf["base"] + inf["n"]):
                continue
            local = i - inf["base"]
            img = W.pattern_bytes([t], inf["entry_bytes"])[0]
            lb, head = divmod(local, H)
            if inf["n_chunks"] == 1:
                got = slab[lb * cb:(lb + 1) * cb]
            else:
                ko = ((lb * 2 + 0) * H + head) * cb
                vo = ((lb * 2 + 1) * H + head) * cb
                got = np.concatenate([slab[ko:ko + cb], slab[vo:vo + cb]])
            assert np.array_equal(got, img), (t, i)
        for t, (qq, s) in on_host.items():
            if qq == q:
                assert np.array_equal(ring[s], W.pattern_bytes([t], inf["entry_bytes"])[0]), (t, s)


def test_demote_promote_round_trip_conservation_and_byte_identity():
    r = np.random.default_rng(21)
    pool = _tiny_pool(layers=2, heads=4, blocks=16, ring=40)
    _fill(pool)
    eb = pool.info(0)["entry_bytes"]
    for epoch in range(12):
        ev = r.integers(0, pool.N, 50).astype(np.uint32)
        assert pool.epoch_score(epoch, ev, (r.random(50) < 0.5).astype(np.uint8)) == O.OK
        rc, v = pool.select_victims(13)
        assert rc == O.OK
        meta = {int(pool.tag[i]): (int(pool.pair[i]), float(pool.ema[i]), float(pool.decay[i]),
                                   int(pool.last_epoch[i])) for i in v}
        cur = pool.info(0)["cursor"]
        assert pool.demote(v) == O.OK
        assert pool.info(0)["cursor"] == (cur + 13) % 40
        live = pool.part_array(0, "r_live")
        slots = np.flatnonzero(live)[::3][:5].astype(np.uint64)
        tags = pool.part_array(0, "r_tag")[slots.astype(np.int64)].copy()
        free_before = np.flatnonzero(pool.state == O.FREE)[:len(slots)]
        assert pool.promote(0, slots) == O.OK
        # j-th promoted goes to the j-th lowest free id, metadata restored verbatim
        assert np.array_equal(pool.tag[free_before], tags)
        for f, t in zip(free_before, tags):
            if int(t) in meta:
                assert (int(pool.pair[f]), float(pool.ema[f]), float(pool.decay[f]),
                        int(pool.last_epoch[f])) == meta[int(t)]
        in_hbm, on_host = _check_conservation(pool, pool.next_tag)
        _check_payload(pool, in_hbm, on_host)
        _fill(pool, epoch=epoch, seed=100 + epoch)
        assert not (pool.state == O.FREE).any()
    st = pool.stats()
    assert st["bytes_demoted"] == 12 * 13 * eb and st["bytes_promoted"] == 12 * 5 * eb
    assert st["bytes_dropped"] > 0 and st["bytes_dropped"] % eb == 0      # the 40-slot ring wrapped
    n_dropped = int((pool.loc[:pool.next_tag] == O.NONE).sum())
    assert st["bytes_dropped"] == n_dropped * eb


def test_demote_promote_error_paths_change_nothing():
    pool = _tiny_pool(blocks=8, ring=6)
    _fill(pool)
    pool.epoch_score(0, [], [])
    snap = pool.state.copy()
    assert pool.demote(np.arange(7, dtype=np.uint32)) == O.ERR_HOST_TIER_TOO_SMALL
    assert pool.demote(np.array([3, 2], np.uint32)) == O.ERR_INVALID_ARG
    assert np.array_equal(snap, pool.state)
    assert pool.demote(np.array([1, 2, 3], np.uint32)) == O.OK
    assert pool.promote(0, np.array([0, 0], np.uint64)) == O.ERR_BAD_HOST_SLOT     # duplicate
    assert pool.promote(0, np.array([4], np.uint64)) == O.ERR_BAD_HOST_SLOT        # dead slot
    assert pool.promote(0, np.array([9], np.uint64)) == O.ERR_BAD_HOST_SLOT        # out of range
    assert pool.promote(0, np.array([0, 1, 2], np.uint64)) == O.OK
    assert pool.promote(0, np.array([], np.uint64)) == O.OK
    assert (pool.state == O.RESIDENT).all()
    pool.demote(np.array([5], np.uint32))
    pool.promote(0, np.array([3], np.uint64))
    pool.demote(np.array([6], np.uint32))      # slot 4
    pool.admit(1, 0.9, np.zeros(1, np.uint8), W.pattern_bytes([pool.next_tag], pool.info(0)["entry_bytes"]))
    assert pool.promote(0, np.array([4], np.uint64)) == O.ERR_NO_FREE_SLOT


def test_mla_and_multi_partition_layout():
    parts = [dict(model=O.model(variant=O.MHA, n_layers=2, n_q_heads=3, n_kv_heads=3, head_dim=8),
                  block_tokens=4, blocks_per_layer=5, ring_slots=16),
             dict(model=O.model(n_layers=3, n_q_heads=16, n_kv_heads=16, head_dim=8, d_latent=12, d_rope=4),
                  block_tokens=4, blocks_per_layer=6, ring_slots=8),
             dict(model=O.model(n_layers=2, n_q_heads=4, n_kv_heads=1, head_dim=8),
                  block_tokens=4, blocks_per_layer=7, ring_slots=8)]
    pool = O.OraclePool(parts, n_tags=1024, payload=True)
    assert [pool.info(q)["n"] for q in range(3)] == [30, 18, 14]
    assert [pool.info(q)["base"] for q in range(3)] == [0, 30, 48]
    assert [pool.info(q)["entry_bytes"] for q in range(3)] == [2 * 4 * 8 * 2, 16 * 4 * 2, 2 * 4 * 8 * 2]
    assert [pool.info(q)["n_chunks"] for q in range(3)] == [2, 1, 2]
    _fill(pool)
    r = np.random.default_rng(8)
    for epoch in range(6):
        ev = r.integers(0, pool.N, 40).astype(np.uint32)
        pool.epoch_score(epoch, ev, np.ones(40, np.uint8))
        rc, v = pool.select_victims(12)
        assert rc == O.OK and pool.demote(v) == O.OK
        for q in range(3):
            live = np.flatnonzero(pool.part_array(q, "r_live"))
            inf = pool.info(q)
            n_free = int((pool.state[inf["base"]:inf["base"] + inf["n"]] == O.FREE).sum())
            take = live[:min(2, n_free)].astype(np.uint64)
            assert pool.promote(q, take) == O.OK
        in_hbm, on_host = _check_conservation(pool, pool.next_tag)
        _check_payload(pool, in_hbm, on_host)
        _fill(pool, epoch=epoch, seed=epoch)
