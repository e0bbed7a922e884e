"""Pins for the oracle's per-layer prefetch window and prefetch list (RoPE-aware
prefetching section: promotion requests for the blocks covering positions [n, n+w]
-- or [n-w, n], the range the section calls likeliest to be read next -- with a
window w that adapts per layer to the observed attention span, narrow for local
layers and wide for global ones).  The section prints no formula, so the tests pin
what it states in words and the arithmetic of the reading:
    S[l] <- d*S[l] + (1-d)*x[l]  (tokens);  w[l] = clamp(ceil(S[l]/block_tokens), 1, w_max);
    list = ring slots of the host-tier blocks at distance < w[l] from the current
           position-block, ordered by (distance, layer, head).
"""
import numpy as np
import pytest

from oracle import kv_oracle as O

L, H, NB, BT = 3, 2, 16, 4


def _pool(layers=L, hkv=H, blocks=NB, bt=BT, ring=256):
    m = O.model(variant=O.GQA, n_layers=layers, n_q_heads=4 * hkv, n_kv_heads=hkv, head_dim=8)
    parts = [dict(model=m, block_tokens=bt, blocks_per_layer=blocks, ring_slots=ring)]
    p = O.OraclePool(parts, n_tags=1 << 14, payload=False)
    p.admit(0, 0.5, np.zeros(p.N, dtype=np.uint8), None)
    return p


def _table(p, layers=L, hkv=H, blocks=NB):
    """Sequence whose position-block pb lives in slab block pb: handles [pb][l][h]."""
    tag = p.tag.reshape(layers, blocks, hkv)
    return np.ascontiguousarray(tag.transpose(1, 0, 2)).copy()


def test_default_window_is_2048_tokens_in_blocks_and_bounds():
    p = _pool()
    assert np.array_equal(p.prefetch_array(0, "span"), np.full(L, 2048.0, np.float32))
    assert np.array_equal(p.prefetch_array(0, "window"), np.full(L, 2048 // BT, np.uint32))
    q = _pool(bt=16)
    assert np.array_equal(q.prefetch_array(0, "window"), np.full(L, 128, np.uint32))
    assert q.set_prefetch_window(0, 2048.0, 100) == O.OK          # the cap
    assert np.array_equal(q.prefetch_array(0, "window"), np.full(L, 100, np.uint32))
    assert q.set_prefetch_window(0, 0.0, 100) == O.OK             # never less than one block
    assert np.array_equal(q.prefetch_array(0, "window"), np.full(L, 1, np.uint32))
    for tokens, want in ((16.0, 1), (16.5, 2), (17.0, 2), (32.0, 2), (33.0, 3), (1.0, 1)):
        assert q.set_prefetch_window(0, tokens, 1000) == O.OK     # ceiling: a started block counts
        assert int(q.prefetch_array(0, "window")[0]) == want


def test_span_recurrence_closed_forms():
    p = _pool()
    d = 0.875
    x = np.array([64.0, 512.0, 4096.0], np.float32)
    assert p.set_prefetch_window(0, 1024.0, 1 << 16) == O.OK
    for t in range(1, 40):
        assert p.prefetch_window_update(0, x, d) == O.OK
        want = x.astype(np.float64) + (1024.0 - x.astype(np.float64)) * d ** t   # S_t = x + (S_0 - x) d^t
        got = p.prefetch_array(0, "span").astype(np.float64)
        assert np.all(np.abs(got - want) <= 1e-5 * np.abs(want))
        w = p.prefetch_array(0, "window")
        assert np.array_equal(w, np.ceil(p.prefetch_array(0, "span").astype(np.float64) / BT).astype(np.uint32))
        assert w[0] < w[1] < w[2]                  # narrow for the local layer, wide for the global one
    # converges to x (binary32 stalls within a few ulps of it, about ulp/(1-d), and a span
    # a hair over a block boundary starts the next block)
    for _ in range(400):
        p.prefetch_window_update(0, x, d)
    assert np.all(np.abs(p.prefetch_array(0, "span").astype(np.float64) - x) <= 2e-6 * x)
    assert np.all(np.abs(p.prefetch_array(0, "window").astype(np.int64) - np.array([16, 128, 1024])) <= 1)
    # d = 0 replaces, d = 1 keeps
    assert p.prefetch_window_update(0, np.array([8, 9, 10], np.float32), 0.0) == O.OK
    assert np.array_equal(p.prefetch_array(0, "span"), np.array([8, 9, 10], np.float32))
    assert np.array_equal(p.prefetch_array(0, "window"), np.array([2, 3, 3], np.uint32))
    assert p.prefetch_window_update(0, np.zeros(3, np.float32), 1.0) == O.OK
    assert np.array_equal(p.prefetch_array(0, "span"), np.array([8, 9, 10], np.float32))


def test_recurrence_is_binary32_one_rounding_per_operation():
    p = _pool()
    r = np.random.default_rng(5)
    s = np.full(L, 2048.0, np.float32)
    for _ in range(50):
        x = (r.random(L) * 8192).astype(np.float32)
        d = np.float32(r.random())
        assert p.prefetch_window_update(0, x, float(d)) == O.OK
        s = (d * s).astype(np.float32) + ((np.float32(1.0) - d) * x).astype(np.float32)
        assert np.array_equal(p.prefetch_array(0, "span").view(np.uint32), s.astype(np.float32).view(np.uint32))


def test_window_is_monotone_in_the_span():
    p = _pool()
    last = 0
    for tokens in np.linspace(0, 5000, 301):
        assert p.set_prefetch_window(0, float(tokens), 1 << 16) == O.OK
        w = int(p.prefetch_array(0, "window")[0])
        assert w >= last and (w - 1) * BT < max(float(np.float32(tokens)), 1e-30) <= w * BT or tokens == 0
        last = w


def test_invalid_arguments():
    p = _pool()
    x = np.ones(L, np.float32)
    assert p.prefetch_window_update(1, x, 0.5) == O.ERR_INVALID_ARG
    assert p.prefetch_window_update(0, x, -0.1) == O.ERR_INVALID_ARG
    assert p.prefetch_window_update(0, x, 1.5) == O.ERR_INVALID_ARG
    assert p.prefetch_window_update(0, x, float("nan")) == O.ERR_INVALID_ARG
    assert p.prefetch_window_update(0, np.array([1, -1, 1], np.float32), 0.5) == O.ERR_INVALID_ARG
    assert p.prefetch_window_update(0, np.array([1, np.inf, 1], np.float32), 0.5) == O.ERR_INVALID_ARG
    assert p.prefetch_window_update(0, np.array([1, np.nan, 1], np.float32), 0.5) == O.ERR_INVALID_ARG
    assert np.array_equal(p.prefetch_array(0, "span"), np.full(L, 2048.0, np.float32))   # nothing changed
    assert p.set_prefetch_window(0, -1.0, 4) == O.ERR_INVALID_ARG
    assert p.set_prefetch_window(0, 8.0, 0) == O.ERR_INVALID_ARG
    t = _table(p)
    assert p.prefetch_list(0, t, NB, 1)[0] == O.ERR_INVALID_ARG      # position outside the table
    assert p.prefetch_list(0, t, 0, 0)[0] == O.ERR_INVALID_ARG       # no direction
    assert p.prefetch_list(1, t, 0, 1)[0] == O.ERR_INVALID_ARG


def _demote_blocks(p, blocks):
    """Demotes every (layer, head) entry of the given slab blocks; returns {tag: ring slot}."""
    ids = np.array([(l * NB + b) * H + h for b in blocks for l in range(L) for h in range(H)], np.uint32)
    ids.sort()
    tags = p.tag[ids].copy()
    assert p.demote(ids) == O.OK
    loc = p.loc
    assert np.all(loc[tags] & 0x80000000)
    return {int(t): int(loc[t] & 0x7FFFFFFF) for t in tags}


def _brute(table, win, where, pos0, direction):
    """The definition, written as a sort: all (distance, layer, head) inside the windows."""
    n_pos = table.shape[0]
    keys = []
    for pb in range(n_pos):
        dist = (pb - pos0) * direction
        if dist < 0:
            continue
        for l in range(table.shape[1]):
            for h in range(table.shape[2]):
                if dist < win[l] and int(table[pb, l, h]) in where:
                    keys.append((dist, l, h, where[int(table[pb, l, h])]))
    return [k[3] for k in sorted(keys)]


def test_list_on_a_hand_built_table():
    p = _pool()
    t = _table(p)
    where = _demote_blocks(p, [2, 3, 4, 6, 9])
    assert p.prefetch_window_update(0, np.array([4.0, 12.0, 40.0], np.float32), 0.0) == O.OK
    win = p.prefetch_array(0, "window")
    assert np.array_equal(win, np.array([1, 3, 10], np.uint32))
    # at block 2 going forward: layer 0 wants block 2; layer 1 blocks 2..4; layer 2 blocks 2..11
    rc, slots, n = p.prefetch_list(0, t, 2, 1)
    assert rc == O.OK
    s = lambda b, l, h: where[int(t[b, l, h])]
    want = [s(2, 0, 0), s(2, 0, 1), s(2, 1, 0), s(2, 1, 1), s(2, 2, 0), s(2, 2, 1),
            s(3, 1, 0), s(3, 1, 1), s(3, 2, 0), s(3, 2, 1),
            s(4, 1, 0), s(4, 1, 1), s(4, 2, 0), s(4, 2, 1),
            s(6, 2, 0), s(6, 2, 1), s(9, 2, 0), s(9, 2, 1)]
    assert n == len(want) and slots.tolist() == want
    # backward from block 9: layer 0 wants 9; layer 1 wants 9, 8, 7; layer 2 wants 9 .. 0
    rc, slots, n = p.prefetch_list(0, t, 9, -1)
    want = [s(9, l, h) for l in range(3) for h in range(2)]
    want += [s(6, 2, 0), s(6, 2, 1)] + [s(b, 2, h) for b in (4, 3, 2) for h in range(2)]
    assert rc == O.OK and n == len(want) and slots.tolist() == want
    # a cut list reports the full count and fills only max_out
    rc, slots, n = p.prefetch_list(0, t, 2, 1, max_out=5)
    assert rc == O.OK and n == 18 and slots.tolist() == [s(2, 0, 0), s(2, 0, 1), s(2, 1, 0), s(2, 1, 1), s(2, 2, 0)]
    # nothing on the host inside the windows
    rc, slots, n = p.prefetch_list(0, t, 12, 1)
    assert rc == O.OK and n == 0 and slots.size == 0


@pytest.mark.parametrize("seed", range(6))
def test_list_equals_brute_force_and_promotes(seed):
    r = np.random.default_rng(seed)
    p = _pool()
    t = _table(p)
    perm = r.permutation(NB)                    # the sequence's blocks are scattered over the slab
    t = t[perm]
    where = _demote_blocks(p, r.choice(NB, 7, replace=False).tolist())
    t[r.integers(0, NB), r.integers(0, L), r.integers(0, H)] = 0xFFFFFFFF      # a handle never admitted
    t[r.integers(0, NB), r.integers(0, L), r.integers(0, H)] = (1 << 14) + 3   # beyond the handle space
    assert p.prefetch_window_update(0, (r.random(L) * 60).astype(np.float32), 0.0) == O.OK
    win = p.prefetch_array(0, "window")
    for pos0 in (0, 5, NB - 1):
        for direction in (1, -1):
            rc, slots, n = p.prefetch_list(0, t, pos0, direction)
            want = _brute(t, win, where, pos0, direction)
            assert rc == O.OK and n == len(want) and slots.tolist() == want
    rc, slots, n = p.prefetch_list(0, t, 3, 1)
    if n:
        assert len(set(slots.tolist())) == n                   # a promote list names a slot once
        assert p.promote(0, slots) == O.OK
        loc = p.loc
        rc, again, n2 = p.prefetch_list(0, t, 3, 1)
        assert rc == O.OK and n2 == 0                          # they are in HBM now
