"""CUDA library against the CPU oracle, element by element, through the C ABI.

Everything compared is bit-exact: victim lists, states, tags, block tables, ring
contents, byte counters, and (because both sides do the same rounded binary32
operations in the same order) EMA values, posteriors and scores, which is
stricter than the 1e-6 relative tolerance the scores are allowed.
"""
import numpy as np
import pytest

from oracle import kv_oracle as O
from paper_2604_26968_b200 import binding as B
from paper_2604_26968_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_config1_tiny_gqa_50_epochs_bit_exact():
    from lockstep import Lockstep
    w = W.config(1)
    ls = Lockstep(w, payload=True, batch_bytes=256 << 10)
    tot = dict(events=0, promoted=0, admitted=0)
    for e in range(w.epochs):
        r = ls.epoch(e)
        for k_ in tot:
            tot[k_] += r[k_]
    # 819 drawn touches per epoch plus one miss event per block admitted the epoch before
    assert tot["events"] >= 50 * 819 + 4096 and tot["promoted"] > 0 and tot["admitted"] > 0
    assert ls.ora.stats()["bytes_dropped"] > 0       # the 4,096-slot ring wrapped
    ls.close()


@pytest.mark.parametrize("cfg,scale,epochs", [(2, 1 / 64, 6), (3, 1 / 192, 4), (4, 1 / 128, 5), (5, 1 / 128, 5)])
def test_scaled_pools_full_payload(cfg, scale, epochs):
    """Pools 2-5 shrunk so the oracle can hold every byte: several tiles, ragged
    tails, MLA chunks, four partitions, ring wrap."""
    from lockstep import Lockstep
    w = W.config(cfg, scale=scale)
    if cfg == 5:    # ties send most victims to the first partition: give every ring room for k
        for p in w.parts:
            p.ring_slots = w.k + 64
    ls = Lockstep(w, payload=True, batch_bytes=8 << 20)
    for e in range(epochs):
        r = ls.epoch(e)
        assert r["events"] > 0
    assert ls.gpu.pool.kv_get_stats()["bytes_promoted"] > 0
    ls.close()


def _geom(kind):
    if kind == "gqa_odd":      # N = 1*37*3 = 111: not a multiple of 4, 8 or 2048
        return [W.gqa(1, 6, 3, 8, 4, 37, 40, "entry")]
    if kind == "mla_small":    # H = 1, one 320-byte chunk per entry
        return [W.mla(3, 32, 8, 4, 5, 9, "entry")]
    if kind == "two_parts":    # partition boundary not tile aligned
        return [W.mha(1, 3, 8, 4, 701, 1000, "entry"), W.mla(2, 24, 8, 2, 333, 1000, "entry")]
    raise ValueError(kind)


@pytest.mark.parametrize("kind", ["gqa_odd", "mla_small", "two_parts"])
@pytest.mark.parametrize("batch_entries", [1, 3, 1000])
def test_odd_geometries_and_tiny_batches(kind, batch_entries):
    """Ragged sizes, single-entry chunks (many launches, both staging buffers, ring wrap
    inside a call), every k from 0 to all resident entries."""
    from lockstep import Lockstep
    parts = _geom(kind)
    w = W.Workload(kind, parts, 0.2, 0.1, seed=11, promote_style="recent", epochs=12)
    eb = max(p.entry_bytes for p in parts)
    ls = Lockstep(w, payload=True, batch_bytes=batch_entries * eb, staging_bytes=batch_entries * (eb + 24) + 512)
    N = w.N
    ks = [0, 1, N // 7, N // 3, 0, 5, N // 5, N // 9, 2, N // 4, 7, N // 6]
    for e in range(12):
        k = ks[e]
        if parts[0].ring_slots < k:
            k = parts[0].ring_slots
        ls.epoch(e, k=k)
    ls.close()


def test_select_all_resident_and_all_ties():
    from lockstep import Lockstep
    w = W.Workload("ties", [W.gqa(2, 8, 2, 8, 4, 1100, 5000, "entry")], 0.1, 0.0, seed=3)
    ls = Lockstep(w, payload=False, batch_bytes=1 << 20)
    g, o = ls.gpu, ls.ora
    N = w.N
    # epoch with no events at all: every score is +0 -> ties everywhere -> first k ids
    assert o.epoch_score(0, [], []) == O.OK
    g.check(g.pool.kv_epoch_score(0, None, None, 0), "kv_epoch_score")
    import torch
    big = torch.empty(N, dtype=torch.int32, device=g.pool.device)
    for k in (1, 777, N):
        rc, v = o.select_victims(k)
        assert rc == O.OK and v.tolist() == list(range(k))
        big.fill_(-1)
        g.check(g.pool.kv_select_victims(k, big), "kv_select_victims")
        g.pool.sync()
        assert np.array_equal(big[:k].cpu().numpy(), np.arange(k))
        assert int(big[k:].max().item()) == -1 if k < N else True     # nothing written past k
    assert g.pool.kv_select_victims(N + 1, big) == B.KV_ERR_K_TOO_LARGE
    ls.compare_state("ties")
    ls.close()


def test_denormal_ema_and_huge_touch_count():
    """decay 1e-20 drives an untouched EMA through the denormal range (1 -> 1e-20 ->
    1e-40 -> 0): flush-to-zero on either side would break bit equality.  One entry
    also receives 2^24 + 3 touches in one epoch (not representable exactly in binary32)."""
    from lockstep import Lockstep
    w = W.Workload("denormal", [W.gqa(1, 8, 2, 8, 4, 300, 1000, "entry")], 0.05, 0.02, seed=5, decay=1e-20,
                   promote_style="recent")
    ls = Lockstep(w, payload=False, batch_bytes=1 << 20)
    saw_denormal = False
    for e in range(5):
        ls.epoch(e)
        ema = ls.ora.ema
        saw_denormal |= bool(((ema > 0) & (ema < np.finfo(np.float32).tiny)).any())
    assert saw_denormal
    g, o = ls.gpu, ls.ora
    n = (1 << 24) + 3
    ev = np.full(n, 17, np.uint32)
    hit = np.ones(n, np.uint8)
    d_e, d_h, nn = g.stage_events(ev, hit)
    assert o.epoch_score(9, ev, hit) == O.OK
    g.check(g.pool.kv_epoch_score(9, d_e, d_h, nn), "kv_epoch_score")
    ls.compare_state("huge touch")
    assert o.ema[17] == np.float32(n)      # rounds to 2^24 + 4
    ls.close()


def test_signed_zero_negative_and_infinite_scores_order_like_floats():
    """The key transform must order every non-NaN float like `<` does, with -0 == +0."""
    import torch
    from lockstep import Lockstep
    w = W.Workload("keys", [W.gqa(1, 8, 2, 8, 4, 1500, 100, "entry")], 0.1, 0.0, seed=9)
    ls = Lockstep(w, payload=False, batch_bytes=1 << 20)
    g, o = ls.gpu, ls.ora
    N = w.N
    r = np.random.default_rng(0)
    special = np.array([0.0, -0.0, 1e-45, -1e-45, 1.0, -1.0, np.inf, -np.inf, 3e38, -3e38, 1e-38, 2.5], np.float32)
    sc = special[r.integers(0, special.size, N)]
    sc[::7] = r.standard_normal(sc[::7].size).astype(np.float32)
    o.score[:] = sc
    g.pool.score[:N].copy_(torch.from_numpy(sc))
    out = torch.empty(N, dtype=torch.int32, device=g.pool.device)
    for k in (1, 10, N // 2, N - 1, N):
        rc, v = o.select_victims(k)
        assert rc == O.OK
        g.check(g.pool.kv_select_victims(k, out), "kv_select_victims")
        g.pool.sync()
        assert np.array_equal(out[:k].cpu().numpy().view(np.uint32), v), k
    assert g.pool.kv_device_status() == 0
    ls.close()


def test_error_paths_leave_state_untouched():
    from lockstep import Lockstep
    w = W.Workload("errors", [W.gqa(1, 8, 2, 8, 4, 64, 20, "entry")], 0.1, 0.05, seed=2, promote_style="recent")
    ls = Lockstep(w, payload=True, batch_bytes=1 << 16)
    g, o, p = ls.gpu, ls.ora, ls.gpu.pool
    ls.epoch(0)
    eb = w.parts[0].entry_bytes
    # more victims than ring slots
    rc, v = o.select_victims(21)
    assert rc == O.OK
    import torch
    vict = torch.from_numpy(v.view(np.int32)).to(p.device)
    assert p.kv_demote(vict, 21, 1 << 16) == B.KV_ERR_HOST_TIER_TOO_SMALL == o.demote(v)
    # batch smaller than one entry, larger than staging
    assert p.kv_demote(vict, 5, eb - 16) == B.KV_ERR_INVALID_ARG
    assert p.kv_demote(vict, 5, 1 << 30) == B.KV_ERR_INVALID_ARG
    ls.compare_state("after refused demotes", scores=False)
    ls.compare_ring("after refused demotes")
    # promote: dead slot, duplicate, out of range, then more than the free slots
    cur, n_live, live = p.kv_ring_query(0)
    dead = int(np.flatnonzero(live == 0)[0])
    alive = np.flatnonzero(live)[:3].astype(np.uint64)
    for bad in ([dead], [int(alive[0]), int(alive[0])], [20]):
        assert p.kv_promote(0, np.array(bad, np.uint64), 1 << 16) == B.KV_ERR_BAD_HOST_SLOT
        assert o.promote(0, np.array(bad, np.uint64)) == O.ERR_BAD_HOST_SLOT
    assert p.kv_promote(0, alive, 1 << 16) == B.KV_ERR_NO_FREE_SLOT == o.promote(0, alive)   # pool is full
    assert p.kv_promote(0, np.zeros(0, np.uint64), 1 << 16) == B.KV_OK
    ls.compare_state("after refused promotes", scores=False)
    ls.compare_ring("after refused promotes")
    # an event on a FREE entry is skipped and flagged; an id beyond N likewise
    assert o.demote(v[:4]) == O.OK
    g.check(p.kv_demote(vict, 4, 1 << 16), "kv_demote")
    ev = np.array([int(v[0]), w.N + 5, int(v[5])], np.uint32)
    d_e, d_h, n = g.stage_events(ev, np.ones(3, np.uint8))
    g.check(p.kv_epoch_score(7, d_e, d_h, n), "kv_epoch_score")
    assert p.kv_device_status() == 1 | 2
    assert o.epoch_score(7, ev[2:], np.ones(1, np.uint8)) == O.OK   # the oracle refuses the bad ones up front
    ls.compare_state("after flagged events")
    ls.close()


def test_full_size_pool2_state_exact_payload_sampled():
    """The benchmark's pool (3,145,728 entries, 24 GiB) in its launch configuration:
    every state array compared in full, block bytes on samples."""
    from lockstep import Lockstep, sample_payload
    w = W.config(2)
    ls = Lockstep(w, payload=False, batch_bytes=64 << 20)
    for e in range(3):
        r = ls.epoch(e)
        assert r["events"] > 100000
        sample_payload(ls, n=96, seed=e)
    assert ls.gpu.pool.kv_get_stats()["bytes_demoted"] == 3 * w.k * 8192
    ls.close()


def _fit_scale(w_factory, headroom=6 << 30):
    """Largest scale <= 1 whose pool fits the free device memory (never skipped silently)."""
    import gc
    import torch
    gc.collect()
    torch.cuda.empty_cache()      # earlier tests' pools sit in torch's caching allocator
    free, _total = torch.cuda.mem_get_info()
    scale = 1.0
    while True:
        w = w_factory(scale)
        need = sum(p.slab_bytes for p in w.parts) + 48 * w.N + 4 * w.n_tags + (1 << 30)
        if need + headroom <= free or scale < 0.05:
            if scale < 1.0:
                print("pool scaled by %.3f to fit %.1f GiB of free device memory" % (scale, free / 2**30))
            return w, scale
        scale *= 0.8


@pytest.mark.parametrize("cfg,epochs", [(3, 2), (4, 3), (5, 3)])
def test_full_size_pools_3_4_5_state_exact_payload_sampled(cfg, epochs):
    """Pools 3 (90 GiB, 11.8 M entries), 4 (MLA, 62.5 GiB) and 5 (four partitions, 150 GiB,
    18.8 M entries) at full size when the device has room: state in full, bytes on samples."""
    from lockstep import Lockstep, sample_payload
    w, scale = _fit_scale(lambda s: W.config(cfg, scale=s))
    ls = Lockstep(w, payload=False, batch_bytes=256 << 20)
    for e in range(epochs):
        r = ls.epoch(e)
        assert r["events"] > 0 and r["promoted"] > 0
        sample_payload(ls, n=48, seed=e)
    if cfg == 5:
        assert sum(1 for c in ls.gpu.pool.kv_last_demote_counts() if c > 0) >= 3   # victims in several partitions
    st = ls.gpu.pool.kv_get_stats()
    assert st["victims"] == epochs * w.k and st["n_entries"] == w.N
    ls.close()
