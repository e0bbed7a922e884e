"""kv_epoch_score_select (per-entry scoring and selection in one kernel) against the CPU
oracle, bit for bit: the same lockstep runs as the two-call path, plus the cases
the fused kernel treats differently (slices larger than its shared-memory key
cache, k = 0, refused arguments, flagged events)."""
import numpy as np
import pytest

from oracle import kv_oracle as O
from paper_2604_26968_b200 import binding as B
from paper_2604_26968_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_fused_config1_50_epochs_bit_exact():
    from lockstep import Lockstep
    w = W.config(1)
    ls = Lockstep(w, payload=True, batch_bytes=256 << 10, fused=True)
    launches0 = ls.gpu.pool.kv_get_stats()["kernel_launches"]
    ls.gpu.check(ls.gpu.pool.kv_epoch_score_select(0, None, None, 0, 0, None), "k = 0, no events")
    assert ls.ora.epoch_score(0, [], []) == O.OK
    # k = 0 scores only: the two scoring kernels (no events: one), never the selection
    assert ls.gpu.pool.kv_get_stats()["kernel_launches"] - launches0 <= 2
    ls.compare_state("score only")
    for e in range(1, w.epochs):
        ls.epoch(e)
    assert ls.ora.stats()["bytes_dropped"] > 0
    ls.close()


def test_fused_is_two_launches():
    from lockstep import Lockstep
    w = W.config(1)
    ls = Lockstep(w, payload=False, batch_bytes=256 << 10, fused=True)
    g, o = ls.gpu, ls.ora
    ev_entry, ev_hit = w.events(0, o.pair, ls.fresh)
    d_e, d_h, n = g.stage_events(ev_entry, ev_hit)
    before = g.pool.kv_get_stats()["kernel_launches"]
    g.check(g.pool.kv_epoch_score_select(0, d_e, d_h, n, w.k, g.victims), "kv_epoch_score_select")
    assert g.pool.kv_get_stats()["kernel_launches"] - before == 2    # event reduction, then everything else
    assert o.epoch_score(0, ev_entry, ev_hit) == O.OK
    rc, v = o.select_victims(w.k)
    g.pool.sync()
    assert np.array_equal(g.victims[:w.k].cpu().numpy().view(np.uint32), v)
    ls.compare_state("two launches")
    ls.close()


@pytest.mark.parametrize("cfg,scale,epochs", [(2, 1 / 64, 5), (3, 1 / 192, 3), (4, 1 / 128, 4), (5, 1 / 128, 4)])
def test_fused_scaled_pools(cfg, scale, epochs):
    from lockstep import Lockstep
    w = W.config(cfg, scale=scale)
    if cfg == 5:
        for p in w.parts:
            p.ring_slots = w.k + 64
    ls = Lockstep(w, payload=True, batch_bytes=8 << 20, fused=True)
    for e in range(epochs):
        assert ls.epoch(e)["events"] > 0
    ls.close()


@pytest.mark.parametrize("kind", ["gqa_odd", "mla_small", "two_parts"])
def test_fused_odd_geometries_every_k(kind):
    from lockstep import Lockstep
    from test_gpu_parity import _geom
    parts = _geom(kind)
    w = W.Workload(kind, parts, 0.2, 0.1, seed=13, promote_style="recent", epochs=12)
    eb = max(p.entry_bytes for p in parts)
    ls = Lockstep(w, payload=True, batch_bytes=64 * eb, fused=True)
    N = w.N
    ks = [0, 1, N // 7, N // 3, 0, 5, N // 5, N // 9, 2, N // 4, 7, N // 6]
    for e in range(12):
        ls.epoch(e, k=min(ks[e], parts[0].ring_slots))
    ls.close()


@pytest.mark.parametrize("policy,blend", [(B.KV_POLICY_EMA, None), (B.KV_POLICY_LRU, None),
                                          (B.KV_POLICY_BAYESIAN, (50.0, 5)), (B.KV_POLICY_BAYESIAN, (0.5, 64))])
def test_fused_policies_and_blend(policy, blend):
    from lockstep import Lockstep
    w = W.config(1)
    ls = Lockstep(w, payload=False, batch_bytes=256 << 10, policy=policy, blend=blend, fused=True)
    for e in range(12 if blend is None or blend[1] < 30 else 70):
        ls.epoch(e)
    ls.close()


def test_fused_alternating_with_the_two_call_path():
    """Both paths leave the same state behind, so they can be mixed freely."""
    from lockstep import Lockstep
    w = W.config(2, scale=1 / 64)
    ls = Lockstep(w, payload=False, batch_bytes=8 << 20, blend=(100.0, 3))
    for e in range(8):
        ls.fused = bool(e & 1)
        ls.epoch(e)
    ls.close()


@pytest.mark.parametrize("cfg", [3, 5])
def test_fused_slices_beyond_the_key_cache(cfg):
    """11.8 M and 18.8 M entries (blocks shrunk to a few bytes): every CTA's slice is longer
    than the keys it can hold in shared memory, so part of it is re-read from the scores."""
    from lockstep import Lockstep
    w = W.config(cfg, tiny_entries=True)
    assert w.N > 148 * 49152
    ls = Lockstep(w, payload=False, batch_bytes=64 << 20, fused=True)
    for e in range(2):
        assert ls.epoch(e)["events"] > 0
    ls.close()


def test_fused_full_size_pool2():
    """The benchmark's pool in the benchmark's launch configuration."""
    from lockstep import Lockstep, sample_payload
    w = W.config(2)
    ls = Lockstep(w, payload=False, batch_bytes=64 << 20, fused=True)
    for e in range(3):
        assert ls.epoch(e)["events"] > 100000
        sample_payload(ls, n=64, seed=e)
    ls.close()


def test_fused_refusals_and_flagged_events():
    from lockstep import Lockstep
    import torch
    w = W.Workload("errors", [W.gqa(1, 8, 2, 8, 4, 64, 64, "entry")], 0.1, 0.05, seed=2, promote_style="recent")
    ls = Lockstep(w, payload=False, batch_bytes=1 << 16, fused=True)
    g, o, p = ls.gpu, ls.ora, ls.gpu.pool
    ls.epoch(0)
    st0 = p.kv_get_stats()
    ev = np.array([3, 4, 5, 6], np.uint32)
    d_e, d_h, n = g.stage_events(ev, np.ones(4, np.uint8))
    # refused before anything runs: k above the resident count, misaligned or missing pointers
    assert p.kv_epoch_score_select(1, d_e, d_h, n, w.N + 1, g.victims) == B.KV_ERR_K_TOO_LARGE
    assert p.lib.kv_epoch_score_select(p._h, 1, d_e.data_ptr() + 4, d_h.data_ptr(), 3, 1, g.victims.data_ptr(),
                                       None) == B.KV_ERR_INVALID_ARG
    assert p.lib.kv_epoch_score_select(p._h, 1, d_e.data_ptr(), d_h.data_ptr(), 4, 1, None,
                                       None) == B.KV_ERR_INVALID_ARG
    st1 = p.kv_get_stats()
    assert st1["epochs"] == st0["epochs"] and st1["events"] == st0["events"]
    ls.compare_state("after refusals", scores=False)
    # events on a FREE entry and beyond N are skipped and flagged, the rest counted
    rc, v = o.select_victims(4)
    assert o.demote(v) == O.OK
    vict = torch.from_numpy(v.view(np.int32)).to(p.device)
    g.check(p.kv_demote(vict, 4, 1 << 16), "kv_demote")
    keep = [i for i in range(w.N) if i not in set(v.tolist())][:3]      # still RESIDENT
    ev = np.array([int(v[0]), w.N + 5] + keep, np.uint32)
    d_e, d_h, n = g.stage_events(ev, np.array([1, 1, 0, 1, 1], np.uint8))
    g.check(p.kv_epoch_score_select(7, d_e, d_h, n, 9, g.victims), "kv_epoch_score_select")
    assert p.kv_device_status() == 1 | 2
    assert o.epoch_score(7, ev[2:], np.array([0, 1, 1], np.uint8)) == O.OK
    rc, v9 = o.select_victims(9)
    p.sync()
    assert np.array_equal(g.victims[:9].cpu().numpy().view(np.uint32), v9)
    ls.compare_state("after flagged events")
    ls.close()
