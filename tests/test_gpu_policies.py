"""Policy variants and the confidence-weighted reuse estimate: CUDA library
against the CPU oracle, bit for bit, through the C ABI."""
import numpy as np
import pytest

from paper_2604_26968_b200 import binding as B
from paper_2604_26968_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("policy", [B.KV_POLICY_EMA, B.KV_POLICY_LRU])
def test_lru_and_ema_only_policies_match_the_oracle(policy):
    from lockstep import Lockstep
    w = W.config(1)
    ls = Lockstep(w, payload=False, batch_bytes=256 << 10, policy=policy)
    for e in range(12):
        ls.epoch(e)
    if policy == B.KV_POLICY_LRU:      # scores are epochs: small integers, massive ties, resolved by id
        sc = ls.ora.score[ls.ora.state == 1]
        assert np.all(sc == np.round(sc)) and sc.max() <= 11
    ls.close()


@pytest.mark.parametrize("kappa,window", [(50.0, 5), (4000.0, 1), (0.5, 64)])
def test_confidence_blend_matches_the_oracle(kappa, window):
    from lockstep import Lockstep
    w = W.config(1)
    ls = Lockstep(w, payload=False, batch_bytes=256 << 10, blend=(kappa, window))
    differs = False
    for e in range(window + 6 if window < 30 else 70):
        ls.epoch(e)
        differs |= not np.array_equal(ls.ora.estimate, ls.ora.P)
    assert differs          # the blend really moved the estimate away from the posterior
    ls.close()


def test_blend_and_policy_on_a_four_partition_pool_and_switching_mid_run():
    from lockstep import Lockstep
    w = W.config(5, scale=1 / 256)
    for p in w.parts:
        p.ring_slots = w.k + 64
    ls = Lockstep(w, payload=False, batch_bytes=4 << 20, blend=(200.0, 3))
    g, o = ls.gpu.pool, ls.ora
    for e in range(4):
        ls.epoch(e)
    assert g.kv_set_policy(B.KV_POLICY_LRU) == 0 and o.set_policy(2) == 0
    ls.epoch(4)
    assert g.kv_set_confidence_blend(10.0, 0) == 0 and o.set_confidence_blend(10.0, 0) == 0   # off
    assert g.kv_set_policy(B.KV_POLICY_BAYESIAN) == 0 and o.set_policy(0) == 0
    ls.epoch(5)
    assert np.array_equal(o.estimate, o.P)
    # refused arguments
    assert g.kv_set_policy(3) == B.KV_ERR_INVALID_ARG
    assert g.kv_set_confidence_blend(0.0, 4) == B.KV_ERR_INVALID_ARG
    assert g.kv_set_confidence_blend(1.0, 65) == B.KV_ERR_INVALID_ARG
    ls.close()


@pytest.mark.parametrize("cfg,scale", [(1, 1.0), (2, 1 / 32), (5, 1 / 128)])
def test_block_granular_selection_matches_the_oracle(cfg, scale):
    """Whole paged blocks evicted by weighted aggregate over heads: single-partition pools
    (count known on the host) and the four-architecture pool (weights 1 / 8 / 32 / 128)."""
    from lockstep import Lockstep
    w = W.config(cfg, scale=scale)
    n_blocks = sum(p.n_layers * p.blocks_per_layer for p in w.parts)
    for p in w.parts:
        # room for every block a call may take from one partition
        p.ring_slots = p.n_entries + 64 if cfg == 5 else max(p.ring_slots, min(p.n_entries, w.N // 4) + 64)
    ls = Lockstep(w, payload=(cfg != 2), batch_bytes=4 << 20)
    seen_parts = set()
    for e, kb in enumerate([n_blocks // 20, 1, 0, n_blocks // 9, n_blocks // 20]):
        ls.epoch(e, k_blocks=kb)
        seen_parts |= {q for q, c in enumerate(ls.gpu.pool.kv_last_demote_counts()) if c > 0}
    if cfg == 5:
        assert len(seen_parts) >= 2
    # more blocks than exist is refused on the host
    rc, _ = ls.gpu.pool.kv_select_victim_blocks(n_blocks + 1, ls.gpu.victims)
    assert rc == B.KV_ERR_K_TOO_LARGE
    ls.close()


def test_block_selection_skips_partially_resident_blocks():
    import torch
    from lockstep import Lockstep
    from oracle import kv_oracle as O
    w = W.Workload("partial", [W.gqa(2, 8, 4, 8, 4, 50, 500, "entry")], 0.05, 0.0, seed=6)
    ls = Lockstep(w, payload=False, batch_bytes=1 << 20)
    g, o = ls.gpu, ls.ora
    ls.epoch(0)
    # knock single heads out of a few blocks, then score again: those blocks stop being candidates
    holes = np.array([1, 6, 40, 41, 399], np.uint32)
    assert o.demote(holes) == O.OK
    g.check(g.pool.kv_demote(torch.from_numpy(holes.view(np.int32)).to(g.pool.device), len(holes), 1 << 20),
            "kv_demote")
    assert o.epoch_score(1, [], []) == O.OK
    g.check(g.pool.kv_epoch_score(1, None, None, 0), "kv_epoch_score")
    n_cand = 100 - 4
    for kb in (10, n_cand):
        rc, v = o.select_victim_blocks(kb)
        assert rc == O.OK
        rc, m = g.pool.kv_select_victim_blocks(kb, g.victims)
        assert rc == 0 and m == len(v) == 4 * kb
        g.pool.sync()
        assert np.array_equal(g.victims[:m].cpu().numpy().view(np.uint32), v)
        assert not (set(v.tolist()) & {0, 2, 3, 4, 5, 7, 42, 43, 396, 397, 398})
    assert g.pool.kv_device_status() == 0
    rc, _ = o.select_victim_blocks(n_cand + 1)
    assert rc == O.ERR_K_TOO_LARGE
    rc, m = g.pool.kv_select_victim_blocks(n_cand + 1, g.victims)      # the host cannot know: flagged on the device
    assert rc == 0
    assert g.pool.kv_device_status() == 4
    ls.close()
