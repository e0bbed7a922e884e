"""Head-granular importance weighting (importance matrix per (layer, query head),
GQA group maximum, task-transition multipliers): CUDA library against the CPU
oracle, bit for bit, through the C ABI."""
import numpy as np
import pytest

from oracle import kv_oracle as O
from paper_2604_26968_b200 import binding as B
from paper_2604_26968_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("policy", [B.KV_POLICY_BAYESIAN, B.KV_POLICY_EMA, B.KV_POLICY_LRU])
def test_head_weights_config1(policy, fused):
    from lockstep import Lockstep
    w = W.config(1)           # GQA, 16 query heads over 4 KV heads
    ls = Lockstep(w, payload=False, batch_bytes=256 << 10, policy=policy, fused=fused, heads=(0.8, 4))
    for e in range(10):
        ls.epoch(e)
    wts = ls.ora.head_array(0, "weights")
    assert wts.min() < wts.max()                  # the matrix really differentiates heads
    ls.close()


@pytest.mark.parametrize("cfg,scale", [(2, 1 / 64), (4, 1 / 128), (5, 1 / 128)])
def test_head_weights_scaled_pools(cfg, scale):
    """GQA group 4, MLA ([layer][1]) and the four-architecture pool (MHA group 1, GQA 8, MQA 32, MLA)."""
    from lockstep import Lockstep
    w = W.config(cfg, scale=scale)
    if cfg == 5:
        for p in w.parts:
            p.ring_slots = w.k + 64
    ls = Lockstep(w, payload=False, batch_bytes=8 << 20, fused=True, heads=(0.9, 3), blend=(100.0, 3))
    for e in range(5):
        ls.epoch(e)
    ls.close()


def test_head_weights_odd_partition_boundaries_and_block_selection():
    """Partition bases that are not multiples of 4 (a 16-byte vector of entries straddles two
    partitions with different matrices); whole-block selection on weighted scores."""
    from lockstep import Lockstep
    from test_gpu_parity import _geom
    parts = _geom("two_parts")
    w = W.Workload("two_parts", parts, 0.2, 0.1, seed=21, promote_style="recent", epochs=8)
    ls = Lockstep(w, payload=False, batch_bytes=1 << 20, heads=(0.5, 2))
    n_blocks = sum(p.n_layers * p.blocks_per_layer for p in parts)
    for e in range(6):
        if e % 2:
            ls.epoch(e, k_blocks=n_blocks // 10)
        else:
            ls.epoch(e)
    ls.close()


def test_only_one_partition_weighted_and_unit_matrix_is_identity():
    from lockstep import Lockstep
    w = W.config(5, scale=1 / 256)
    for p in w.parts:
        p.ring_slots = w.k + 64
    ls = Lockstep(w, payload=False, batch_bytes=4 << 20, fused=True)
    g, o = ls.gpu, ls.ora
    ls.epoch(0)
    # partition 1 only
    x = w.head_observations(0, 1)
    assert o.head_importance_update(1, x, 0.0) == O.OK
    d_x = g.to_device(x.reshape(-1), None)
    g.check(g.pool.kv_head_importance_update(1, d_x, 0.0), "kv_head_importance_update")
    ls.epoch(1)
    # a unit matrix leaves partition 0's scores as they would be unweighted
    ones = np.ones(w.parts[0].n_layers * w.parts[0].n_q_heads, np.float32)
    assert o.head_importance_update(0, ones, 0.3) == O.OK
    d_1 = g.to_device(ones, None)
    g.check(g.pool.kv_head_importance_update(0, d_1, 0.3), "kv_head_importance_update")
    ls.epoch(2)
    ls.close()


def test_bad_values_are_skipped_and_flagged_and_bad_arguments_refused():
    from lockstep import Lockstep
    import torch
    w = W.config(1)
    ls = Lockstep(w, payload=False, batch_bytes=256 << 10)
    g, o, p = ls.gpu, ls.ora, ls.gpu.pool
    x = w.head_observations(0, 0)
    good = x.copy()
    x[1, 3], x[0, 0], x[1, 9] = -1.0, np.nan, np.inf
    d_x = g.to_device(x.reshape(-1), None)
    g.check(p.kv_head_importance_update(0, d_x, 0.5), "kv_head_importance_update")
    p.sync()
    assert p.kv_device_status() == B.KV_DEV_BAD_HEAD_VALUE
    got = p.kv_head_importance(0).cpu().numpy().reshape(2, 16)
    want = np.float32(0.5) * np.float32(1.0) + np.float32(0.5) * good      # M started at 1
    bad = np.zeros((2, 16), bool)
    bad[1, 3] = bad[0, 0] = bad[1, 9] = True
    assert np.array_equal(got[~bad], want[~bad]) and np.all(got[bad] == 1.0)
    assert o.head_importance_update(0, x, 0.5) == O.ERR_INVALID_ARG       # the oracle refuses the lot
    m = np.ones((2, 4), np.float32)
    m[0, 2] = -3.0
    d_m = g.to_device(m.reshape(-1), None)
    g.check(p.kv_set_head_multipliers(0, d_m), "kv_set_head_multipliers")
    p.sync()
    assert p.kv_device_status() == B.KV_DEV_BAD_HEAD_VALUE
    assert p.kv_head_importance_update(1, d_x, 0.5) == B.KV_ERR_INVALID_ARG      # no such partition
    assert p.kv_head_importance_update(0, d_x, 1.5) == B.KV_ERR_INVALID_ARG
    assert p.lib.kv_head_importance_update(p._h, 0, d_x.data_ptr() + 4, 0.5, None) == B.KV_ERR_INVALID_ARG
    assert p.lib.kv_head_importance_update(p._h, 0, None, 0.5, None) == B.KV_ERR_INVALID_ARG
    assert p.kv_set_head_multipliers(2, None) == B.KV_ERR_INVALID_ARG
    ls.close()
