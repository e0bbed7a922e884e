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
