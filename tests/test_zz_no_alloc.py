"""kv_select_victims_static against the oracle and against kv_select_victims.

Some users of the library cannot allocate device memory when they need a
selection (an inference server that has already carved the whole GPU into its
own pools, or code on a path where cudaMalloc is not allowed), so they cannot
give the library a workspace.  The static entry point keeps its scratch inside
the library instead.  Here it is called twice in a row through the C ABI, on
different scores and different k, and must return exactly the ids the CPU
oracle selects from the same scores and states (the two sides are compared bit
for bit first) -- which are also the ids of the pool-based entry point
(selection is integer work: bit-exact).

This file is named so that pytest collects it last.
"""
import numpy as np
import pytest

from oracle import kv_oracle as O
from paper_2604_26968_b200 import binding as B
from paper_2604_26968_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_static_selection_matches_the_oracle_on_two_calls_in_a_row():
    import torch
    from lockstep import Lockstep
    # 2 x 613 x 4 = 4,904 entries: several 2,048-entry tiles and a ragged tail
    w = W.Workload("static-select", [W.gqa(2, 16, 4, 64, 16, 613, 2048, "entry")], 0.05, 0.02, seed=7)
    ls = Lockstep(w, payload=False, batch_bytes=1 << 20)
    g, o = ls.gpu, ls.ora
    pool = g.pool
    N = w.N
    status = torch.zeros(4, dtype=torch.int32, device=pool.device)
    fresh = ls.fresh
    for call, k in enumerate((N // 20, N // 3)):
        if call == 0:
            ev_entry, ev_hit = w.events(call, o.pair, fresh)
        else:              # (no touches on the pool with FREE holes: a trace would name some of them)
            ev_entry, ev_hit = np.zeros(0, np.uint32), np.zeros(0, np.uint8)
        d_e, d_h, n = g.stage_events(ev_entry, ev_hit)
        assert o.epoch_score(call, ev_entry, ev_hit) == O.OK
        g.check(pool.kv_epoch_score(call, d_e, d_h, n), "kv_epoch_score")
        ls.compare_state("scores of call %d" % call)       # same scores and states on both sides
        rc, want = o.select_victims(k)
        assert rc == O.OK
        ref = torch.full((max(k, 4),), -1, dtype=torch.int32, device=pool.device)
        got = torch.full((max(k, 4),), -1, dtype=torch.int32, device=pool.device)
        rc = B.kv_select_victims_static(pool.score, pool.state, N, k, got, status, pool.compute)
        assert rc == B.KV_OK
        g.check(pool.kv_select_victims(k, ref), "kv_select_victims")
        pool.sync()
        assert np.array_equal(got[:k].cpu().numpy().view(np.uint32), want), "static entry point vs oracle"
        assert np.array_equal(ref[:k].cpu().numpy().view(np.uint32), want), "pool entry point vs oracle"
        assert int(status[0].item()) == 0 and pool.kv_device_status() == 0
        if call == 0:      # FREE holes for the second call: demote the first call's victims
            assert o.demote(want) == O.OK
            g.check(pool.kv_demote(ref, k, g.batch_bytes), "kv_demote")
    # sizes beyond the built-in scratch are refused, and so is k > n
    assert B.kv_select_victims_static(pool.score, pool.state, (1 << 22) + 1, 1, got, None, pool.compute) \
        == B.KV_ERR_INVALID_ARG
    assert B.kv_select_victims_static(pool.score, pool.state, N, N + 1, got, None, pool.compute) \
        == B.KV_ERR_K_TOO_LARGE
    ls.close()
