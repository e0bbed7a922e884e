"""kv_select_victims_static against kv_select_victims.

Some users of the library cannot allocate device memory when they need a
selection (an inference server that has already carved the whole GPU into its
own pools, or code on a path where cudaMalloc is not allowed), so they cannot
give the library a workspace.  The static entry point keeps its scratch inside
the library instead.  Here it is called twice in a row through the C ABI, on
different scores and different k, and must return exactly the ids the
pool-based entry point returns (selection is integer work: bit-exact).

This file is named so that pytest collects it last.
"""
import numpy as np
import pytest

from paper_2604_26968_b200 import binding as B
from paper_2604_26968_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_static_selection_matches_pool_selection_on_two_calls_in_a_row():
    import torch
    from paper_2604_26968_b200.harness import EpochRunner
    # 2 x 613 x 4 = 4,904 entries: several 2,048-entry tiles and a ragged tail
    w = W.Workload("static-select", [W.gqa(2, 16, 4, 64, 16, 613, 2048, "entry")], 0.05, 0.02, seed=7)
    r = EpochRunner(w, batch_bytes=1 << 20)
    pool = r.pool
    N = w.N
    status = torch.zeros(4, dtype=torch.int32, device=pool.device)
    for call, k in enumerate((N // 20, N // 3)):
        ev_entry, ev_hit = r.next_events(call)
        d_e, d_h, n = r.stage_events(ev_entry, ev_hit)
        r.check(pool.kv_epoch_score(call, d_e, d_h, n), "kv_epoch_score")
        if call == 1:      # FREE holes: demote the first call's victims
            r.check(pool.kv_demote(ref, len(first), r.batch_bytes), "kv_demote")
            r.check(pool.kv_epoch_score(call + 1, None, None, 0), "kv_epoch_score")
        ref = torch.full((max(k, 4),), -1, dtype=torch.int32, device=pool.device)
        got = torch.full((max(k, 4),), -1, dtype=torch.int32, device=pool.device)
        r.check(pool.kv_select_victims(k, ref), "kv_select_victims")
        rc = B.kv_select_victims_static(pool.score, pool.state, N, k, got, status, pool.compute)
        assert rc == B.KV_OK
        pool.sync()
        first = ref[:k].cpu().numpy()
        assert np.array_equal(first, got[:k].cpu().numpy())
        assert len(set(first.tolist())) == k and np.all(np.diff(first) > 0)
        assert int(status[0].item()) == 0 and pool.kv_device_status() == 0
    # sizes beyond the built-in scratch are refused, and so is k > n
    assert B.kv_select_victims_static(pool.score, pool.state, (1 << 22) + 1, 1, got, None, pool.compute) \
        == B.KV_ERR_INVALID_ARG
    assert B.kv_select_victims_static(pool.score, pool.state, N, N + 1, got, None, pool.compute) \
        == B.KV_ERR_K_TOO_LARGE
    r.close()
