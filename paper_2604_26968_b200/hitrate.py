"""Cache hit rates of the three eviction policies on a synthetic trace.

    python -m paper_2604_26968_b200.hitrate POOL SCALE EPOCHS

The paper's table of cache hit rates compares a reactive policy (LRU), a
pattern-aware one (EMA only) and the Bayesian predictor on real traces, which are
not available offline; this replays a synthetic trace of the same shape through
the CUDA library once per policy and counts, for every touch of an epoch, where
the block that lived in the touched slot one epoch earlier is now: still (or
again) in HBM, in the pinned host tier, or dropped from it.  A touch of a block
that the previous epoch evicted is what a serving engine would see as a miss of
tier 0.  The traces address physical slots, so the victims a policy picks do not
change the trace: the three runs see the same touches.  Context for the paper's
table, not a reproduction of it.
"""
import sys

import numpy as np


POLICIES = (("LRU", 2), ("EMA only", 1), ("Bayesian", 0))


def replay(cfg, scale, epochs, policy, seed_offset=0):
    """Returns (touches, found in HBM, found on the host, dropped) summed over the epochs."""
    from . import binding as B
    from . import workloads as W
    from .harness import EpochRunner
    w = W.config(cfg, scale=scale)
    w.seed += seed_offset
    w.epochs = epochs + 2
    r = EpochRunner(w, batch_bytes=64 << 20, fill_pattern=False, host_meta=False)
    p = r.pool
    r.check(p.kv_set_policy(policy), "kv_set_policy")
    p.kv_set_deferred_packing(True)
    tot = np.zeros(4, np.int64)
    tags_before = None
    for e in range(epochs):
        ev_entry, ev_hit = r.next_events(e)
        n_trace = ev_entry.size - (0 if r.fresh is None else len(r.fresh))   # without the admissions' own touches
        if tags_before is not None and n_trace > 0:
            touched = np.unique(ev_entry[:n_trace])
            loc = r.host_array("loc")
            where = loc[tags_before[touched]]
            hbm = int(((where & B.KV_LOC_HOST) == 0).sum())       # (KV_NONE has bit 31 set)
            dropped = int((where == B.KV_NONE).sum())
            tot += (touched.size, hbm, touched.size - hbm - dropped, dropped)
        d_e, d_h, n = r.stage_events(ev_entry, ev_hit)
        tags_before = r.host_array("tag").copy()       # who lives where while this epoch's touches arrive
        r.step(e, d_e, d_h, n)
    assert p.kv_device_status() == 0
    r.close()
    return tot


def main(argv):
    if len(argv) != 4:
        raise SystemExit(__doc__)
    cfg, scale, epochs = int(argv[1]), float(argv[2]), int(argv[3])
    print("| pool | scale | epochs | policy | touches | in HBM | on the host | dropped | HBM hit rate |")
    print("|---|---|---|---|---|---|---|---|---|")
    for name, pol in POLICIES:
        t = replay(cfg, scale, epochs, pol)
        print("| %d | %.4g | %d | %s | %d | %d | %d | %d | %.1f %% |" % (
            cfg, scale, epochs, name, t[0], t[1], t[2], t[3], 100.0 * t[1] / max(t[0], 1)), flush=True)


if __name__ == "__main__":
    main(sys.argv)
