"""Drives a workload through the CUDA library, epoch by epoch.

Only sequencing and input staging live here; the tests drive the CPU oracle
with the same inputs from their own code.
"""
import numpy as np

from . import binding as B
from . import workloads as W

INITIAL_EPOCH_KEY = 1 << 20   # rng stream key of the initial fill (no real epoch uses it)


class EpochRunner:
    def __init__(self, workload: W.Workload, batch_bytes=64 << 20, staging_bytes=None,
                 fill_pattern=True, host_meta=True, device="cuda:0"):
        import torch
        self.torch = torch
        self.w = workload
        self.batch_bytes = int(batch_bytes)
        max_eb = max(p.entry_bytes for p in workload.parts)
        if staging_bytes is None:
            staging_bytes = self.batch_bytes + (self.batch_bytes // min(p.entry_bytes for p in workload.parts) + 2) * 24 + 64
        staging_bytes = max(int(staging_bytes), max_eb + 256)
        self.pool = B.Pool(workload.parts, workload.n_tags, workload.alpha0, workload.beta0,
                           staging_bytes=staging_bytes, max_promote=self.max_promote(workload),
                           host_meta=host_meta, device=device)
        self.fill_pattern = fill_pattern
        self.k = workload.k
        self.victims = torch.empty(max(self.k, 4), dtype=torch.int32, device=self.pool.device)
        self.fresh = None      # entries admitted by the last admit() (input of the next epoch's trace)
        self.check(self.admit(0, key=INITIAL_EPOCH_KEY), "initial kv_admit")

    @staticmethod
    def max_promote(w):
        """Longest promote list a harness call gives the pool: the workload's promotion share of
        its largest partition (never less than 4,096, for tests that promote by hand)."""
        return max(4096, int(w.promote_frac * max(p.n_entries for p in w.parts)) + 16)

    def next_events(self, epoch):
        """Draws the epoch's trace from the pool's current pair ids and last admissions."""
        return self.w.events(epoch, self.host_array("pair"), self.fresh)

    def check(self, rc, what):
        if isinstance(rc, tuple):
            rc = rc[0]
        if rc != B.KV_OK:
            raise B.KVError(rc, what)

    def to_device(self, arr, dtype):
        t = self.torch.from_numpy(np.ascontiguousarray(arr))
        with self.torch.cuda.stream(self.pool.compute):
            d = t.to(self.pool.device, non_blocking=False)
        return d.view(dtype) if dtype is not None else d

    def stage_events(self, ev_entry, ev_hit):
        """Copies an epoch's events into device memory (padded so the pointers stay valid)."""
        n = int(ev_entry.size)
        e = np.zeros(max(n, 4), np.uint32)
        h = np.zeros(max(n, 16), np.uint8)
        e[:n], h[:n] = ev_entry, ev_hit
        return self.to_device(e.view(np.int32), None), self.to_device(h, None), n

    def admit(self, epoch, key=None, n_free=None):
        n_free = self.pool.kv_get_stats()["n_free"] if n_free is None else n_free
        self.fresh = np.flatnonzero(self.host_array("state") == B.KV_STATE_FREE).astype(np.uint32)
        assert self.fresh.size == n_free
        pairs = self.w.new_pairs(epoch if key is None else key, n_free)
        d_pairs = self.to_device(np.concatenate([pairs, np.zeros(16, np.uint8)]), None)
        rc = self.pool.kv_admit(epoch, self.w.decay, d_pairs, self.fill_pattern)
        self._keep = d_pairs   # the kernel reads it asynchronously
        return rc

    def demote(self, k=None):
        """Demotes the victims of the last selection.  A pool of several partitions needs the
        victims per partition on the host: the selection left them in pinned memory, so the
        caller waits for its own stream here and passes them on (the library itself never
        blocks on this path)."""
        k = self.k if k is None else k
        p = self.pool
        if len(self.w.parts) == 1 or k == 0:
            return p.kv_demote(self.victims, k, self.batch_bytes)
        p.compute.synchronize()
        return p.kv_demote_counted(self.victims, k, p.kv_victim_counts(), self.batch_bytes)

    def promote_lists(self, epoch):
        """Per-partition promote lists for the state the ring is in right now."""
        counts = self.pool.kv_last_demote_counts()
        out = []
        for q, p in enumerate(self.w.parts):
            cur, n_live, live = self.pool.kv_ring_query(q)
            m_q = min(int(self.w.promote_frac * p.n_entries), counts[q], int(n_live))
            out.append(self.w.promote_list(epoch, q, m_q, cur, live, just_written=counts[q]))
        return out

    def step(self, epoch, d_ev_entry, d_ev_hit, n_events, promote_lists=None, admit=True, fused=True):
        """One full epoch.  Returns the promote lists used."""
        p = self.pool
        if fused:
            self.check(p.kv_epoch_score_select(epoch, d_ev_entry, d_ev_hit, n_events, self.k, self.victims),
                       "kv_epoch_score_select")
        else:
            self.check(p.kv_epoch_score(epoch, d_ev_entry, d_ev_hit, n_events), "kv_epoch_score")
            self.check(p.kv_select_victims(self.k, self.victims), "kv_select_victims")
        self.check(self.demote(), "kv_demote")
        if promote_lists is None:
            promote_lists = self.promote_lists(epoch)
        for q, lst in enumerate(promote_lists):
            self.check(p.kv_promote(q, lst, self.batch_bytes), "kv_promote")
        self.check(p.kv_flush(), "kv_flush")
        if admit:
            self.check(self.admit(epoch), "kv_admit")
        return promote_lists

    def host_array(self, name):
        """Copy of a device state array as numpy (synchronises)."""
        self.pool.sync()
        t = getattr(self.pool, name)
        n = {"hits": 16, "misses": 16, "P": 16, "loc": self.pool.n_tags}.get(name, self.pool.N)
        a = t[:n].cpu().numpy()
        if name in ("touch", "last_epoch", "tag", "loc"):
            a = a.view(np.uint32)
        if name in ("hits", "misses"):
            a = a.view(np.uint64)
        return a

    def close(self):
        self.pool.close()
