"""Runs the CUDA library and the CPU oracle side by side on identical inputs and
compares every piece of state after every call."""
import numpy as np

from oracle import kv_oracle as O
from paper_2604_26968_b200 import workloads as W
from paper_2604_26968_b200.harness import EpochRunner, INITIAL_EPOCH_KEY


def oracle_parts(w):
    return [dict(model=O.Model(p.variant, p.n_layers, p.n_q_heads, p.n_kv_heads, p.head_dim,
                               p.d_latent, p.d_rope, p.dtype_bits),
                 block_tokens=p.block_tokens, blocks_per_layer=p.blocks_per_layer,
                 ring_slots=p.ring_slots) for p in w.parts]


def oracle_admit(w, pool, epoch, key=None):
    """Admits into every FREE slot of the oracle pool; payload = pattern(tag).
    Returns the ids admitted (ascending)."""
    fresh = np.flatnonzero(pool.state == O.FREE).astype(np.uint32)
    n_free = int(fresh.size)
    pairs = w.new_pairs(epoch if key is None else key, n_free)
    payload = None
    if pool.payload and n_free:
        imgs, t = [], pool.next_tag
        for q in range(pool.n_parts):
            inf = pool.info(q)
            nf = int((pool.state[inf["base"]:inf["base"] + inf["n"]] == O.FREE).sum())
            imgs.append(W.pattern_bytes(np.arange(t, t + nf), inf["entry_bytes"]).reshape(-1))
            t += nf
        payload = np.concatenate(imgs)
    got = pool.admit(epoch, w.decay, pairs, payload)
    assert got == n_free, got
    return fresh


class Lockstep:
    def __init__(self, w, payload=True, batch_bytes=1 << 20, staging_bytes=None, host_meta=True,
                 policy=0, blend=None, deferred=False, fused=False, heads=None, lazy=False,
                 split_promote=1, counted=False, select_variant=1, l2_budget=None):
        self.w = w
        self.payload = payload
        self.gpu = EpochRunner(w, batch_bytes=batch_bytes, staging_bytes=staging_bytes,
                               fill_pattern=True, host_meta=host_meta)
        self.options = (policy, blend)
        self.deferred = deferred
        self.fused = fused   # score and select through the single fused call
        self.split_promote = split_promote   # each partition's promote list goes in this many calls
        self.counted = counted   # pools of several partitions: demote with the counts the selection left
        # heads = (decay, every): importance matrices of all partitions updated before every
        # epoch's scoring, multipliers set on epochs divisible by `every` and reset on the next
        self.heads = heads
        if deferred:
            assert self.gpu.pool.kv_set_deferred_packing(True) == 0
        assert self.gpu.pool.kv_set_select_variant(select_variant) == 0
        if l2_budget is not None:   # one state array kept in the persisting part of the L2
            assert self.gpu.pool.kv_set_l2_residency(l2_budget) == 0
        # room for any k a test may ask for
        self.gpu.victims = self.gpu.torch.empty(max(w.N, 4), dtype=self.gpu.torch.int32,
                                                device=self.gpu.pool.device)
        self.ora = O.OraclePool(oracle_parts(w), w.alpha0, w.beta0, n_tags=w.n_tags, payload=payload)
        self.fresh = oracle_admit(w, self.ora, 0, key=INITIAL_EPOCH_KEY)
        assert np.array_equal(self.fresh, self.gpu.fresh)
        assert self.ora.set_policy(policy) == O.OK and self.gpu.pool.kv_set_policy(policy) == 0
        if blend is not None:
            assert self.ora.set_confidence_blend(*blend) == O.OK
            assert self.gpu.pool.kv_set_confidence_blend(*blend) == 0
        if lazy:   # promoted entries catch up on the EMA steps they missed on the host
            assert self.ora.set_lazy_decay(True) == O.OK and self.gpu.pool.kv_set_lazy_decay(True) == 0
        self.compare_state("initial fill")
        if payload:
            self.compare_payload("initial fill")

    # ---- comparisons (bit-exact everywhere) --------------------------------
    def compare_state(self, where, scores=True):
        g, o = self.gpu, self.ora
        st = g.host_array("state")
        assert np.array_equal(st, o.state), where
        res = o.state == O.RESIDENT
        for name in ("pair", "decay", "ema", "last_epoch", "tag", "touch"):
            a, b = g.host_array(name), getattr(o, name)
            if name == "tag":
                assert np.array_equal(a, b), (where, name)
            else:   # arrays of FREE slots are don't-care on both sides
                assert np.array_equal(a[res].view(np.uint32 if a.dtype.itemsize == 4 else a.dtype),
                                      b[res].view(np.uint32 if b.dtype.itemsize == 4 else b.dtype)), (where, name)
        if scores:
            assert np.array_equal(g.host_array("score").view(np.uint32), o.score.view(np.uint32)), where
        assert np.array_equal(g.host_array("hits"), o.hits), where
        assert np.array_equal(g.host_array("misses"), o.misses), where
        assert np.array_equal(g.host_array("P").view(np.uint32), o.P.view(np.uint32)), where
        g.pool.sync()
        est = g.pool.kv_reuse_estimate().cpu().numpy()
        assert np.array_equal(est.view(np.uint32), o.estimate.view(np.uint32)), where
        assert np.array_equal(g.host_array("loc"), o.loc), where
        assert g.pool.kv_device_status() == 0, where

    def compare_ring(self, where):
        g, o = self.gpu, self.ora
        g.pool.sync()
        for q, p in enumerate(self.w.parts):
            cur, n_live, live = g.pool.kv_ring_query(q)
            o_live = o.part_array(q, "r_live")
            assert cur == o.info(q)["cursor"], where
            assert np.array_equal(live, o_live), where
            assert n_live == int(o_live.sum())
            meta = g.pool.ring_meta(q)
            lv = o_live != 0
            # the mirror keeps the record of the last demotion into a slot; compare where the
            # oracle still holds that block (a promoted slot is dead and its record stale)
            for name in ("tag", "pair", "last_epoch"):
                assert np.array_equal(meta[name.replace("r_", "")][lv].astype(np.uint32),
                                      o.part_array(q, "r_" + name)[lv].astype(np.uint32)), (where, name)
            assert np.array_equal(meta["demote_epoch"][lv], o.part_array(q, "r_depoch")[lv]), (where, "demote_epoch")
            for name in ("ema", "decay"):
                assert np.array_equal(meta[name][lv].view(np.uint32),
                                      o.part_array(q, "r_" + name)[lv].view(np.uint32)), (where, name)
            if self.payload:
                ring = g.pool.rings[q].numpy()[: p.ring_slots * p.entry_bytes].reshape(p.ring_slots, p.entry_bytes)
                oring = o.part_array(q, "ring").reshape(p.ring_slots, p.entry_bytes)
                assert np.array_equal(ring[lv], oring[lv]), where

    def compare_payload(self, where):
        g, o = self.gpu, self.ora
        g.pool.sync()
        for q in range(len(self.w.parts)):
            slab = g.pool.slabs[q].cpu().numpy()
            oslab = o.part_array(q, "slab")
            inf = o.info(q)
            # bytes of FREE slots are don't-care: compare resident entries only
            res = o.state[inf["base"]:inf["base"] + inf["n"]] == O.RESIDENT
            H, cb, nc = inf["H"], inf["chunk_bytes"], inf["n_chunks"]
            lb = inf["n"] // H
            a = slab.reshape(lb, nc, H, cb)
            b = oslab.reshape(lb, nc, H, cb)
            mask = res.reshape(lb, H)
            for c in range(nc):
                assert np.array_equal(a[:, c][mask], b[:, c][mask]), (where, q, c)

    def head_step(self, e):
        w, g, o = self.w, self.gpu, self.ora
        decay, every = self.heads
        keep = []
        for q in range(len(w.parts)):
            x = w.head_observations(e, q)
            assert o.head_importance_update(q, x, decay) == O.OK
            d_x = g.to_device(x.reshape(-1), None)
            keep.append(d_x)
            g.check(g.pool.kv_head_importance_update(q, d_x, decay), "kv_head_importance_update")
            if e % every == 0:
                m = w.head_multipliers(e, q)
                assert o.set_head_multipliers(q, m) == O.OK
                d_m = g.to_device(m.reshape(-1), None)
                keep.append(d_m)
                g.check(g.pool.kv_set_head_multipliers(q, d_m), "kv_set_head_multipliers")
            elif e % every == 1:
                assert o.set_head_multipliers(q, None) == O.OK
                g.check(g.pool.kv_set_head_multipliers(q, None), "kv_set_head_multipliers")
        g.pool.sync()
        for q in range(len(w.parts)):
            assert np.array_equal(g.pool.kv_head_importance(q).cpu().numpy().view(np.uint32),
                                  o.head_array(q, "importance").view(np.uint32)), ("importance", e, q)
            assert np.array_equal(g.pool.kv_head_weights(q).cpu().numpy().view(np.uint32),
                                  o.head_array(q, "weights").view(np.uint32)), ("weights", e, q)

    # ---- one epoch -----------------------------------------------------------
    def epoch(self, e, k=None, check_payload=None, k_blocks=None, before_demote=None, promote_with=None):
        """One epoch on both sides.  k_blocks selects whole paged blocks instead of k entries.
        before_demote(self) runs once the victims agree; promote_with(self) returns the
        per-partition promote lists to use in place of the workload's."""
        w, g, o = self.w, self.gpu, self.ora
        k = w.k if k is None else k
        ev_entry, ev_hit = w.events(e, o.pair, self.fresh)
        d_e, d_h, n = g.stage_events(ev_entry, ev_hit)
        if self.heads is not None:
            self.head_step(e)
        assert o.epoch_score(e, ev_entry, ev_hit) == O.OK
        fused = self.fused and k_blocks is None
        if fused:
            g.check(g.pool.kv_epoch_score_select(e, d_e, d_h, n, k, g.victims), "kv_epoch_score_select")
        else:
            g.check(g.pool.kv_epoch_score(e, d_e, d_h, n), "kv_epoch_score")
        self.compare_state("epoch %d score" % e)
        if k_blocks is None:
            rc, v = o.select_victims(k)
            assert rc == O.OK
            if not fused:
                g.check(g.pool.kv_select_victims(k, g.victims), "kv_select_victims")
        else:
            rc, v = o.select_victim_blocks(k_blocks)
            assert rc == O.OK
            if self.counted:      # no place for the count: the call must not block
                rc, _ = g.pool.kv_select_victim_blocks(k_blocks, g.victims, wait=False)
                g.check(rc, "kv_select_victim_blocks")
                g.pool.sync()
                per_part = g.pool.kv_victim_counts() if len(w.parts) > 1 else [len(v)]
                k = sum(per_part)
            else:
                rc, k = g.pool.kv_select_victim_blocks(k_blocks, g.victims)
                g.check(rc, "kv_select_victim_blocks")
            assert k == len(v), (k, len(v))
        g.pool.sync()
        got = g.victims[:k].cpu().numpy().view(np.uint32)
        assert np.array_equal(got, v), "epoch %d victims" % e
        if before_demote is not None:
            before_demote(self)
        assert o.demote(v) == O.OK
        if self.counted and len(w.parts) > 1:
            # the counts the selection left in pinned memory (the stream has been synchronised above)
            counts = g.pool.kv_victim_counts()
            inf = [o.info(q) for q in range(len(w.parts))]
            assert counts == [int(((v >= i["base"]) & (v < i["base"] + i["n"])).sum()) for i in inf], counts
            g.check(g.pool.kv_demote_counted(g.victims, k, counts, g.batch_bytes), "kv_demote_counted")
        else:
            g.check(g.pool.kv_demote(g.victims, k, g.batch_bytes), "kv_demote")
        if not self.deferred:   # (a status read would enqueue the deferred chunks and undo the interleaving)
            self.compare_state("epoch %d demote" % e, scores=False)
            self.compare_ring("epoch %d demote" % e)
        lists = g.promote_lists(e) if promote_with is None else promote_with(self)
        for q, lst in enumerate(lists):
            pieces = np.array_split(lst, self.split_promote) if self.split_promote > 1 else [lst]
            for piece in pieces:
                assert o.promote(q, piece) == O.OK
                g.check(g.pool.kv_promote(q, piece, g.batch_bytes), "kv_promote")
        self.compare_state("epoch %d promote" % e, scores=False)
        self.compare_ring("epoch %d promote" % e)
        self.fresh = oracle_admit(w, o, e)
        n_free = int(self.fresh.size)
        g.check(g.admit(e, n_free=n_free), "kv_admit")
        assert np.array_equal(self.fresh, g.fresh)
        self.compare_state("epoch %d admit" % e, scores=False)
        if self.payload and (check_payload is None or check_payload):
            self.compare_payload("epoch %d" % e)
        so, sg = o.stats(), g.pool.kv_get_stats()
        for name in ("epochs", "events", "victims", "promoted", "bytes_demoted", "bytes_promoted",
                     "bytes_dropped"):
            assert so[name] == sg[name], (name, so[name], sg[name])
        return dict(events=n, promoted=sum(len(x) for x in lists), admitted=n_free)

    def close(self):
        self.gpu.close()
        self.ora.close()


def sample_payload(ls, n=256, seed=0):
    """Checks sampled blocks of a (large) pool against the byte pattern of the tag the
    oracle says lives there: n resident HBM entries and n live ring slots per partition."""
    import torch
    g, o, w = ls.gpu, ls.ora, ls.w
    g.pool.sync()
    r = np.random.default_rng(seed)
    for q, p in enumerate(w.parts):
        inf = o.info(q)
        H, cb, nc, eb = inf["H"], inf["chunk_bytes"], inf["n_chunks"], inf["entry_bytes"]
        ids = np.flatnonzero(o.state[inf["base"]:inf["base"] + inf["n"]] == O.RESIDENT)
        ids = r.choice(ids, size=min(n, ids.size), replace=False)
        slab = g.pool.slabs[q]
        for local in ids:
            tag = int(o.tag[inf["base"] + local])
            lb, head = divmod(int(local), H)
            pieces = []
            for c in range(nc):
                off = ((lb * nc + c) * H + head) * cb
                pieces.append(slab[off:off + cb])
            got = torch.cat(pieces).cpu().numpy()
            assert np.array_equal(got, W.pattern_bytes([tag], eb)[0]), (q, int(local), tag)
        live = np.flatnonzero(o.part_array(q, "r_live"))
        if live.size:
            slots = r.choice(live, size=min(n, live.size), replace=False)
            ring = g.pool.rings[q].numpy()
            rt = o.part_array(q, "r_tag")
            for s in slots:
                got = ring[int(s) * eb:(int(s) + 1) * eb]
                assert np.array_equal(got, W.pattern_bytes([int(rt[s])], eb)[0]), (q, int(s))
