"""Per-layer prefetch window and prefetch list (RoPE-aware prefetching section): CUDA
library against the CPU oracle through the C ABI -- spans bit for bit, windows and
lists exactly -- and the lists fed to kv_promote on both sides."""
import numpy as np
import pytest

from oracle import kv_oracle as O
from paper_2604_26968_b200 import binding as B
from paper_2604_26968_b200 import workloads as W

pytestmark = pytest.mark.gpu


class Prefetch:
    """Both sides' prefetch calls for one partition of a Lockstep pair."""

    def __init__(self, ls, q):
        self.ls, self.q = ls, q
        p = ls.w.parts[q]
        self.L, self.H, self.NB = p.n_layers, p.heads, p.blocks_per_layer
        self.table = None

    def update(self, span, decay):
        g, o = self.ls.gpu, self.ls.ora
        assert o.prefetch_window_update(self.q, span, decay) == O.OK
        g.check(g.pool.kv_prefetch_window_update(self.q, g.to_device(np.asarray(span, np.float32), None), decay),
                "kv_prefetch_window_update")
        self.compare_windows()

    def set(self, tokens, cap):
        g, o = self.ls.gpu, self.ls.ora
        assert o.set_prefetch_window(self.q, tokens, cap) == O.OK
        g.check(g.pool.kv_set_prefetch_window(self.q, tokens, cap), "kv_set_prefetch_window")
        self.compare_windows()

    def compare_windows(self):
        g, o = self.ls.gpu, self.ls.ora
        g.pool.sync()
        span = g.pool.kv_prefetch_span(self.q).cpu().numpy()
        win = g.pool.kv_prefetch_window(self.q).cpu().numpy().view(np.uint32)
        assert np.array_equal(span.view(np.uint32), o.prefetch_array(self.q, "span").view(np.uint32))
        assert np.array_equal(win, o.prefetch_array(self.q, "window"))

    def build_table(self, n_pos, seed):
        """A sequence made of n_pos of the partition's paged blocks, in random order, every
        (layer, head) of a block at the same position; handles as they are right now."""
        o = self.ls.ora
        inf = o.info(self.q)
        tag = o.tag[inf["base"]:inf["base"] + inf["n"]].reshape(self.L, self.NB, self.H)
        r = np.random.default_rng(seed)
        blocks = r.permutation(self.NB)[:n_pos]
        self.table = np.ascontiguousarray(tag[:, blocks, :].transpose(1, 0, 2)).copy()
        # handles that name nothing: never admitted, and beyond the handle space
        for bad in (0xFFFFFFFF, self.ls.w.n_tags + 7):
            self.table[r.integers(0, n_pos), r.integers(0, self.L), r.integers(0, self.H)] = bad
        return self.table

    def lists(self, pos0, direction, max_out=None):
        g, o, t = self.ls.gpu, self.ls.ora, self.table
        torch = g.torch
        rc, want, n_want = o.prefetch_list(self.q, t, pos0, direction, max_out=max_out)
        assert rc == O.OK
        cap = t.size if max_out is None else max_out
        d_t = g.to_device(t.reshape(-1).view(np.int32), None)
        d_out = torch.full((max(cap, 1),), -1, dtype=torch.int64, device=g.pool.device)
        d_n = torch.full((1,), -1, dtype=torch.int64, device=g.pool.device)
        g.check(g.pool.kv_prefetch_list(self.q, d_t, t.shape[0], pos0, direction, d_out, cap, d_n),
                "kv_prefetch_list")
        g.pool.sync()
        n = int(d_n.item())
        got = d_out.cpu().numpy().view(np.uint64)
        assert n == n_want, (n, n_want)
        assert np.array_equal(got[:min(n, cap)], want)
        assert np.all(got[min(n, cap):] == np.uint64(0xFFFFFFFFFFFFFFFF))      # nothing written past the list
        return want, n


def _run(w, q, spans, n_pos, epochs=5, payload=True, fused=False, cap=None, batch=1 << 20, deferred=False):
    from lockstep import Lockstep
    ls = Lockstep(w, payload=payload, batch_bytes=batch, fused=fused, deferred=deferred)
    pf = Prefetch(ls, q)
    r = np.random.default_rng(3)
    promoted = 0
    limit = ls.gpu.max_promote(w)
    for e in range(epochs):
        pf.update((r.random(pf.L) * spans).astype(np.float32), 0.5)
        if cap is not None and e == 2:
            pf.set(float(spans), cap)

        def before(ls_, e=e):
            pf.build_table(n_pos, 100 + e)

        def promote(ls_, e=e):
            out = [np.zeros(0, np.uint64) for _ in w.parts]
            for pos0 in (0, n_pos // 3, n_pos - 1):
                for direction in (1, -1):
                    pf.lists(pos0, direction)
            pf.lists(n_pos // 2, 1, max_out=5)           # a cut list
            lst, n = pf.lists(e % n_pos, 1 if e % 2 == 0 else -1)
            inf = ls_.ora.info(q)
            free = int((ls_.ora.state[inf["base"]:inf["base"] + inf["n"]] == 0).sum())   # FREE
            out[q] = lst[:min(limit, free)]
            return out

        st = ls.epoch(e, before_demote=before, promote_with=promote)
        promoted += st["promoted"]
    g = ls.gpu
    assert g.pool.kv_device_status() == 0
    ls.close()
    return promoted


def test_prefetch_config1_windows_lists_and_promotion():
    w = W.config(1)          # 2 layers x 4 KV heads, 512 blocks of 16 tokens
    assert _run(w, 0, spans=600.0, n_pos=96, epochs=6) > 0


def test_prefetch_deferred_packing_and_fused_selection():
    w = W.config(1)
    assert _run(w, 0, spans=900.0, n_pos=200, epochs=5, fused=True, deferred=True) > 0


def test_prefetch_mla_single_column():
    w = W.config(4, scale=1 / 128)      # 61 layers, one column per layer, 64-token blocks
    assert _run(w, 0, spans=3000.0, n_pos=100, epochs=4, payload=False, cap=9) > 0


def test_prefetch_second_partition_of_the_mixed_pool_many_chunks():
    """80 layers x 8 heads x 84 blocks: 53,760 candidates, several chunks and a ragged tail."""
    w = W.config(5, scale=1 / 128)
    for p in w.parts:
        p.ring_slots = w.k + 64
    assert _run(w, 1, spans=2000.0, n_pos=84, epochs=3, payload=False, fused=True, batch=4 << 20) > 0


def test_prefetch_errors_and_edges():
    from lockstep import Lockstep
    w = W.config(1)
    ls = Lockstep(w, payload=False, batch_bytes=1 << 20)
    g, o = ls.gpu, ls.ora
    torch = g.torch
    pf = Prefetch(ls, 0)
    pf.compare_windows()                                  # the defaults: 2,048 tokens = 128 blocks
    assert np.array_equal(o.prefetch_array(0, "window"), np.full(2, 128, np.uint32))
    ls.epoch(0, before_demote=lambda l: pf.build_table(64, 1))
    x = g.to_device(np.ones(2, np.float32), None)
    d_n = torch.zeros(1, dtype=torch.int64, device=g.pool.device)
    d_out = torch.zeros(16, dtype=torch.int64, device=g.pool.device)
    d_t = g.to_device(pf.table.reshape(-1).view(np.int32), None)
    P = g.pool
    assert P.kv_prefetch_window_update(1, x, 0.5) == B.KV_ERR_INVALID_ARG
    assert P.kv_prefetch_window_update(0, None, 0.5) == B.KV_ERR_INVALID_ARG
    assert P.kv_prefetch_window_update(0, x, 1.5) == B.KV_ERR_INVALID_ARG
    assert P.kv_prefetch_window_update(0, x, float("nan")) == B.KV_ERR_INVALID_ARG
    assert P.kv_set_prefetch_window(0, -1.0, 4) == B.KV_ERR_INVALID_ARG
    assert P.kv_set_prefetch_window(0, float("inf"), 4) == B.KV_ERR_INVALID_ARG
    assert P.kv_set_prefetch_window(0, 8.0, 0) == B.KV_ERR_INVALID_ARG
    assert P.kv_prefetch_list(0, d_t, 64, 64, 1, d_out, 16, d_n) == B.KV_ERR_INVALID_ARG
    assert P.kv_prefetch_list(0, d_t, 64, 0, 0, d_out, 16, d_n) == B.KV_ERR_INVALID_ARG
    assert P.kv_prefetch_list(0, None, 64, 0, 1, d_out, 16, d_n) == B.KV_ERR_INVALID_ARG
    assert P.kv_prefetch_list(0, d_t, 64, 0, 1, None, 16, d_n) == B.KV_ERR_INVALID_ARG
    assert P.kv_prefetch_list(0, d_t, 64, 0, 1, d_out, 16, None) == B.KV_ERR_INVALID_ARG
    assert P.kv_prefetch_list(4, d_t, 64, 0, 1, d_out, 16, d_n) == B.KV_ERR_INVALID_ARG
    pf.compare_windows()                                  # none of them changed anything
    # an empty table: count 0, nothing written; counting only (no output array)
    d_n.fill_(-1)
    g.check(P.kv_prefetch_list(0, None, 0, 0, 1, d_out, 16, d_n), "kv_prefetch_list")
    P.sync()
    assert int(d_n.item()) == 0 and int(d_out.abs().sum().item()) == 0
    rc, _, n_want = o.prefetch_list(0, pf.table, 0, 1)
    g.check(P.kv_prefetch_list(0, d_t, 64, 0, 1, None, 0, d_n), "kv_prefetch_list")
    P.sync()
    assert rc == O.OK and int(d_n.item()) == n_want
    # a bad observation: the device flags it and keeps every span, as the oracle refuses the call
    bad = np.array([5.0, -2.0], np.float32)
    assert o.prefetch_window_update(0, bad, 0.5) == O.ERR_INVALID_ARG
    g.check(P.kv_prefetch_window_update(0, g.to_device(bad, None), 0.5), "kv_prefetch_window_update")
    pf.compare_windows()
    assert P.kv_device_status() == B.KV_DEV_BAD_SPAN_VALUE
    # windows wider than the table, and the narrowest one
    for tokens, cap in ((1e9, 1 << 20), (0.0, 1), (3.4e38, 0xFFFFFFFF)):
        pf.set(tokens, cap)
        for pos0 in (0, 63):
            pf.lists(pos0, 1)
            pf.lists(pos0, -1)
    ls.close()


def test_prefetch_list_at_the_launch_limit():
    """1.3 M candidates (2,048 position-blocks x 80 layers x 8 heads, the sequence's table tiled
    from the partition's 84 blocks): the list kernels run their full 1,024 chunks of more than
    one tile each; windows from 1 block to the whole table, both directions, a cut list."""
    from lockstep import Lockstep
    w = W.config(5, scale=1 / 128)
    for p in w.parts:
        p.ring_slots = w.k + 64
    ls = Lockstep(w, payload=False, batch_bytes=4 << 20, fused=True)
    pf = Prefetch(ls, 1)
    state = {}

    def before(ls_):
        t = pf.build_table(pf.NB, 7)
        state["table"] = np.ascontiguousarray(np.tile(t, (25, 1, 1))[:2048])

    ls.epoch(0, before_demote=before)
    ls.epoch(1)
    pf.table = state["table"]
    r = np.random.default_rng(9)
    span = (r.random(pf.L) * 16 * 2048).astype(np.float32)
    span[0], span[-1] = 1.0, 16.0 * 4096
    pf.set(0.0, 4096)
    pf.update(span, 0.0)
    for pos0, direction in ((0, 1), (2047, -1), (1000, 1), (1000, -1)):
        lst, n = pf.lists(pos0, direction)
        assert n > 10000
    pf.lists(5, 1, max_out=1000)
    assert ls.gpu.pool.kv_device_status() == 0
    ls.close()
