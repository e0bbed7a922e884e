"""The persistent selection narrows its first histogram to a bracket of 2^22 keys around
the previous selection's tau (moved on by tau's last change) and falls back to the plain
radix select when rank k lies outside.  Whichever path runs, the victims must be the
oracle's: sequences of selections over drifting, jumping, negative and tied scores, and
thresholds placed exactly on and just outside the bracket's edges."""
import numpy as np
import pytest

from oracle import kv_oracle as O
from paper_2604_26968_b200 import workloads as W

pytestmark = pytest.mark.gpu

HALF = 1 << 21          # the bracket reaches this many keys to either side of its centre


def _key_to_float(key):
    """Inverse of the order-preserving key of a binary32 value."""
    key = np.asarray(key, dtype=np.uint64)
    bits = np.where(key & 0x80000000, key & 0x7FFFFFFF, (~key) & 0xFFFFFFFF).astype(np.uint32)
    return bits.view(np.float32)


class Sel:
    def __init__(self, blocks=40000):
        from lockstep import Lockstep
        import torch
        self.torch = torch
        w = W.Workload("bracket", [W.gqa(2, 8, 2, 8, 4, blocks, 64, "entry")], 0.1, 0.0, seed=31)
        self.ls = Lockstep(w, payload=False, batch_bytes=1 << 20)
        self.N = w.N
        self.out = torch.empty(self.N, dtype=torch.int32, device=self.ls.gpu.pool.device)

    def check(self, scores, k, what):
        g, o = self.ls.gpu, self.ls.ora
        scores = np.ascontiguousarray(scores, dtype=np.float32)
        o.score[:] = scores
        g.pool.score[:self.N].copy_(self.torch.from_numpy(scores))
        rc, v = o.select_victims(k)
        assert rc == O.OK
        self.out.fill_(-1)
        g.check(g.pool.kv_select_victims(k, self.out), "kv_select_victims")
        g.pool.sync()
        assert np.array_equal(self.out[:k].cpu().numpy().view(np.uint32), v), what
        assert g.pool.kv_device_status() == 0, what

    def close(self):
        self.ls.close()


def test_drifting_jumping_negative_and_tied_scores():
    s = Sel()
    r = np.random.default_rng(2)
    base = r.uniform(1.0, 2.0, s.N).astype(np.float32)
    k = s.N // 10
    for step in range(6):                                   # +1 % per call: inside the bracket
        s.check(base * np.float32(1.01 ** step), k, "drift up %d" % step)
    s.check(base * np.float32(100.0), k, "jump up")          # far outside: plain radix select
    s.check(base * np.float32(100.0), k, "same again")
    s.check(base * np.float32(1e-6), k, "jump down")
    for step in range(4):                                   # negative scores: keys below 2^31, order inverted
        s.check(-base * np.float32(0.99 ** step), k, "negative drift %d" % step)
    s.check(np.zeros(s.N, np.float32), k, "all equal")
    s.check(np.zeros(s.N, np.float32), s.N // 3, "all equal, other k")
    tied = base.copy()
    tied[r.random(s.N) < 0.5] = np.float32(1.25)             # half the entries tie at what becomes tau
    for kk in (s.N // 4, s.N // 2, s.N // 2 + 17):
        s.check(tied, kk, "heavy ties k=%d" % kk)
        s.check(tied * np.float32(1.0001), kk, "heavy ties moved k=%d" % kk)
    for kk in (1, s.N, 2, s.N - 1):                          # k swings from one end to the other
        s.check(base, kk, "k=%d" % kk)
    s.close()


@pytest.mark.parametrize("offset", [-HALF - 1, -HALF, -HALF + 1, -1, 0, 1, HALF - 2, HALF - 1, HALF, HALF + 1])
def test_threshold_on_and_beside_the_bracket_edges(offset):
    """Two selections with tau = T fix the bracket's centre at T (no trend); the third has its
    k-th key at T + offset: the first and last keys inside the bracket, and their neighbours
    outside, must all give the oracle's victims."""
    s = Sel(blocks=12000)
    r = np.random.default_rng(5)
    k = s.N // 7
    T = 0x80000000 | 0x3FC00000                              # key of 1.5
    perm = r.permutation(s.N)

    def scores_with_tau(t, ties):
        keys = np.empty(s.N, np.int64)
        # ranks 0..N-1 in permuted order: consecutive keys around t, the k-th smallest is t itself
        keys[perm] = t + (np.arange(s.N) - (k - 1)) // (3 if ties else 1)
        return _key_to_float(keys)

    for ties in (False, True):
        s.check(scores_with_tau(T, ties), k, "centre")
        s.check(scores_with_tau(T, ties), k, "centre again")
        s.check(scores_with_tau(T + offset, ties), k, "offset %d ties %s" % (offset, ties))
    s.close()


@pytest.mark.parametrize("kind", ["gqa", "mla"])
def test_entry_and_block_selections_share_the_scratch(kind):
    """A block-granular selection between two entry selections runs over other keys (and, except
    for MLA, whose blocks have one entry each, over another number of them): a hint left by one
    kind of selection must not spoil the other."""
    from lockstep import Lockstep
    part = W.gqa(2, 8, 4, 16, 8, 3000, 4000, "entry") if kind == "gqa" else W.mla(3, 64, 16, 8, 5000, 4000, "entry")
    w = W.Workload("mix", [part], 0.05, 0.02, seed=13, promote_style="recent")
    ls = Lockstep(w, payload=False, batch_bytes=1 << 20, fused=True)
    for e in range(3):
        ls.epoch(e)
    ls.epoch(3, k_blocks=100)
    ls.epoch(4)
    ls.epoch(5, k_blocks=37)
    ls.epoch(6)
    ls.close()
