"""Seeded synthetic pools and access traces.

This module only *draws inputs*: pool geometries, per-epoch access events,
pair ids of newly admitted blocks, promotion lists and the byte pattern that
fills a block.  It holds none of the method's arithmetic (no EMA, posterior,
score, selection or slot assignment) and is used by the tests, the benchmark
and the smoke check to feed the CUDA library and, in tests, the CPU oracle with
identical arrays.

The paper evaluates on ShareGPT, LMSYS-Chat-1M and a synthetic agentic
simulator (its "Workloads" paragraph); none of those is available offline, so
traces with the same shape stand in: Zipf-distributed shared-prefix reuse and
log-normal prompt lengths for chat, sliding windows for long context, growing
session prefixes that are re-read for agentic sessions.
"""
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

AUTO, MHA, GQA, MQA, MLA = -1, 0, 1, 2, 3


@dataclass
class Partition:
    """One model's paged slab inside a pool (plain integers only)."""
    variant: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_latent: int
    d_rope: int
    dtype_bits: int
    block_tokens: int
    blocks_per_layer: int
    ring_slots: int
    style: str = "chat"   # which trace generator touches this partition

    @property
    def heads(self) -> int:
        if self.variant == MLA:
            return 1
        return self.n_q_heads if self.variant == MHA else self.n_kv_heads

    @property
    def elems_per_token(self) -> int:
        if self.variant == MLA:
            return self.d_latent + self.d_rope
        return 2 * self.heads * self.head_dim

    @property
    def entry_bytes(self) -> int:
        return self.elems_per_token * self.block_tokens * self.dtype_bits // 8 // self.heads

    @property
    def n_entries(self) -> int:
        return self.n_layers * self.blocks_per_layer * self.heads

    @property
    def slab_bytes(self) -> int:
        return self.n_entries * self.entry_bytes


def gqa(layers, q_heads, kv_heads, head_dim, block_tokens, blocks, ring, style="chat"):
    return Partition(GQA, layers, q_heads, kv_heads, head_dim, 0, 0, 16, block_tokens, blocks,
                     ring, style)


def mha(layers, heads, head_dim, block_tokens, blocks, ring, style="chat"):
    return Partition(MHA, layers, heads, heads, head_dim, 0, 0, 16, block_tokens, blocks, ring,
                     style)


def mqa(layers, q_heads, head_dim, block_tokens, blocks, ring, style="chat"):
    return Partition(MQA, layers, q_heads, 1, head_dim, 0, 0, 16, block_tokens, blocks, ring,
                     style)


def mla(layers, d_latent, d_rope, block_tokens, blocks, ring, style="agentic"):
    return Partition(MLA, layers, 128, 128, 128, d_latent, d_rope, 16, block_tokens, blocks,
                     ring, style)


@dataclass
class Workload:
    name: str
    parts: List[Partition]
    evict_frac: float
    promote_frac: float
    seed: int
    decay: float = 0.9
    alpha0: float = 1.0
    beta0: float = 1.0
    epochs: int = 50
    pair_weights: Optional[np.ndarray] = None   # None = uniform over the 16 pairs
    promote_style: str = "runs"                 # "recent", "runs", "position" or "aligned-runs"
    max_run: int = 2048
    _static: dict = field(default_factory=dict, repr=False)

    @property
    def N(self) -> int:
        return sum(p.n_entries for p in self.parts)

    @property
    def k(self) -> int:
        return int(self.evict_frac * self.N)

    @property
    def m(self) -> int:
        return int(self.promote_frac * self.N)

    def bases(self):
        out, b = [], 0
        for p in self.parts:
            out.append(b)
            b += p.n_entries
        return out

    @property
    def n_tags(self) -> int:
        """Upper bound on the logical block handles ever issued."""
        return self.N + (self.epochs + 2) * max(self.k, 1) + 16

    # ---- inputs -----------------------------------------------------------
    def rng(self, epoch: int, stream: int) -> np.random.Generator:
        return np.random.default_rng([self.seed, epoch, stream])

    def new_pairs(self, epoch: int, n: int) -> np.ndarray:
        """Pair ids (0..15) for the n blocks admitted in this epoch."""
        r = self.rng(epoch, 1)
        if self.pair_weights is None:
            return r.integers(0, 16, size=n, dtype=np.uint8)
        return r.choice(16, size=n, p=self.pair_weights).astype(np.uint8)

    def head_observations(self, epoch: int, q: int) -> np.ndarray:
        """Per-(layer, query head) observations of one epoch for partition q, float32
        [layers][query heads] ([layers][1] for MLA): a fixed per-head profile (a few
        heads matter much more than the rest, later layers more than early ones)
        times log-normal noise."""
        p = self.parts[q]
        qh = 1 if p.variant == MLA else p.n_q_heads
        prof = np.random.default_rng([self.seed, 77, q]).lognormal(0.0, 1.0, size=(p.n_layers, qh))
        prof *= np.linspace(0.5, 1.5, p.n_layers)[:, None]
        noise = self.rng(epoch, 7 + 16 * q).lognormal(0.0, 0.25, size=(p.n_layers, qh))
        return (prof * noise).astype(np.float32)

    def head_multipliers(self, epoch: int, q: int) -> np.ndarray:
        """Task-transition multipliers for partition q, float32 [layers][KV heads] in
        {0.5, 1, 2}."""
        p = self.parts[q]
        r = self.rng(epoch, 8 + 16 * q)
        return r.choice(np.array([0.5, 1.0, 2.0], np.float32), size=(p.n_layers, p.heads)).astype(np.float32)

    def events(self, epoch: int, pair: np.ndarray, fresh: Optional[np.ndarray] = None):
        """(ev_entry u32[E], ev_hit u8[E]) of one epoch.

        pair is the current per-entry pair-id array: the hit flag of a touch is
        Bernoulli(q[pair]) with q[p] = (p + 0.5) / 16, which gives each of the
        16 posteriors a known limit.  fresh lists the entries admitted at the end
        of the previous epoch: a block that had to be brought in was a cache miss
        and is being used, so each contributes one touch with a miss flag.
        """
        r = self.rng(epoch, 2)
        chunks = []
        for q, (p, base) in enumerate(zip(self.parts, self.bases())):
            style = p.style
            if style == "mixed":
                style = "chat" if r.random() < 0.5 else "agentic"
            gen = _STYLES[style]
            ids = gen(self, q, p, epoch, r)
            chunks.append(ids.astype(np.int64) + base)
        ids = np.concatenate(chunks) if chunks else np.zeros(0, np.int64)
        ev_entry = ids.astype(np.uint32)
        qhit = (pair[ev_entry].astype(np.float64) + 0.5) / 16.0
        ev_hit = (r.random(ev_entry.size) < qhit).astype(np.uint8)
        if fresh is not None and len(fresh):
            ev_entry = np.concatenate([ev_entry, np.asarray(fresh, dtype=np.uint32)])
            ev_hit = np.concatenate([ev_hit, np.zeros(len(fresh), np.uint8)])
        return ev_entry, ev_hit

    def promote_list(self, epoch: int, q: int, m: int, cursor: int, live: np.ndarray,
                     just_written: int = 0) -> np.ndarray:
        """Host ring slots (u64) to promote into partition q; all live, distinct.

        just_written is the number of slots, ending at the cursor, that this epoch's
        demotion wrote: a prefetcher does not ask back what was evicted a moment ago,
        so the "runs" style leaves them out when enough older slots are live."""
        m = int(min(m, int(live.sum())))
        if m <= 0:
            return np.zeros(0, np.uint64)
        R = live.size
        if self.promote_style != "recent" and just_written > 0:
            idx = (cursor - 1 - np.arange(min(just_written, R))) % R
            if int(live.sum()) - int(live[idx].sum()) >= m:
                live = live.copy()
                live[idx] = 0
        if self.promote_style == "position":
            return self._position_list(epoch, q, m, cursor, live, just_written)
        if self.promote_style == "recent":
            # the m most recently written live slots, oldest first
            order = (cursor - 1 - np.arange(R)) % R
            picked = order[live[order] != 0][:m]
            return picked[::-1].astype(np.uint64)
        if self.promote_style == "aligned-runs":
            return self._aligned_runs(epoch, q, m, live)
        r = self.rng(epoch, 3 + q)
        taken = np.zeros(R, dtype=bool)
        out = []
        n = 0
        live_idx = np.flatnonzero(live)
        guard = 0
        while n < m and guard < 64 * (m // max(self.max_run, 1) + 4):
            guard += 1
            s = int(live_idx[r.integers(0, live_idx.size)])
            e = min(R, s + min(self.max_run, m - n))
            seg = np.arange(s, e)
            ok = (live[seg] != 0) & ~taken[seg]
            if not ok[0]:
                continue
            stop = int(np.argmin(ok)) if not ok.all() else seg.size
            seg = seg[:stop]
            taken[seg] = True
            out.append(seg)
            n += seg.size
        if n < m:   # top up deterministically
            rest = np.flatnonzero((live != 0) & ~taken)[: m - n]
            out.append(rest)
        return np.concatenate(out)[:m].astype(np.uint64)


def _position_list(self, epoch, q, m, cursor, live, just_written):
    """Position-ordered prefetch (long-context pool): round-robin over 64 sequences, for each
    the next window of 128 blocks, ordered by (position, layer, head).  A demotion fills
    the ring in (layer, block, head) order, so the part of the ring older than this
    epoch's demotion is read as n_layers stripes of equal length in which a block's heads
    are neighbours and its layers lie one stripe apart: the list comes out as runs of
    `heads` slots, a stripe apart -- the fragmented case of kv_promote."""
    p = self.parts[q]
    L, H, R = p.n_layers, p.heads, live.size
    seg_len = R - min(just_written, R)
    per_layer = seg_len // L // H * H
    n_blocks = per_layer // H
    if n_blocks == 0:
        return np.flatnonzero(live)[:m].astype(np.uint64)
    n_seq, win = 64, 128
    bps = max(1, n_blocks // n_seq)                     # blocks of one sequence's stripe
    n_win = -(-bps // win)
    lh = (np.arange(L, dtype=np.int64)[:, None] * per_layer + np.arange(H, dtype=np.int64)[None, :]).reshape(-1)
    out, n = [], 0
    for wi in range(n_win):
        w0 = ((epoch + wi) % n_win) * win
        blocks = (np.arange(n_seq, dtype=np.int64)[:, None] * bps
                  + (w0 + np.arange(win, dtype=np.int64))[None, :] % bps).reshape(-1)
        blocks = blocks[blocks < n_blocks]
        slots = (cursor + blocks[:, None] * H + lh[None, :]).reshape(-1) % R
        slots = slots[live[slots] != 0]
        out.append(slots)
        n += slots.size
        if n >= m:
            break
    lst = np.concatenate(out) if out else np.zeros(0, np.int64)
    _, first = np.unique(lst, return_index=True)          # (windows of short stripes can overlap)
    lst = lst[np.sort(first)][:m]
    if lst.size < m:      # a ring still filling up: the rest from whatever else is live, oldest first
        taken = np.zeros(R, dtype=bool)
        taken[lst] = True
        order = (cursor + np.arange(R, dtype=np.int64)) % R
        rest = order[(live[order] != 0) & ~taken[order]][: m - lst.size]
        lst = np.concatenate([lst, rest])
    return lst.astype(np.uint64)


def _aligned_runs(self, epoch, q, m, live):
    """Runs of exactly max_run consecutive live slots at seeded places: the ring is cut into
    rows of max_run slots, every second row is a candidate (so that two chosen runs never
    touch), and a seeded shuffle of the fully live candidates gives the list.  For timing
    kv_promote against the run length; built without a Python loop per run."""
    run, R = int(self.max_run), live.size
    rows = R // run
    full = (live[:rows * run].reshape(rows, run) != 0).all(axis=1)
    cand = np.flatnonzero(full[::2]) * 2
    self.rng(epoch, 3 + q).shuffle(cand)
    cand = cand[: -(-m // run)]
    lst = (cand[:, None].astype(np.int64) * run + np.arange(run, dtype=np.int64)[None, :]).reshape(-1)[:m]
    return lst.astype(np.uint64)


Workload._position_list = _position_list
Workload._aligned_runs = _aligned_runs


# ---- trace styles (each returns local entry ids of one partition) ----------

def zipf_bounded(r: np.random.Generator, s: float, n: int, size: int) -> np.ndarray:
    """Ranks 0..n-1 with P(rank) proportional to (rank+1)^-s (inverse CDF)."""
    w = np.arange(1, n + 1, dtype=np.float64) ** (-s)
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    return np.minimum(np.searchsorted(cdf, r.random(size)), n - 1)


def lognormal_tokens(r, median, sigma, cap, size):
    t = np.exp(np.log(median) + sigma * r.standard_normal(size))
    return np.clip(np.ceil(t), 1, cap).astype(np.int64)


def block_events(p: Partition, blocks: np.ndarray) -> np.ndarray:
    """One event for every (layer, head) of each listed block ("block mode")."""
    blocks = np.asarray(blocks, dtype=np.int64)
    if blocks.size == 0:
        return np.zeros(0, np.int64)
    H, NB, L = p.heads, p.blocks_per_layer, p.n_layers
    lh = (np.arange(L, dtype=np.int64)[:, None] * NB * H + np.arange(H, dtype=np.int64)[None, :])
    return (blocks[:, None, None] * H + lh[None, :, :]).reshape(-1)


def _perm(w: Workload, q: int, n: int) -> np.ndarray:
    key = ("perm", q, n)
    if key not in w._static:
        w._static[key] = np.random.default_rng([w.seed, 1000 + q]).permutation(n)
    return w._static[key]


def _entry_mode(w, q, p, epoch, r):
    """Tiny pool: independent touches, block ~ Zipf(1.1), layer/head uniform."""
    n_draws = int(0.2 * p.n_entries)
    rank = zipf_bounded(r, 1.1, p.blocks_per_layer, n_draws)
    block = _perm(w, q, p.blocks_per_layer)[rank]
    layer = r.integers(0, p.n_layers, n_draws)
    head = r.integers(0, p.heads, n_draws)
    return (layer * p.blocks_per_layer + block) * p.heads + head


def _chat(w, q, p, epoch, r):
    """Shared-prefix chat: Zipf(1.1) over 500 prefixes with log-normal lengths
    (median 600 tokens, sigma 1.0, cap 8K); each request also touches a run of
    fresh prompt blocks once."""
    NB = p.blocks_per_layer
    key = ("chat", q)
    if key not in w._static:
        r0 = np.random.default_rng([w.seed, 2000 + q])
        n_prefix = 500
        lens = lognormal_tokens(r0, 600, 1.0, 8192, n_prefix)
        runs = np.maximum(1, -(-lens // p.block_tokens))
        region = max(1, int(0.6 * NB))
        runs = np.minimum(runs, region)
        starts = (np.cumsum(runs) - runs) % region
        shift = int(r0.integers(0, NB))
        w._static[key] = (runs, starts, region, shift)
    runs, starts, region, shift = w._static[key]
    n_req = max(1, int(round(40 * min(1.0, NB / 12288))))
    pref = zipf_bounded(r, 1.1, runs.size, n_req)
    fresh_len = np.maximum(1, -(-lognormal_tokens(r, 600, 1.0, 8192, n_req) // p.block_tokens))
    fresh_region = max(1, NB - region)
    blocks = []
    for i in range(n_req):
        b = (starts[pref[i]] + np.arange(runs[pref[i]])) % region
        blocks.append((b + shift) % NB)
        fl = int(min(fresh_len[i], fresh_region))
        fs = int(r.integers(0, fresh_region))
        fb = region + (fs + np.arange(fl)) % fresh_region
        blocks.append((fb + shift) % NB)
    return block_events(p, np.concatenate(blocks))


def _long_context(w, q, p, epoch, r):
    """64 concurrent long sequences: every block of each sequence's sliding
    window (last 4K tokens) is touched, plus 5 % of the older blocks."""
    NB = p.blocks_per_layer
    n_seq = 64
    win = max(1, min(4096 // p.block_tokens, (NB * 8 // 9) // n_seq))
    n_window = n_seq * win
    older = NB - n_window
    perm = _perm(w, q, NB)
    blocks = [perm[:n_window]]
    if older > 0:
        n_old = int(0.05 * older)
        blocks.append(perm[n_window + r.choice(older, size=n_old, replace=False)])
    return block_events(p, np.concatenate(blocks))


def _agentic(w, q, p, epoch, r):
    """300 multi-turn sessions (5-40 turns); 30 advance per epoch, each turn
    appends log-normal(median 800) tokens and re-reads its whole session prefix
    with probability 0.7."""
    NB = p.blocks_per_layer
    n_sess = 300
    key = ("agentic", q)
    if key not in w._static:
        r0 = np.random.default_rng([w.seed, 3000 + q])
        w._static[key] = {
            "start": r0.integers(0, NB, n_sess),
            "len": np.zeros(n_sess, np.int64),
            "turns_left": r0.integers(5, 41, n_sess),
            "cap": max(1, NB // 8),
        }
    st = w._static[key]
    active = max(1, int(round(30 * min(1.0, NB / 4096))))
    sess = r.choice(n_sess, size=min(active, n_sess), replace=False)
    blocks = []
    for s in sess:
        if st["turns_left"][s] <= 0:      # session ends; a new one takes its place
            st["start"][s] = int(r.integers(0, NB))
            st["len"][s] = 0
            st["turns_left"][s] = int(r.integers(5, 41))
        add = int(-(-lognormal_tokens(r, 800, 1.0, 1 << 16, 1)[0] // p.block_tokens))
        old_len = int(st["len"][s])
        new_len = min(old_len + add, st["cap"])
        if r.random() < 0.7 and old_len > 0:
            blocks.append((st["start"][s] + np.arange(old_len)) % NB)
        blocks.append((st["start"][s] + np.arange(old_len, max(new_len, old_len + 1))) % NB)
        st["len"][s] = max(new_len, min(old_len + 1, st["cap"]))
        st["turns_left"][s] -= 1
    return block_events(p, np.concatenate(blocks))


_STYLES = {"entry": _entry_mode, "chat": _chat, "long": _long_context, "agentic": _agentic}


# ---- byte pattern of a block ------------------------------------------------

_M64 = (1 << 64) - 1


def splitmix64(x: np.ndarray) -> np.ndarray:
    """SplitMix64 output function (Steele, Lea, Flood 2014) on uint64 arrays."""
    with np.errstate(over="ignore"):
        z = (x + np.uint64(0x9E3779B97F4A7C15))
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        return z ^ (z >> np.uint64(31))


def pattern_bytes(tags: np.ndarray, entry_bytes: int) -> np.ndarray:
    """Entry images (uint8 [len(tags), entry_bytes]): 8-byte word j of the block
    with handle g holds splitmix64(g * 2^20 + j), little endian."""
    assert entry_bytes % 8 == 0 and entry_bytes // 8 < (1 << 20)
    tags = np.asarray(tags, dtype=np.uint64)
    words = entry_bytes // 8
    x = (tags[:, None] << np.uint64(20)) + np.arange(words, dtype=np.uint64)[None, :]
    return splitmix64(x).view(np.uint8).reshape(tags.size, entry_bytes)


# ---- the five pools ---------------------------------------------------------

def config(i: int, scale: float = 1.0, ring_slots: Optional[int] = None,
           tiny_entries: bool = False) -> Workload:
    """Pool i (1..5).  scale < 1 shrinks blocks_per_layer (for tests and for
    devices with less free memory); ring_slots overrides the host ring size of
    every partition."""
    def nb(x):
        return max(8, int(round(x * scale)))

    def ring(default):
        return int(ring_slots) if ring_slots is not None else max(16, int(round(default * scale)))

    if i == 1:
        w = Workload("tiny-gqa", [gqa(2, 16, 4, 64, 16, nb(512), ring(4096), "entry")],
                     0.05, 0.02, seed=0, promote_style="recent")
    elif i == 2:
        w = Workload("llama3-8b-chat", [gqa(32, 32, 8, 128, 16, nb(12288), ring(1 << 20), "chat")],
                     0.10, 0.03, seed=1)
    elif i == 3:
        w = Workload("llama3-70b-longctx", [gqa(80, 64, 8, 128, 16, nb(18432), ring(1 << 22), "long")],
                     0.15, 0.10, seed=2, epochs=10, max_run=81920, promote_style="position")
    elif i == 4:
        w = Workload("deepseek-v3-agentic", [mla(61, 512, 64, 64, nb(14912), ring(1 << 17), "agentic")],
                     0.10, 0.05, seed=3, epochs=40)
    elif i == 5:
        blocks = nb(10720)
        parts = [mha(32, 32, 128, 16, blocks, ring(3 << 20), "mixed"),
                 gqa(80, 64, 8, 128, 16, blocks, ring(1 << 21), "mixed"),
                 mqa(32, 32, 128, 16, blocks, ring(1 << 18), "mixed"),
                 mla(61, 512, 64, 16, blocks, ring(1 << 18), "mixed")]
        w = Workload("mixed-fleet", parts, 0.10, 0.03, seed=4, epochs=8)
        w.pair_weights = np.random.default_rng([4, 77]).dirichlet(np.full(16, 0.5))
    else:
        raise ValueError("config index must be 1..5")
    if tiny_entries:
        # same entries, states and traces, but 32-64 byte blocks: for profiling the scoring
        # and selection kernels at full entry count without holding the payload
        for p in w.parts:
            if p.variant == MLA:
                p.d_latent, p.d_rope = 8, 0
            else:
                p.head_dim = 1
    return w
