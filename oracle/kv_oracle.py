"""ctypes/numpy front end of the CPU oracle (TEST INFRASTRUCTURE).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this module.  It wraps oracle/kv_oracle.cpp, which states what the hot path
computes (sizing per Eq. "unified", the Beta posterior of Eq. "reuse", and this
build's readings of the EMA, score, selection, demotion and promotion steps).
All arrays handed out are live numpy views of the oracle's own state.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

AUTO, MHA, GQA, MQA, MLA = -1, 0, 1, 2, 3
OK = 0
ERR_INVALID_ARG = -1
ERR_UNSUPPORTED_VARIANT = -2
ERR_K_TOO_LARGE = -3
ERR_NO_FREE_SLOT = -4
ERR_BAD_HOST_SLOT = -5
ERR_HOST_TIER_TOO_SMALL = -6
ERR_TAGS_EXHAUSTED = -10
NONE = 0xFFFFFFFF
HOST_BIT = 0x80000000
FREE, RESIDENT = 0, 1


class Model(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("variant", "n_layers", "n_q_heads", "n_kv_heads", "head_dim",
                 "d_latent", "d_rope", "dtype_bits")]


class PartDesc(C.Structure):
    _fields_ = [("model", Model), ("block_tokens", C.c_int32), ("reserved", C.c_int32),
                ("blocks_per_layer", C.c_int64), ("ring_slots", C.c_int64)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        L.okv_size_bytes.restype = C.c_int64
        L.okv_size_bytes.argtypes = [C.POINTER(Model), C.c_int64, C.c_int32]
        L.okv_infer_variant.restype = C.c_int32
        L.okv_infer_variant.argtypes = [C.POINTER(Model)]
        L.okv_entry_bytes.restype = C.c_int64
        L.okv_entry_bytes.argtypes = [C.POINTER(Model), C.c_int32]
        L.okv_max_batch.restype = C.c_int64
        L.okv_max_batch.argtypes = [C.POINTER(Model), C.c_int64, C.c_int64]
        L.okv_create.restype = C.c_void_p
        L.okv_create.argtypes = [C.c_int32, C.POINTER(PartDesc), C.c_float, C.c_float,
                                 C.c_uint64, C.c_int32]
        L.okv_destroy.argtypes = [C.c_void_p]
        L.okv_num_entries.restype = C.c_int64
        L.okv_num_entries.argtypes = [C.c_void_p]
        L.okv_array.restype = C.c_void_p
        L.okv_array.argtypes = [C.c_void_p, C.c_int32]
        L.okv_part_array.restype = C.c_void_p
        L.okv_part_array.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
        L.okv_part_info.restype = C.c_int64
        L.okv_part_info.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
        L.okv_get_stats.argtypes = [C.c_void_p, C.c_void_p]
        L.okv_next_tag.restype = C.c_uint64
        L.okv_next_tag.argtypes = [C.c_void_p]
        L.okv_set_policy.restype = C.c_int32
        L.okv_set_policy.argtypes = [C.c_void_p, C.c_int32]
        L.okv_entry_image.restype = C.c_int64
        L.okv_entry_image.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p]
        L.okv_set_lazy_decay.restype = C.c_int32
        L.okv_set_lazy_decay.argtypes = [C.c_void_p, C.c_int32]
        L.okv_set_confidence_blend.restype = C.c_int32
        L.okv_set_confidence_blend.argtypes = [C.c_void_p, C.c_float, C.c_int32]
        L.okv_estimate.restype = C.c_void_p
        L.okv_estimate.argtypes = [C.c_void_p]
        L.okv_head_importance_update.restype = C.c_int32
        L.okv_head_importance_update.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_float]
        L.okv_set_head_multipliers.restype = C.c_int32
        L.okv_set_head_multipliers.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
        L.okv_head_array.restype = C.c_void_p
        L.okv_head_array.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
        L.okv_prefetch_window_update.restype = C.c_int32
        L.okv_prefetch_window_update.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_float]
        L.okv_set_prefetch_window.restype = C.c_int32
        L.okv_set_prefetch_window.argtypes = [C.c_void_p, C.c_int32, C.c_float, C.c_uint32]
        L.okv_prefetch_array.restype = C.c_void_p
        L.okv_prefetch_array.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
        L.okv_prefetch_list.restype = C.c_int32
        L.okv_prefetch_list.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_uint64, C.c_uint64, C.c_int32,
                                        C.c_void_p, C.c_uint64, C.c_void_p]
        L.okv_epoch_score.restype = C.c_int32
        L.okv_epoch_score.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_uint64]
        L.okv_select_victims.restype = C.c_int32
        L.okv_select_victims.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p]
        L.okv_select_victim_blocks.restype = C.c_int32
        L.okv_select_victim_blocks.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p, C.POINTER(C.c_uint64)]
        L.okv_demote.restype = C.c_int32
        L.okv_demote.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64]
        L.okv_promote.restype = C.c_int32
        L.okv_promote.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_uint64]
        L.okv_admit.restype = C.c_int64
        L.okv_admit.argtypes = [C.c_void_p, C.c_uint32, C.c_float, C.c_void_p, C.c_uint64,
                                C.c_void_p]
        _lib = L
    return _lib


def model(variant=AUTO, n_layers=1, n_q_heads=0, n_kv_heads=0, head_dim=0, d_latent=0,
          d_rope=0, dtype_bits=16):
    return Model(variant, n_layers, n_q_heads, n_kv_heads, head_dim, d_latent, d_rope, dtype_bits)


def size_bytes(m, n_tokens, per_layer=True):
    return lib().okv_size_bytes(C.byref(m), n_tokens, 1 if per_layer else 0)


def infer_variant(m):
    return lib().okv_infer_variant(C.byref(m))


def entry_bytes(m, block_tokens):
    return lib().okv_entry_bytes(C.byref(m), block_tokens)


def max_batch(m, budget_bytes, n_max):
    return lib().okv_max_batch(C.byref(m), budget_bytes, n_max)


def _view(ptr, dtype, n):
    if n == 0 or not ptr:
        return np.zeros(0, dtype=dtype)
    buf = (C.c_uint8 * (n * np.dtype(dtype).itemsize)).from_address(ptr)
    return np.frombuffer(buf, dtype=dtype, count=n)


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None and a.size else None


class OraclePool:
    """One pool of up to four partitions.

    parts: list of dicts {model: Model, block_tokens, blocks_per_layer, ring_slots}.
    """

    _ARR = {"ema": (0, np.float32), "decay": (1, np.float32), "touch": (2, np.uint32),
            "last_epoch": (3, np.uint32), "pair": (4, np.uint8), "state": (5, np.uint8),
            "tag": (6, np.uint32), "score": (7, np.float32)}
    _PARR = {"slab": (0, np.uint8), "ring": (1, np.uint8), "r_tag": (2, np.uint32),
             "r_pair": (3, np.uint8), "r_ema": (4, np.float32), "r_decay": (5, np.float32),
             "r_last_epoch": (6, np.uint32), "r_live": (7, np.uint8), "r_depoch": (8, np.uint32)}

    def __init__(self, parts, alpha0=1.0, beta0=1.0, n_tags=None, payload=True):
        L = lib()
        arr = (PartDesc * len(parts))()
        for q, p in enumerate(parts):
            arr[q] = PartDesc(p["model"], p["block_tokens"], 0, p["blocks_per_layer"],
                              p["ring_slots"])
        self.n_parts = len(parts)
        self._parts = list(parts)
        self._n_tags = int(n_tags) if n_tags is not None else 0
        self._h = L.okv_create(len(parts), arr, alpha0, beta0, self._n_tags, 1 if payload else 0)
        if not self._h:
            raise ValueError("oracle: invalid pool description")
        self.payload = bool(payload)
        self.N = L.okv_num_entries(self._h)

    def close(self):
        if self._h:
            lib().okv_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def __getattr__(self, name):
        if name in OraclePool._ARR:
            which, dt = OraclePool._ARR[name]
            return _view(lib().okv_array(self._h, which), dt, self.N)
        raise AttributeError(name)

    @property
    def hits(self):
        return _view(lib().okv_array(self._h, 8), np.uint64, 16)

    @property
    def misses(self):
        return _view(lib().okv_array(self._h, 9), np.uint64, 16)

    @property
    def P(self):
        return _view(lib().okv_array(self._h, 10), np.float32, 16)

    @property
    def loc(self):
        return _view(lib().okv_array(self._h, 11), np.uint32, self._n_tags)

    @property
    def next_tag(self):
        return int(lib().okv_next_tag(self._h))

    @property
    def estimate(self):
        """The 16 reuse estimates the Bayesian score uses (posterior, or its blend)."""
        return _view(lib().okv_estimate(self._h), np.float32, 16)

    def set_policy(self, policy):
        return lib().okv_set_policy(self._h, policy)

    def set_lazy_decay(self, on=True):
        """Promoted entries catch up on the EMA steps they missed while on the host."""
        return lib().okv_set_lazy_decay(self._h, int(bool(on)))

    def set_confidence_blend(self, kappa, window):
        return lib().okv_set_confidence_blend(self._h, kappa, window)

    def head_importance_update(self, q, x, decay):
        """EMA step of partition q's [layer][query head] importance matrix with observations x."""
        x = np.ascontiguousarray(x, dtype=np.float32)
        if not 0 <= q < self.n_parts:
            return ERR_INVALID_ARG
        assert x.size == self._head_shape(q, 0)
        return lib().okv_head_importance_update(self._h, q, _ptr(x), float(decay))

    def set_head_multipliers(self, q, mult):
        if not 0 <= q < self.n_parts:
            return ERR_INVALID_ARG
        if mult is not None:
            mult = np.ascontiguousarray(mult, dtype=np.float32)
            assert mult.size == self._head_shape(q, 1)
        return lib().okv_set_head_multipliers(self._h, q, _ptr(mult) if mult is not None else None)

    def _head_shape(self, q, which):
        m = self._parts[q]["model"]
        mla = lib().okv_infer_variant(C.byref(m)) == 3
        qh = 1 if mla else m.n_q_heads
        return m.n_layers * (qh if which == 0 else self.info(q)["H"])

    def head_array(self, q, name):
        """'importance' [L*QH], 'multipliers' [L*H] or 'weights' [L*H] of partition q."""
        which = {"importance": 0, "multipliers": 1, "weights": 2}[name]
        return _view(lib().okv_head_array(self._h, q, which), np.float32, self._head_shape(q, min(which, 1)))

    def prefetch_window_update(self, q, span, decay):
        """EMA step of partition q's per-layer attention span (tokens); recomputes the windows."""
        if not 0 <= q < self.n_parts:
            return ERR_INVALID_ARG
        span = np.ascontiguousarray(span, dtype=np.float32)
        assert span.size == self._parts[q]["model"].n_layers
        return lib().okv_prefetch_window_update(self._h, q, _ptr(span), float(decay))

    def set_prefetch_window(self, q, tokens, max_blocks):
        if not 0 <= q < self.n_parts:
            return ERR_INVALID_ARG
        return lib().okv_set_prefetch_window(self._h, q, float(tokens), int(max_blocks))

    def prefetch_array(self, q, name):
        """'span' (float32 [L], tokens) or 'window' (uint32 [L], blocks) of partition q."""
        which = {"span": 0, "window": 1}[name]
        n_layers = self._parts[q]["model"].n_layers
        return _view(lib().okv_prefetch_array(self._h, q, which), (np.float32, np.uint32)[which], n_layers)

    def prefetch_list(self, q, table, pos0, direction=1, max_out=None):
        """Ring slots of the host-tier blocks inside the per-layer windows of a sequence at
        position-block pos0; table is [n_pos][L][H] block handles.  Returns (rc, slots, count)."""
        if not 0 <= q < self.n_parts:
            return ERR_INVALID_ARG, None, 0
        table = np.ascontiguousarray(table, dtype=np.uint32)
        m = self._parts[q]["model"]
        per = m.n_layers * self.info(q)["H"]
        assert table.size % per == 0
        n_pos = table.size // per
        cap = table.size if max_out is None else int(max_out)
        out = np.zeros(max(cap, 1), dtype=np.uint64)
        n = C.c_uint64(0)
        rc = lib().okv_prefetch_list(self._h, q, _ptr(table) if table.size else None, n_pos, int(pos0),
                                     int(direction), _ptr(out), cap, C.byref(n))
        return rc, out[:min(cap, n.value)].copy(), int(n.value)

    def info(self, q):
        L = lib()
        names = ("base", "n", "entry_bytes", "chunk_bytes", "n_chunks", "H", "R", "cursor")
        return {n: int(L.okv_part_info(self._h, q, i)) for i, n in enumerate(names)}

    def part_array(self, q, name):
        which, dt = OraclePool._PARR[name]
        inf = self.info(q)
        if name == "slab":
            n = inf["n"] * inf["entry_bytes"] if self.payload else 0
        elif name == "ring":
            n = inf["R"] * inf["entry_bytes"] if self.payload else 0
        else:
            n = inf["R"]
        return _view(lib().okv_part_array(self._h, q, which), dt, n)

    def stats(self):
        out = np.zeros(8, dtype=np.uint64)
        lib().okv_get_stats(self._h, _ptr(out))
        names = ("epochs", "events", "victims", "promoted", "admitted", "bytes_demoted",
                 "bytes_promoted", "bytes_dropped")
        return {n: int(v) for n, v in zip(names, out)}

    def entry_image(self, i):
        """Bytes of entry i as one image: K chunk then V chunk (or the MLA chunk)."""
        q = max(q for q in range(self.n_parts) if self.info(q)["base"] <= i)
        out = np.zeros(self.info(q)["entry_bytes"], dtype=np.uint8)
        assert lib().okv_entry_image(self._h, int(i), _ptr(out)) == out.size
        return out

    def entry_digests(self, ids):
        """SHA-256 of each listed entry's image (content-addressable deduplication
        section: blocks are indexed by the SHA-256 hash of their content); uint8 [m, 32]."""
        return np.stack([sha256_bytes(self.entry_image(i)) for i in ids]) if len(ids) else \
            np.zeros((0, 32), np.uint8)

    def epoch_score(self, epoch, ev_entry, ev_hit):
        ev_entry = np.ascontiguousarray(ev_entry, dtype=np.uint32)
        ev_hit = np.ascontiguousarray(ev_hit, dtype=np.uint8)
        assert ev_entry.size == ev_hit.size
        return lib().okv_epoch_score(self._h, epoch, _ptr(ev_entry), _ptr(ev_hit), ev_entry.size)

    def select_victims(self, k):
        out = np.zeros(int(k), dtype=np.uint32)
        rc = lib().okv_select_victims(self._h, int(k), _ptr(out))
        return rc, out

    def select_victim_blocks(self, k_blocks):
        out = np.zeros(int(self.N), dtype=np.uint32)
        n = C.c_uint64(0)
        rc = lib().okv_select_victim_blocks(self._h, int(k_blocks), _ptr(out), C.byref(n))
        return rc, out[: n.value].copy()

    def demote(self, victims):
        victims = np.ascontiguousarray(victims, dtype=np.uint32)
        return lib().okv_demote(self._h, _ptr(victims), victims.size)

    def promote(self, q, slots):
        slots = np.ascontiguousarray(slots, dtype=np.uint64)
        return lib().okv_promote(self._h, q, _ptr(slots), slots.size)

    def admit(self, epoch, decay, new_pairs, new_payload=None):
        new_pairs = np.ascontiguousarray(new_pairs, dtype=np.uint8)
        if new_payload is not None:
            new_payload = np.ascontiguousarray(new_payload, dtype=np.uint8)
        return int(lib().okv_admit(self._h, epoch, decay, _ptr(new_pairs), new_pairs.size,
                                   _ptr(new_payload) if new_payload is not None else None))


# ---- content-addressable deduplication -----------------------------------------
def sha256_bytes(data):
    """SHA-256 (FIPS 180-4) of a byte string, as 32 uint8; the library routine is the step."""
    import hashlib
    return np.frombuffer(hashlib.sha256(bytes(memoryview(np.ascontiguousarray(data)))).digest(), dtype=np.uint8)


def dedup(digests):
    """Deduplication of a list of blocks by content hash (content-addressable
    deduplication section: a new block's hash is checked against the store; on a
    match a reference count is incremented instead of duplicating the block).
    Blocks are taken in list order, so the first block with a digest is the stored
    copy.  Returns (canon, refcount, n_unique): canon[j] = position of the stored
    copy block j refers to (j itself if it is the copy), refcount[i] = references
    to stored copy i, itself included (0 for blocks that are not stored)."""
    digests = np.asarray(digests, dtype=np.uint8).reshape(-1, 32)
    store = {}
    canon = np.zeros(len(digests), np.uint32)
    refcount = np.zeros(len(digests), np.uint32)
    for j, d in enumerate(digests):
        i = store.setdefault(d.tobytes(), j)
        canon[j] = i
        refcount[i] += 1
    return canon, refcount, len(store)
