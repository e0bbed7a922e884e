"""Thin ctypes binding of libkvtier.so (include/kvtier.h).

Argument marshalling only: every step of the path runs in the CUDA library.
PyTorch is used for device memory, pinned host memory and streams.  There is no
fallback: if the library cannot be loaded, loading raises.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

KV_OK = 0
KV_ERR_INVALID_ARG = -1
KV_ERR_UNSUPPORTED_VARIANT = -2
KV_ERR_K_TOO_LARGE = -3
KV_ERR_NO_FREE_SLOT = -4
KV_ERR_BAD_HOST_SLOT = -5
KV_ERR_HOST_TIER_TOO_SMALL = -6
KV_ERR_CUDA = -7
KV_ERR_INTERNAL = -8
KV_ERR_UNIMPLEMENTED = -9
KV_ERR_TAGS_EXHAUSTED = -10
KV_AUTO, KV_MHA, KV_GQA, KV_MQA, KV_MLA = -1, 0, 1, 2, 3
KV_STATE_FREE, KV_STATE_RESIDENT = 0, 1
KV_POLICY_BAYESIAN, KV_POLICY_EMA, KV_POLICY_LRU = 0, 1, 2
KV_NONE = 0xFFFFFFFF
KV_DEV_BAD_INDEX = 16
KV_DEV_BAD_HEAD_VALUE = 64
KV_DEV_BAD_SPAN_VALUE = 128
KV_LOC_HOST = 0x80000000


class kv_model_desc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("variant", "n_layers", "n_q_heads", "n_kv_heads", "head_dim", "d_latent",
                 "d_rope", "dtype_bits")]


class kv_partition_desc(C.Structure):
    _fields_ = [("model", kv_model_desc), ("block_tokens", C.c_int32), ("reserved", C.c_int32),
                ("blocks_per_layer", C.c_int64), ("d_slab", C.c_void_p), ("h_ring", C.c_void_p),
                ("ring_slots", C.c_uint64), ("h_meta", C.c_void_p)]


class kv_pool_desc(C.Structure):
    _fields_ = [("n_partitions", C.c_int32), ("reserved", C.c_int32),
                ("part", kv_partition_desc * 4),
                ("d_ema", C.c_void_p), ("d_decay", C.c_void_p), ("d_touch", C.c_void_p),
                ("d_last_epoch", C.c_void_p), ("d_pair", C.c_void_p), ("d_state", C.c_void_p),
                ("d_tag", C.c_void_p), ("d_score", C.c_void_p),
                ("d_hits", C.c_void_p), ("d_misses", C.c_void_p), ("d_P", C.c_void_p),
                ("alpha0", C.c_float), ("beta0", C.c_float),
                ("d_loc", C.c_void_p), ("n_tags", C.c_uint64),
                ("d_staging", C.c_void_p * 4), ("staging_bytes", C.c_uint64),
                ("max_promote", C.c_uint64),
                ("d_workspace", C.c_void_p), ("workspace_bytes", C.c_uint64),
                ("h_workspace", C.c_void_p), ("h_workspace_bytes", C.c_uint64)]


class kv_stats(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in
                ("epochs", "events", "victims", "promoted", "admitted", "bytes_demoted",
                 "bytes_promoted", "bytes_dropped", "n_entries", "n_free", "kernel_launches", "host_waits", "gathered")]


class kv_select_stats(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in ("selections", "hint_hits", "hint_misses", "reread_ctas")]


class kv_timing(C.Structure):
    _fields_ = [("pack_ms", C.c_double), ("unpack_ms", C.c_double),
                ("pack_launches", C.c_uint64), ("unpack_launches", C.c_uint64),
                ("pack_bytes", C.c_uint64), ("unpack_bytes", C.c_uint64),
                ("gather_ms", C.c_double), ("gather_launches", C.c_uint64), ("gather_bytes", C.c_uint64)]


class kv_slot_meta(C.Structure):
    _fields_ = [("tag", C.c_uint32), ("last_epoch", C.c_uint32), ("ema", C.c_float),
                ("decay", C.c_float), ("pair", C.c_uint32), ("demote_epoch", C.c_uint32)]


SLOT_META_DTYPE = np.dtype([("tag", "<u4"), ("last_epoch", "<u4"), ("ema", "<f4"),
                            ("decay", "<f4"), ("pair", "<u4"), ("demote_epoch", "<u4")])

EXPORTS = ("kv_size_bytes", "kv_infer_variant", "kv_entry_bytes", "kv_workspace_bytes",
           "kv_pool_create", "kv_pool_destroy", "kv_epoch_score", "kv_epoch_score_select", "kv_epoch_events", "kv_epoch_counts",
           "kv_epoch_update", "kv_set_policy", "kv_set_lazy_decay", "kv_hash_entries", "kv_dedup_table_slots", "kv_dedup_digests", "kv_set_confidence_blend", "kv_reuse_estimate", "kv_head_importance_update", "kv_set_head_multipliers", "kv_head_importance", "kv_head_weights", "kv_prefetch_window_update", "kv_set_prefetch_window", "kv_prefetch_span", "kv_prefetch_window", "kv_prefetch_list", "kv_select_victims", "kv_select_victim_blocks", "kv_select_victims_static", "kv_demote",
           "kv_promote", "kv_set_deferred_packing", "kv_flush", "kv_max_batch_bytes", "kv_admit", "kv_get_stats", "kv_ring_query",
           "kv_last_demote_counts", "kv_device_status", "kv_timing_enable", "kv_timing_read",
           "kv_set_select_variant", "kv_selection_stats", "kv_demote_counted", "kv_victim_counts", "kv_set_gather_threshold", "kv_set_l2_residency", "kv_last_cuda_error", "kv_status_string",
           "kv_version")

_lib = None


def load():
    """Loads (building first if the source is newer) libkvtier.so."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build()
    if not os.path.exists(path):
        raise RuntimeError("libkvtier.so is missing and could not be built")
    L = C.CDLL(path)
    vp, u64, i32, i64, u32 = C.c_void_p, C.c_uint64, C.c_int32, C.c_int64, C.c_uint32
    L.kv_size_bytes.restype = i64
    L.kv_size_bytes.argtypes = [C.POINTER(kv_model_desc), i64, i32]
    L.kv_infer_variant.restype = i32
    L.kv_infer_variant.argtypes = [C.POINTER(kv_model_desc)]
    L.kv_entry_bytes.restype = i64
    L.kv_entry_bytes.argtypes = [C.POINTER(kv_model_desc), i32]
    L.kv_workspace_bytes.restype = i32
    L.kv_workspace_bytes.argtypes = [C.POINTER(kv_pool_desc), C.POINTER(u64), C.POINTER(u64)]
    L.kv_pool_create.restype = i32
    L.kv_pool_create.argtypes = [C.POINTER(kv_pool_desc), vp, C.POINTER(vp)]
    L.kv_pool_destroy.restype = i32
    L.kv_pool_destroy.argtypes = [vp]
    L.kv_epoch_score.restype = i32
    L.kv_epoch_score.argtypes = [vp, u32, vp, vp, u64, vp]
    L.kv_epoch_score_select.restype = i32
    L.kv_epoch_score_select.argtypes = [vp, u32, vp, vp, u64, u64, vp, vp]
    L.kv_epoch_events.restype = i32
    L.kv_epoch_events.argtypes = [vp, vp, vp, u64, vp]
    L.kv_epoch_counts.restype = vp
    L.kv_epoch_counts.argtypes = [vp]
    L.kv_epoch_update.restype = i32
    L.kv_epoch_update.argtypes = [vp, u32, vp]
    L.kv_set_policy.restype = i32
    L.kv_set_policy.argtypes = [vp, i32]
    L.kv_set_lazy_decay.restype = i32
    L.kv_set_lazy_decay.argtypes = [vp, i32]
    L.kv_hash_entries.restype = i32
    L.kv_hash_entries.argtypes = [vp, vp, u64, vp, vp]
    L.kv_dedup_table_slots.restype = u64
    L.kv_dedup_table_slots.argtypes = [u64]
    L.kv_dedup_digests.restype = i32
    L.kv_dedup_digests.argtypes = [vp, u64, vp, vp, vp, u64, vp, vp, vp]
    L.kv_set_confidence_blend.restype = i32
    L.kv_set_confidence_blend.argtypes = [vp, C.c_float, i32, vp]
    L.kv_reuse_estimate.restype = vp
    L.kv_reuse_estimate.argtypes = [vp]
    L.kv_head_importance_update.restype = i32
    L.kv_head_importance_update.argtypes = [vp, i32, vp, C.c_float, vp]
    L.kv_set_head_multipliers.restype = i32
    L.kv_set_head_multipliers.argtypes = [vp, i32, vp, vp]
    L.kv_head_importance.restype = vp
    L.kv_head_importance.argtypes = [vp, i32]
    L.kv_head_weights.restype = vp
    L.kv_head_weights.argtypes = [vp, i32]
    L.kv_set_l2_residency.restype = i32
    L.kv_set_l2_residency.argtypes = [vp, C.c_uint64]
    L.kv_prefetch_window_update.restype = i32
    L.kv_prefetch_window_update.argtypes = [vp, i32, vp, C.c_float, vp]
    L.kv_set_prefetch_window.restype = i32
    L.kv_set_prefetch_window.argtypes = [vp, i32, C.c_float, C.c_uint32, vp]
    L.kv_prefetch_span.restype = vp
    L.kv_prefetch_span.argtypes = [vp, i32]
    L.kv_prefetch_window.restype = vp
    L.kv_prefetch_window.argtypes = [vp, i32]
    L.kv_prefetch_list.restype = i32
    L.kv_prefetch_list.argtypes = [vp, i32, vp, C.c_uint64, C.c_uint64, i32, vp, C.c_uint64, vp, vp]
    L.kv_select_victims.restype = i32
    L.kv_select_victims.argtypes = [vp, u64, vp, vp]
    L.kv_select_victim_blocks.restype = i32
    L.kv_select_victim_blocks.argtypes = [vp, u64, vp, C.POINTER(u64), vp]
    L.kv_select_victims_static.restype = i32
    L.kv_select_victims_static.argtypes = [vp, vp, u64, u64, vp, vp, vp]
    L.kv_demote.restype = i32
    L.kv_demote.argtypes = [vp, vp, u64, u64, vp, vp]
    L.kv_promote.restype = i32
    L.kv_promote.argtypes = [vp, i32, vp, u64, u64, vp, vp]
    L.kv_set_deferred_packing.restype = i32
    L.kv_set_deferred_packing.argtypes = [vp, i32]
    L.kv_flush.restype = i32
    L.kv_flush.argtypes = [vp]
    L.kv_max_batch_bytes.restype = u64
    L.kv_max_batch_bytes.argtypes = [vp, i32]
    L.kv_admit.restype = i32
    L.kv_admit.argtypes = [vp, u32, C.c_float, vp, u64, i32, C.POINTER(u64), vp]
    L.kv_get_stats.restype = i32
    L.kv_get_stats.argtypes = [vp, C.POINTER(kv_stats)]
    L.kv_ring_query.restype = i32
    L.kv_ring_query.argtypes = [vp, i32, C.POINTER(u64), C.POINTER(u64), vp]
    L.kv_last_demote_counts.restype = i32
    L.kv_last_demote_counts.argtypes = [vp, C.POINTER(u64 * 4)]
    L.kv_device_status.restype = i32
    L.kv_device_status.argtypes = [vp, vp, C.POINTER(u32)]
    L.kv_timing_enable.restype = i32
    L.kv_timing_enable.argtypes = [vp, i32]
    L.kv_timing_read.restype = i32
    L.kv_timing_read.argtypes = [vp, C.POINTER(kv_timing)]
    L.kv_set_select_variant.restype = i32
    L.kv_set_select_variant.argtypes = [vp, i32]
    L.kv_demote_counted.restype = i32
    L.kv_demote_counted.argtypes = [vp, vp, u64, vp, u64, vp, vp]
    L.kv_victim_counts.restype = vp
    L.kv_victim_counts.argtypes = [vp]
    L.kv_set_gather_threshold.restype = i32
    L.kv_set_gather_threshold.argtypes = [vp, u64]
    L.kv_selection_stats.restype = i32
    L.kv_selection_stats.argtypes = [vp, vp, vp]
    L.kv_last_cuda_error.restype = i32
    L.kv_last_cuda_error.argtypes = [vp]
    L.kv_status_string.restype = C.c_char_p
    L.kv_status_string.argtypes = [i32]
    L.kv_version.restype = C.c_char_p
    L.kv_version.argtypes = []
    _lib = L
    return L


class KVError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__("%s: %s (%d)" % (what, load().kv_status_string(status).decode(), status))


def model_desc(p) -> kv_model_desc:
    """kv_model_desc from a workloads.Partition (or anything with those fields)."""
    return kv_model_desc(p.variant, p.n_layers, p.n_q_heads, p.n_kv_heads, p.head_dim, p.d_latent,
                         p.d_rope, p.dtype_bits)


def kv_size_bytes(model: kv_model_desc, n_tokens: int, per_layer: bool = True) -> int:
    return load().kv_size_bytes(C.byref(model), n_tokens, 1 if per_layer else 0)


def kv_infer_variant(model: kv_model_desc) -> int:
    return load().kv_infer_variant(C.byref(model))


def kv_entry_bytes(model: kv_model_desc, block_tokens: int) -> int:
    return load().kv_entry_bytes(C.byref(model), block_tokens)


def _stream_ptr(s):
    return C.c_void_p(s.cuda_stream if s is not None else 0)


def kv_dedup_table_slots(m: int) -> int:
    return int(load().kv_dedup_table_slots(int(m)))


def kv_dedup_digests(d_digests, m, d_canon, d_refcount, d_table, d_n_unique, d_status, stream=None) -> int:
    """First position per digest and reference counts; arguments are torch device tensors."""
    return load().kv_dedup_digests(d_digests.data_ptr(), int(m), d_canon.data_ptr(), d_refcount.data_ptr(),
                                   d_table.data_ptr(), int(d_table.numel()),
                                   d_n_unique.data_ptr() if d_n_unique is not None else None,
                                   d_status.data_ptr(), _stream_ptr(stream) if stream is not None else None)


def kv_select_victims_static(d_score, d_state, n, k, d_victims, d_status=None, stream=None) -> int:
    """Selection with the library's built-in scratch: for callers that cannot
    allocate a workspace.  Arguments are torch device tensors; returns the status."""
    return load().kv_select_victims_static(
        d_score.data_ptr(), d_state.data_ptr(), int(n), int(k),
        d_victims.data_ptr() if d_victims is not None else None,
        d_status.data_ptr() if d_status is not None else None, _stream_ptr(stream))


class Pool:
    """A pool whose memory is owned by torch tensors and whose every operation is
    one call into the C library.  `parts` is a list of workloads.Partition."""

    def __init__(self, parts, n_tags, alpha0=1.0, beta0=1.0, staging_bytes=64 << 20,
                 max_promote=None, host_meta=True, device="cuda:0", stream=None):
        import torch
        self.torch = torch
        self.lib = load()
        self.device = torch.device(device)
        self.parts = list(parts)
        self.N = sum(p.n_entries for p in self.parts)
        self.n_tags = int(n_tags)
        self.max_promote = int(max_promote if max_promote is not None else self.N)
        self.staging_bytes = int(staging_bytes)
        dev = self.device

        def dz(n, dt):
            return torch.empty(max(int(n), 4), dtype=dt, device=dev)

        N = self.N
        self.ema = dz(N, torch.float32)
        self.decay = dz(N, torch.float32)
        self.touch = dz(N, torch.int32)
        self.last_epoch = dz(N, torch.int32)
        self.pair = dz(N, torch.uint8)
        self.state = dz(N, torch.uint8)
        self.tag = dz(N, torch.int32)
        self.score = dz(N, torch.float32)
        self.hits = dz(16, torch.int64)
        self.misses = dz(16, torch.int64)
        self.P = dz(16, torch.float32)
        self.loc = dz(self.n_tags, torch.int32)
        self.staging = [torch.empty(self.staging_bytes, dtype=torch.uint8, device=dev) for _ in range(4)]
        self.slabs, self.rings, self.metas = [], [], []
        d = kv_pool_desc()
        d.n_partitions = len(self.parts)
        self.entry_bytes = []
        for q, p in enumerate(self.parts):
            # sizes come from the library's own sizing calls (Eq. "unified"), not from the workload
            m = model_desc(p)
            eb = kv_entry_bytes(m, p.block_tokens)
            per_block = kv_size_bytes(m, p.block_tokens, per_layer=True)
            if eb <= 0 or per_block <= 0:
                raise KVError(min(eb, per_block), "kv_entry_bytes / kv_size_bytes")
            self.entry_bytes.append(eb)
            slab = torch.empty(p.n_layers * p.blocks_per_layer * per_block, dtype=torch.uint8, device=dev)
            ring = torch.empty(max(p.ring_slots * eb, 16), dtype=torch.uint8, pin_memory=True)
            meta = (torch.zeros(max(p.ring_slots * 24, 16), dtype=torch.uint8, pin_memory=True)
                    if host_meta else None)
            self.slabs.append(slab)
            self.rings.append(ring)
            self.metas.append(meta)
            d.part[q] = kv_partition_desc(model_desc(p), p.block_tokens, 0, p.blocks_per_layer,
                                          slab.data_ptr(), ring.data_ptr(), p.ring_slots,
                                          meta.data_ptr() if meta is not None else None)
        d.d_ema, d.d_decay = self.ema.data_ptr(), self.decay.data_ptr()
        d.d_touch, d.d_last_epoch = self.touch.data_ptr(), self.last_epoch.data_ptr()
        d.d_pair, d.d_state = self.pair.data_ptr(), self.state.data_ptr()
        d.d_tag, d.d_score = self.tag.data_ptr(), self.score.data_ptr()
        d.d_hits, d.d_misses, d.d_P = self.hits.data_ptr(), self.misses.data_ptr(), self.P.data_ptr()
        d.alpha0, d.beta0 = alpha0, beta0
        d.d_loc, d.n_tags = self.loc.data_ptr(), self.n_tags
        for b in range(4):
            d.d_staging[b] = self.staging[b].data_ptr()
        d.staging_bytes = self.staging_bytes
        d.max_promote = self.max_promote
        dev_b, host_b = C.c_uint64(0), C.c_uint64(0)
        rc = self.lib.kv_workspace_bytes(C.byref(d), C.byref(dev_b), C.byref(host_b))
        if rc != KV_OK:
            raise KVError(rc, "kv_workspace_bytes")
        self.workspace = torch.empty(max(dev_b.value, 16), dtype=torch.uint8, device=dev)
        self.h_workspace = torch.empty(max(host_b.value, 16), dtype=torch.uint8, pin_memory=True)
        d.d_workspace, d.workspace_bytes = self.workspace.data_ptr(), dev_b.value
        d.h_workspace, d.h_workspace_bytes = self.h_workspace.data_ptr(), host_b.value
        self.desc = d
        self.compute = stream if stream is not None else torch.cuda.Stream(device=dev)
        self.copy = torch.cuda.Stream(device=dev)        # D2H copies of demotions
        self.copy_h2d = torch.cuda.Stream(device=dev)    # H2D copies of promotions (overlap the D2H ones)
        self._h = C.c_void_p()
        with torch.cuda.device(dev):
            rc = self.lib.kv_pool_create(C.byref(d), _stream_ptr(self.compute), C.byref(self._h))
        if rc != KV_OK:
            raise KVError(rc, "kv_pool_create")

    def close(self):
        if getattr(self, "_h", None):
            self.sync()
            self.lib.kv_pool_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def sync(self):
        self.compute.synchronize()
        self.copy.synchronize()
        self.copy_h2d.synchronize()

    # -- the five calls, plus the harness extras; each returns the status --------
    def kv_epoch_score(self, epoch, d_ev_entry, d_ev_hit, n_events=None):
        n = int(n_events if n_events is not None else (d_ev_entry.numel() if d_ev_entry is not None else 0))
        return self.lib.kv_epoch_score(self._h, epoch,
                                       d_ev_entry.data_ptr() if n else None,
                                       d_ev_hit.data_ptr() if n else None, n, _stream_ptr(self.compute))

    def kv_epoch_score_select(self, epoch, d_ev_entry, d_ev_hit, n_events, k, d_victims):
        n = int(n_events)
        return self.lib.kv_epoch_score_select(self._h, epoch,
                                              d_ev_entry.data_ptr() if n else None,
                                              d_ev_hit.data_ptr() if n else None, n, int(k),
                                              d_victims.data_ptr() if k else None,
                                              _stream_ptr(self.compute))

    def kv_epoch_events(self, d_ev_entry, d_ev_hit, n_events=None):
        n = int(n_events if n_events is not None else (d_ev_entry.numel() if d_ev_entry is not None else 0))
        return self.lib.kv_epoch_events(self._h, d_ev_entry.data_ptr() if n else None,
                                        d_ev_hit.data_ptr() if n else None, n, _stream_ptr(self.compute))

    def kv_epoch_counts(self):
        """The 32 epoch counters as an int64 tensor aliasing the library's device memory."""
        addr = self.lib.kv_epoch_counts(self._h)
        off = addr - self.workspace.data_ptr()
        return self.workspace[off:off + 256].view(self.torch.int64)

    def kv_epoch_update(self, epoch):
        return self.lib.kv_epoch_update(self._h, epoch, _stream_ptr(self.compute))

    def kv_set_policy(self, policy):
        return self.lib.kv_set_policy(self._h, int(policy))

    def kv_hash_entries(self, d_ids, m, d_digests):
        """SHA-256 of the images of entries d_ids[:m] (None: entries 0..m-1) into d_digests (uint8 [m, 32])."""
        return self.lib.kv_hash_entries(self._h, d_ids.data_ptr() if d_ids is not None else None, int(m),
                                        d_digests.data_ptr(), _stream_ptr(self.compute))

    def kv_set_lazy_decay(self, on=True):
        return self.lib.kv_set_lazy_decay(self._h, int(bool(on)))

    def kv_set_confidence_blend(self, kappa, window):
        return self.lib.kv_set_confidence_blend(self._h, float(kappa), int(window), _stream_ptr(self.compute))

    def kv_reuse_estimate(self):
        """The 16 reuse estimates as a float32 tensor aliasing the library's device memory."""
        off = self.lib.kv_reuse_estimate(self._h) - self.workspace.data_ptr()
        return self.workspace[off:off + 64].view(self.torch.float32)

    def kv_head_importance_update(self, q, d_x, decay):
        return self.lib.kv_head_importance_update(self._h, int(q), d_x.data_ptr(), float(decay),
                                                  _stream_ptr(self.compute))

    def kv_set_head_multipliers(self, q, d_mult):
        return self.lib.kv_set_head_multipliers(self._h, int(q), d_mult.data_ptr() if d_mult is not None else None,
                                                _stream_ptr(self.compute))

    def _head_view(self, ptr, n):
        off = ptr - self.workspace.data_ptr()
        return self.workspace[off:off + 4 * n].view(self.torch.float32)

    def kv_head_importance(self, q):
        """Partition q's [layers][query heads] importance matrix (float32 tensor aliasing device memory)."""
        p = self.parts[q]
        qh = 1 if p.variant == KV_MLA else p.n_q_heads
        return self._head_view(self.lib.kv_head_importance(self._h, int(q)), p.n_layers * qh)

    def kv_head_weights(self, q):
        """Partition q's [layers][KV heads] score weights."""
        p = self.parts[q]
        return self._head_view(self.lib.kv_head_weights(self._h, int(q)), p.n_layers * p.heads)

    def kv_prefetch_window_update(self, q, d_span, decay):
        return self.lib.kv_prefetch_window_update(self._h, int(q), d_span.data_ptr() if d_span is not None else None,
                                                  float(decay), _stream_ptr(self.compute))

    def kv_set_prefetch_window(self, q, tokens, max_blocks):
        return self.lib.kv_set_prefetch_window(self._h, int(q), float(tokens), int(max_blocks),
                                               _stream_ptr(self.compute))

    def kv_prefetch_span(self, q):
        """Partition q's per-layer attention-span EMA in tokens (float32 tensor aliasing device memory)."""
        return self._head_view(self.lib.kv_prefetch_span(self._h, int(q)), self.parts[q].n_layers)

    def kv_prefetch_window(self, q):
        """Partition q's per-layer prefetch window in blocks (int32 view of the device's uint32 values)."""
        off = self.lib.kv_prefetch_window(self._h, int(q)) - self.workspace.data_ptr()
        return self.workspace[off:off + 4 * self.parts[q].n_layers].view(self.torch.int32)

    def kv_prefetch_list(self, q, d_table, n_pos, pos0, direction, d_out_slots, max_out, d_out_count):
        return self.lib.kv_prefetch_list(self._h, int(q), d_table.data_ptr() if d_table is not None else None,
                                         int(n_pos), int(pos0), int(direction),
                                         d_out_slots.data_ptr() if d_out_slots is not None else None, int(max_out),
                                         d_out_count.data_ptr() if d_out_count is not None else None,
                                         _stream_ptr(self.compute))

    def kv_set_l2_residency(self, budget_bytes):
        return self.lib.kv_set_l2_residency(self._h, int(budget_bytes))

    def kv_select_victims(self, k, d_victims):
        return self.lib.kv_select_victims(self._h, int(k), d_victims.data_ptr() if k else None,
                                          _stream_ptr(self.compute))

    def kv_select_victim_blocks(self, k_blocks, d_victims, wait=True):
        """Returns (status, number of entries written).  wait=False passes no place for the
        number: the call then never blocks, and the entries per partition are in
        kv_victim_counts() once the compute stream has run (the number returned is 0)."""
        n = C.c_uint64(0)
        rc = self.lib.kv_select_victim_blocks(self._h, int(k_blocks), d_victims.data_ptr() if k_blocks else None,
                                              C.byref(n) if wait else None, _stream_ptr(self.compute))
        return rc, n.value

    def kv_demote(self, d_victims, m, batch_bytes):
        return self.lib.kv_demote(self._h, d_victims.data_ptr() if m else None, int(m), int(batch_bytes),
                                  _stream_ptr(self.compute), _stream_ptr(self.copy))

    def kv_demote_counted(self, d_victims, m, counts, batch_bytes):
        c = (C.c_uint64 * 4)(*([int(x) for x in counts] + [0] * (4 - len(counts))))
        return self.lib.kv_demote_counted(self._h, d_victims.data_ptr() if m else None, int(m), C.byref(c),
                                          int(batch_bytes), _stream_ptr(self.compute), _stream_ptr(self.copy))

    def kv_victim_counts(self):
        """Victims per partition of the last selection (read after synchronising the compute stream)."""
        addr = self.lib.kv_victim_counts(self._h)
        return [int(x) for x in (C.c_uint64 * 4).from_address(addr)][:len(self.parts)]

    def kv_promote(self, partition, h_slots, batch_bytes):
        h_slots = np.ascontiguousarray(h_slots, dtype=np.uint64)
        return self.lib.kv_promote(self._h, partition, h_slots.ctypes.data_as(C.c_void_p) if h_slots.size else None,
                                   h_slots.size, int(batch_bytes), _stream_ptr(self.compute),
                                   _stream_ptr(self.copy_h2d))

    def kv_admit(self, epoch, decay, d_new_pairs, fill_pattern=True):
        n = C.c_uint64(0)
        rc = self.lib.kv_admit(self._h, epoch, decay, d_new_pairs.data_ptr(), d_new_pairs.numel(),
                               1 if fill_pattern else 0, C.byref(n), _stream_ptr(self.compute))
        return rc, n.value

    def kv_set_gather_threshold(self, run_bytes):
        return self.lib.kv_set_gather_threshold(self._h, int(run_bytes))

    def kv_set_deferred_packing(self, on=True):
        return self.lib.kv_set_deferred_packing(self._h, 1 if on else 0)

    def kv_flush(self):
        return self.lib.kv_flush(self._h)

    def kv_max_batch_bytes(self, partition=0):
        return int(self.lib.kv_max_batch_bytes(self._h, partition))

    def kv_get_stats(self):
        s = kv_stats()
        rc = self.lib.kv_get_stats(self._h, C.byref(s))
        if rc != KV_OK:
            raise KVError(rc, "kv_get_stats")
        return {n: int(getattr(s, n)) for n, _ in kv_stats._fields_}

    def kv_ring_query(self, partition, want_live=True):
        cur, nl = C.c_uint64(0), C.c_uint64(0)
        live = np.zeros(self.parts[partition].ring_slots, dtype=np.uint8) if want_live else None
        rc = self.lib.kv_ring_query(self._h, partition, C.byref(cur), C.byref(nl),
                                    live.ctypes.data_as(C.c_void_p) if live is not None and live.size else None)
        if rc != KV_OK:
            raise KVError(rc, "kv_ring_query")
        return cur.value, nl.value, live

    def kv_last_demote_counts(self):
        c = (C.c_uint64 * 4)()
        self.lib.kv_last_demote_counts(self._h, C.byref(c))
        return [int(x) for x in c]

    def kv_device_status(self):
        bits = C.c_uint32(0)
        rc = self.lib.kv_device_status(self._h, _stream_ptr(self.compute), C.byref(bits))
        if rc != KV_OK:
            raise KVError(rc, "kv_device_status")
        return bits.value

    def kv_set_select_variant(self, variant):
        return self.lib.kv_set_select_variant(self._h, int(variant))

    def kv_selection_stats(self):
        s = kv_select_stats()
        rc = self.lib.kv_selection_stats(self._h, _stream_ptr(self.compute), C.byref(s))
        if rc != KV_OK:
            raise KVError(rc, "kv_selection_stats")
        return {n: int(getattr(s, n)) for n, _ in kv_select_stats._fields_}

    def kv_timing_enable(self, on=True):
        return self.lib.kv_timing_enable(self._h, 1 if on else 0)

    def kv_timing_read(self):
        t = kv_timing()
        rc = self.lib.kv_timing_read(self._h, C.byref(t))
        if rc != KV_OK:
            raise KVError(rc, "kv_timing_read")
        return {n: getattr(t, n) for n, _ in kv_timing._fields_}

    def ring_meta(self, partition):
        """numpy view of the pinned per-slot metadata mirror (after sync)."""
        return self.metas[partition].numpy().view(SLOT_META_DTYPE)[: self.parts[partition].ring_slots]
