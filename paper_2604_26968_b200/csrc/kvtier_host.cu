// C ABI of kvtier: argument checking, host-side bookkeeping (ring cursors, live
// slots, free counts), and the stream/event choreography of demotion and
// promotion.  Every step of the path itself runs in the kernels of kv_score.cu,
// kv_select.cu and kv_move.cu.
#include <cstdlib>
#include <cstring>
#include <limits>
#include <new>
#include <vector>

#include "kvtier_internal.cuh"

using namespace kvt;

namespace kvt {
std::atomic<uint64_t> g_kernel_launches{0};
}

namespace {

constexpr uint64_t kAlign = 256;
// promote lists in flight: pinned host buffers (and their device copies) used in turn, so that
// kv_promote only ever has to wait for the copy of the list given kListBufs calls earlier
constexpr int kListBufs = 8;
inline uint64_t align_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---- sizing (sizing section, Eq. "unified") ---------------------------------------
int32_t infer_variant(const kv_model_desc& m) {
  if (m.variant != KV_AUTO) {
    if (m.variant < KV_MHA || m.variant > KV_MLA) return KV_ERR_UNSUPPORTED_VARIANT;
    return m.variant;
  }
  if (m.d_latent > 0) return KV_MLA;
  if (m.n_q_heads <= 0 || m.n_kv_heads <= 0) return KV_ERR_INVALID_ARG;
  if (m.n_q_heads == m.n_kv_heads) return KV_MHA;
  if (m.n_kv_heads == 1) return KV_MQA;
  if (m.n_kv_heads < m.n_q_heads) return KV_GQA;
  return KV_ERR_UNSUPPORTED_VARIANT;
}

// elements of KV state per token per layer, or a negative status
int64_t token_elems(const kv_model_desc& m, int32_t variant) {
  if (variant == KV_MLA) {
    if (m.d_latent <= 0 || m.d_rope < 0) return KV_ERR_INVALID_ARG;
    return (int64_t)m.d_latent + (int64_t)m.d_rope;
  }
  if (m.head_dim <= 0) return KV_ERR_INVALID_ARG;
  int64_t heads;
  if (variant == KV_MHA) {
    heads = m.n_q_heads;
  } else {
    heads = m.n_kv_heads;
    if (variant == KV_MQA && heads != 1) return KV_ERR_INVALID_ARG;
  }
  if (heads <= 0) return KV_ERR_INVALID_ARG;
  return 2 * heads * (int64_t)m.head_dim;
}

int64_t kv_heads(const kv_model_desc& m, int32_t variant) {
  if (variant == KV_MLA) return 1;
  return variant == KV_MHA ? m.n_q_heads : m.n_kv_heads;
}

struct PartHost {
  int32_t variant = 0;
  uint64_t cursor = 0;
  uint64_t n_live = 0;
  uint64_t n_free = 0;
  std::vector<uint8_t> live;
  uint8_t* h_ring = nullptr;
  uint8_t* h_meta = nullptr;
  const uint8_t* ring_dev = nullptr;   // where the device sees h_ring (nullptr: it cannot)
};

}  // namespace

struct kv_pool {
  kv_pool_desc desc;
  int n_parts = 0;
  PartGeom geom[4];
  PartHost host[4];
  uint64_t bases[5] = {0, 0, 0, 0, 0};
  EntryState st;
  Workspace ws;
  uint8_t* staging[4] = {nullptr, nullptr, nullptr, nullptr};  // [0,1] demotion, [2,3] promotion
  uint64_t staging_bytes = 0;
  uint64_t max_promote = 0;
  uint32_t* h_list[kListBufs] = {};
  uint64_t* h_counts = nullptr;
  uint32_t* h_status = nullptr;
  uint64_t next_tag = 0;
  kv_stats stats;
  uint64_t last_counts[4] = {0, 0, 0, 0};
  cudaEvent_t ev_staging_free[4], ev_ready[4], ev_list_copied[kListBufs], ev_list_free[kListBufs], ev_counts;
  // copies in flight: the last two demotions per partition (ring slot range + completion event of
  // their D2H copies) and the last promotion's H2D copies
  struct D2H { cudaEvent_t ev; uint64_t start = 0, count = 0; bool valid = false; };
  D2H d2h[4][2];
  cudaEvent_t ev_h2d_done;
  bool h2d_valid = false;
  bool events_made = false;
  int demote_turn = 0, promote_turn = 0, list_turn = 0;
  int last_cuda_error = 0;
  ScoreOptions score_opt;   // eviction policy and confidence blend
  uint64_t gather_run_bytes = 1u << 20;    // promote lists whose runs average less go through the gather kernel
  // promotions run their kernels on the copy stream they are given; the compute stream joins
  // them (waits for ev_promoted) before the next kernel that reads what they wrote
  cudaEvent_t ev_promote_ready, ev_promoted[4];
  bool promote_open[4] = {false, false, false, false};
  int select_variant = 1;   // 1 = persistent cooperative selection, 0 = one launch per phase
  PartCounts pc;            // partition bases and where selections leave the victims per partition
  uint32_t* h_sel_stats = nullptr;
  HeadWeights head{};       // head-granular importance matrices and weights
  uint32_t n_head_imp = 0, n_head_w = 0;
  PrefetchState prefetch{}; // per-layer prefetch windows
  // a demotion whose later chunks are not enqueued yet (deferred packing)
  struct Pending {
    bool active = false, meta_done = false;
    const uint32_t* victims = nullptr;
    uint64_t off[4] = {0, 0, 0, 0}, kq[4] = {0, 0, 0, 0}, per[4] = {0, 0, 0, 0};
    uint64_t next[4] = {0, 0, 0, 0}, cursor0[4] = {0, 0, 0, 0};
    uint64_t promoted[4] = {0, 0, 0, 0};  // entries promoted into the partition since this demotion began
    cudaStream_t compute = nullptr, copy = nullptr;
  };
  Pending pending;
  bool deferred_packing = false;
  BlockGeom bgeom;          // paged blocks of all partitions in one index space
  // optional per-launch timing of the pack / unpack kernels
  struct Timed { cudaEvent_t a, b; int kind; uint64_t bytes; bool pending; };
  bool timing = false;
  std::vector<Timed> timed;
  size_t timed_next = 0;
  kv_timing totals;
};

namespace {

constexpr float kPrefetchSpanTokens = 2048.0f;   // span every layer starts with
constexpr uint32_t kPrefetchWindowCap = 65535;      // default cap on a window, blocks

struct Layout {
  uint64_t head_imp, head_mult, head_w;
  uint64_t pf_span, pf_win, pf_counts;
  uint64_t delta, hist, sel, status, blend, block_score, block_state, block_victims, part_counts, tile_counts, tile_offsets, free_list, slot_list[kListBufs];
  uint64_t ring[4][6];
  uint64_t dev_total;
  uint64_t h_list[kListBufs], h_counts, h_status, h_sel_stats, host_total;
  uint32_t n_tiles;
};

struct Derived {
  int n_parts;
  int32_t variant[4];
  uint64_t heads[4], n[4], entry_bytes[4], chunk_bytes[4], n_chunks[4];
  uint64_t bases[5];
  uint64_t N;
  uint64_t blocks[4], n_blocks;   // paged blocks (layer x block) per partition and in total
  uint64_t layers[4], q_heads[4];  // importance matrix of a partition: [layers][q_heads] (q_heads 1 for MLA)
  uint64_t n_head_imp, n_head_w;   // matrix elements / (layer, KV head) pairs over all partitions
};

int32_t derive(const kv_pool_desc* d, Derived* out) {
  if (!d || d->n_partitions < 1 || d->n_partitions > 4) return KV_ERR_INVALID_ARG;
  out->n_parts = d->n_partitions;
  uint64_t base = 0;
  for (int q = 0; q < d->n_partitions; ++q) {
    const kv_partition_desc& p = d->part[q];
    const int32_t v = infer_variant(p.model);
    if (v < 0) return v;
    const int64_t eb = kv_entry_bytes(&p.model, p.block_tokens);
    if (eb < 0) return (int32_t)eb;
    if (p.model.n_layers <= 0 || p.blocks_per_layer <= 0) return KV_ERR_INVALID_ARG;
    if (p.ring_slots >= 0x80000000ull) return KV_ERR_INVALID_ARG;
    out->variant[q] = v;
    out->heads[q] = (uint64_t)kv_heads(p.model, v);
    out->n_chunks[q] = (v == KV_MLA) ? 1 : 2;
    out->entry_bytes[q] = (uint64_t)eb;
    out->chunk_bytes[q] = (uint64_t)eb / out->n_chunks[q];
    if (out->chunk_bytes[q] % 16 != 0 || (uint64_t)eb >= (1ull << 23)) return KV_ERR_INVALID_ARG;
    out->n[q] = (uint64_t)p.model.n_layers * (uint64_t)p.blocks_per_layer * out->heads[q];
    out->bases[q] = base;
    base += out->n[q];
    out->blocks[q] = (uint64_t)p.model.n_layers * (uint64_t)p.blocks_per_layer;
    out->layers[q] = (uint64_t)p.model.n_layers;
    out->q_heads[q] = (v == KV_MLA) ? 1 : (uint64_t)p.model.n_q_heads;
    // every KV head serves a whole group of query heads
    if (out->q_heads[q] < out->heads[q] || out->q_heads[q] % out->heads[q] != 0) return KV_ERR_INVALID_ARG;
    if (out->layers[q] * out->q_heads[q] >= (1ull << 24)) return KV_ERR_INVALID_ARG;
    if ((uint64_t)p.blocks_per_layer * out->heads[q] >= (1ull << 32)) return KV_ERR_INVALID_ARG;
  }
  out->n_head_imp = out->n_head_w = 0;
  for (int q = 0; q < d->n_partitions; ++q) {
    out->n_head_imp += out->layers[q] * out->q_heads[q];
    out->n_head_w += out->layers[q] * out->heads[q];
  }
  for (int q = d->n_partitions; q <= 4; ++q) out->bases[q] = base;
  if (base == 0 || base >= 0x80000000ull) return KV_ERR_INVALID_ARG;  // ids must fit 31 bits
  out->N = base;
  out->n_blocks = 0;
  for (int q = 0; q < d->n_partitions; ++q) out->n_blocks += out->blocks[q];
  return KV_OK;
}

void make_layout(const kv_pool_desc* d, const Derived& g, Layout* L) {
  uint64_t o = 0;
  auto take = [&o](uint64_t bytes) { uint64_t at = o; o = align_up(o + bytes, kAlign); return at; };
  L->n_tiles = (uint32_t)((g.N + kTileEntries - 1) / kTileEntries + 2);
  L->delta = take(32 * 8);
  L->hist = take(3 * kHistBins * 4);
  L->sel = take(sizeof(SelectScalars));
  L->status = take(4);
  L->blend = take(sizeof(BlendState));
  L->head_imp = take(g.n_head_imp * 4);
  L->head_mult = take(g.n_head_w * 4);
  L->head_w = take(g.n_head_w * 4);
  {
    uint64_t layers = 0;
    for (int q = 0; q < g.n_parts; ++q) layers += g.layers[q];
    L->pf_span = take(layers * 4);
    L->pf_win = take(layers * 4);
    L->pf_counts = take(kPrefetchChunks * 4);
  }
  L->block_score = take(g.n_blocks * 4);
  L->block_state = take(g.n_blocks);
  L->block_victims = take(g.n_blocks * 4);
  L->part_counts = take(4 * 8);
  L->tile_counts = take((uint64_t)L->n_tiles * 8);
  L->tile_offsets = take((uint64_t)L->n_tiles * 8);
  L->free_list = take((g.N + 4096) * 4);   // (the selection's note scratch is addressed by whole chunks of 4,096)
  for (int b = 0; b < kListBufs; ++b) L->slot_list[b] = take(d->max_promote * 4);
  for (int q = 0; q < g.n_parts; ++q) {
    const uint64_t R = d->part[q].ring_slots;
    for (int a = 0; a < 4; ++a) L->ring[q][a] = take(R * 4);
    L->ring[q][4] = take(R);
    L->ring[q][5] = take(R * 4);
  }
  L->dev_total = o;
  uint64_t h = 0;
  auto htake = [&h](uint64_t bytes) { uint64_t at = h; h = align_up(h + bytes, kAlign); return at; };
  for (int b = 0; b < kListBufs; ++b) L->h_list[b] = htake(d->max_promote * 4);
  L->h_counts = htake(4 * 8);
  L->h_status = htake(4);
  L->h_sel_stats = htake(16);
  L->host_total = h;
}

inline cudaStream_t S(kv_stream_t s) { return static_cast<cudaStream_t>(s); }

int32_t cuda_fail(kv_pool* p, cudaError_t e) {
  p->last_cuda_error = (int)e;
  return KV_ERR_CUDA;
}

#define KV_CUDA(pool, call)                          \
  do {                                               \
    cudaError_t e__ = (call);                        \
    if (e__ != cudaSuccess) return cuda_fail(pool, e__); \
  } while (0)

// On a pool of several partitions every selection leaves the victims per partition in the
// pinned host workspace (kv_victim_counts): the kernels write them there themselves where
// the device can address that memory, else a 32-byte copy follows them.
int32_t counts_to_host(kv_pool* p, cudaStream_t s) {
  if (p->n_parts == 1 || p->pc.h_counts) return KV_OK;
  const cudaError_t e = cudaMemcpyAsync(p->h_counts, p->ws.part_counts, 4 * sizeof(uint64_t), cudaMemcpyDeviceToHost, s);
  if (e != cudaSuccess) { p->last_cuda_error = (int)e; return KV_ERR_CUDA; }
  return KV_OK;
}

// A scoring pass has been enqueued.
void scoring_pass_enqueued(kv_pool* p, uint32_t epoch) {
  p->stats.epochs += 1;
  for (int q = 0; q < p->n_parts; ++q) p->geom[q].epoch_now = epoch;
}

// every event object the pool owns (the timing events apart)
std::vector<cudaEvent_t*> all_events(kv_pool* p) {
  std::vector<cudaEvent_t*> evs;
  for (int b = 0; b < 4; ++b) { evs.push_back(&p->ev_staging_free[b]); evs.push_back(&p->ev_ready[b]); }
  for (int q = 0; q < 4; ++q) { evs.push_back(&p->d2h[q][0].ev); evs.push_back(&p->d2h[q][1].ev); }
  evs.push_back(&p->ev_h2d_done);
  for (int b = 0; b < kListBufs; ++b) { evs.push_back(&p->ev_list_copied[b]); evs.push_back(&p->ev_list_free[b]); }
  evs.push_back(&p->ev_counts);
  evs.push_back(&p->ev_promote_ready);
  for (int q = 0; q < 4; ++q) evs.push_back(&p->ev_promoted[q]);
  return evs;
}

void timing_settle(kv_pool* p, kv_pool::Timed& t) {
  if (!t.pending) return;
  float ms = 0.f;
  if (cudaEventSynchronize(t.b) == cudaSuccess && cudaEventElapsedTime(&ms, t.a, t.b) == cudaSuccess) {
    if (t.kind == 0) { p->totals.pack_ms += ms; p->totals.pack_launches += 1; p->totals.pack_bytes += t.bytes; }
    else if (t.kind == 1) { p->totals.unpack_ms += ms; p->totals.unpack_launches += 1; p->totals.unpack_bytes += t.bytes; }
    else { p->totals.gather_ms += ms; p->totals.gather_launches += 1; p->totals.gather_bytes += t.bytes; }
  }
  t.pending = false;
}

// Brackets one kernel launch with timing events when timing is on.
struct TimedScope {
  kv_pool* p; kv_pool::Timed* t = nullptr; cudaStream_t s;
  TimedScope(kv_pool* pool, int kind, uint64_t bytes, cudaStream_t stream) : p(pool), s(stream) {
    if (!p->timing || p->timed.empty()) return;
    t = &p->timed[p->timed_next];
    p->timed_next = (p->timed_next + 1) % p->timed.size();
    timing_settle(p, *t);
    t->kind = kind;
    t->bytes = bytes;
    cudaEventRecord(t->a, s);
  }
  ~TimedScope() {
    if (!t) return;
    cudaEventRecord(t->b, s);
    t->pending = true;
  }
};

// entries of one chunk: payload plus (optional) metadata records must fit a staging buffer
uint64_t entries_per_batch(const kv_pool* p, int q, uint64_t batch_bytes) {
  const uint64_t eb = p->geom[q].entry_bytes;
  const uint64_t meta = p->host[q].h_meta ? sizeof(kv_slot_meta) : 0;
  const uint64_t by_batch = batch_bytes / eb;
  const uint64_t by_staging = (p->staging_bytes >= 16 ? p->staging_bytes - 16 : 0) / (eb + meta);
  return by_batch < by_staging ? by_batch : by_staging;
}

}  // namespace

namespace {

// Enqueues one chunk of a demotion: pack victims [c0, c0+cnt) of partition q into
// a staging buffer on the compute stream, then copy it to the ring on the copy stream.
int32_t enqueue_pack_chunk(kv_pool* p, int q, uint64_t c0, uint64_t cnt) {
  kv_pool::Pending& pd = p->pending;
  const PartGeom& g = p->geom[q];
  PartHost& h = p->host[q];
  const uint64_t eb = g.entry_bytes, R = g.ring_slots;
  cudaStream_t compute = pd.compute, copy = pd.copy;
  const int b = p->demote_turn;
  p->demote_turn ^= 1;
  KV_CUDA(p, cudaStreamWaitEvent(compute, p->ev_staging_free[b], 0));
  const uint64_t meta_off = h.h_meta ? align_up(cnt * eb, 16) : ~0ull;
  const uint64_t slot0 = (pd.cursor0[q] + c0) % R;
  const uint32_t* victims = pd.victims + pd.off[q] + c0;
  {
    TimedScope ts(p, 0, cnt * eb, compute);
    KV_CUDA(p, launch_pack_tma(g, p->st, p->desc.d_loc, victims, cnt, slot0, p->staging[b], meta_off, p->ws,
                               compute, pd.meta_done ? 2u : 0u));
  }
  KV_CUDA(p, cudaEventRecord(p->ev_ready[b], compute));
  KV_CUDA(p, cudaStreamWaitEvent(copy, p->ev_ready[b], 0));
  const uint64_t first = (cnt < R - slot0) ? cnt : R - slot0;
  KV_CUDA(p, cudaMemcpyAsync(h.h_ring + slot0 * eb, p->staging[b], first * eb, cudaMemcpyDeviceToHost, copy));
  if (cnt > first)
    KV_CUDA(p, cudaMemcpyAsync(h.h_ring, p->staging[b] + first * eb, (cnt - first) * eb,
                               cudaMemcpyDeviceToHost, copy));
  if (h.h_meta) {
    const uint64_t mb = sizeof(kv_slot_meta);
    KV_CUDA(p, cudaMemcpyAsync(h.h_meta + slot0 * mb, p->staging[b] + meta_off, first * mb,
                               cudaMemcpyDeviceToHost, copy));
    if (cnt > first)
      KV_CUDA(p, cudaMemcpyAsync(h.h_meta, p->staging[b] + meta_off + first * mb, (cnt - first) * mb,
                                 cudaMemcpyDeviceToHost, copy));
  }
  KV_CUDA(p, cudaEventRecord(p->ev_staging_free[b], copy));
  return KV_OK;
}

// Enqueues pending chunks of the last demotion: of partition q_only until `need` of its
// victims are packed (the other partitions' chunks stay where they are: every partition has
// its own ring, so their order among each other is free), or, with q_only < 0, of every
// partition in order; never more than `max_chunks`.
int32_t drain_pending(kv_pool* p, int q_only, uint64_t need, uint64_t max_chunks) {
  kv_pool::Pending& pd = p->pending;
  if (!pd.active) return KV_OK;
  uint64_t done = 0;
  for (int q = 0; q < p->n_parts; ++q) {
    if (q_only >= 0 && q != q_only) continue;
    while (pd.next[q] < pd.kq[q]) {
      if (q_only >= 0 && pd.next[q] >= need) break;
      if (done >= max_chunks) return KV_OK;
      const uint64_t c0 = pd.next[q];
      const uint64_t cnt = (pd.kq[q] - c0 < pd.per[q]) ? pd.kq[q] - c0 : pd.per[q];
      const int32_t rc = enqueue_pack_chunk(p, q, c0, cnt);
      if (rc != KV_OK) return rc;
      pd.next[q] = c0 + cnt;
      ++done;
      if (pd.next[q] == pd.kq[q]) {
        // all copies of this partition are enqueued: remember the slots they write and when they end
        kv_pool::D2H older = p->d2h[q][1];
        p->d2h[q][1] = p->d2h[q][0];
        p->d2h[q][0] = older;  // reuse the older record's event object
        p->d2h[q][0].start = pd.cursor0[q];
        p->d2h[q][0].count = pd.kq[q];
        p->d2h[q][0].valid = true;
        KV_CUDA(p, cudaEventRecord(p->d2h[q][0].ev, pd.copy));
      }
    }
  }
  bool left = false;
  for (int q = 0; q < p->n_parts; ++q) left = left || pd.next[q] < pd.kq[q];
  pd.active = left;
  return KV_OK;
}

#define KV_DRAIN_ALL(pool)                                                  \
  do {                                                                      \
    const int32_t rc__ = drain_pending(pool, -1, 0, ~0ull);                  \
    if (rc__ != KV_OK) return rc__;                                         \
  } while (0)

// Makes `s` wait for the promotions whose kernels may still be running on their copy streams
// (all of them, or partition q's only).
int32_t join_promotions(kv_pool* p, cudaStream_t s, int q_only = -1) {
  for (int q = 0; q < p->n_parts; ++q) {
    if (!p->promote_open[q] || (q_only >= 0 && q != q_only)) continue;
    KV_CUDA(p, cudaStreamWaitEvent(s, p->ev_promoted[q], 0));
    p->promote_open[q] = false;
  }
  return KV_OK;
}

// Every call that reads or changes entry state first enqueues what deferred packing holds back
// and lets its stream wait for the promotions in flight.
#define KV_SETTLE(pool, stream)                                             \
  do {                                                                      \
    KV_DRAIN_ALL(pool);                                                     \
    const int32_t rc2__ = join_promotions(pool, S(stream));                 \
    if (rc2__ != KV_OK) return rc2__;                                       \
  } while (0)

}  // namespace

extern "C" {

int64_t kv_size_bytes(const kv_model_desc* model, int64_t n_tokens, int32_t per_layer) {
  if (!model || n_tokens < 0 || model->dtype_bits <= 0) return KV_ERR_INVALID_ARG;
  if (!per_layer && model->n_layers <= 0) return KV_ERR_INVALID_ARG;
  const int32_t v = infer_variant(*model);
  if (v < 0) return v;
  const int64_t elems = token_elems(*model, v);
  if (elems < 0) return elems;
  // 128-bit intermediate: n_tokens is caller-chosen
  const __int128 bits = (__int128)elems * model->dtype_bits * n_tokens;
  if (bits % 8 != 0) return KV_ERR_INVALID_ARG;
  __int128 bytes = bits / 8;
  if (!per_layer) bytes *= model->n_layers;
  if (bytes > (__int128)INT64_MAX) return KV_ERR_INVALID_ARG;
  return (int64_t)bytes;
}

int32_t kv_infer_variant(const kv_model_desc* model) {
  if (!model) return KV_ERR_INVALID_ARG;
  return infer_variant(*model);
}

int64_t kv_entry_bytes(const kv_model_desc* model, int32_t block_tokens) {
  if (!model || block_tokens <= 0) return KV_ERR_INVALID_ARG;
  const int64_t b = kv_size_bytes(model, block_tokens, 1);
  if (b < 0) return b;
  const int64_t h = kv_heads(*model, infer_variant(*model));
  if (h <= 0 || b % h != 0) return KV_ERR_INVALID_ARG;
  const int64_t eb = b / h;
  if (eb <= 0 || eb % 16 != 0) return KV_ERR_INVALID_ARG;
  return eb;
}

int32_t kv_workspace_bytes(const kv_pool_desc* desc, uint64_t* dev_bytes, uint64_t* host_bytes) {
  Derived g;
  const int32_t rc = derive(desc, &g);
  if (rc != KV_OK) return rc;
  Layout L;
  make_layout(desc, g, &L);
  if (dev_bytes) *dev_bytes = L.dev_total;
  if (host_bytes) *host_bytes = L.host_total;
  return KV_OK;
}

int32_t kv_pool_create(const kv_pool_desc* desc, kv_stream_t stream, kv_pool** out) {
  if (!out) return KV_ERR_INVALID_ARG;
  *out = nullptr;
  Derived g;
  const int32_t rc = derive(desc, &g);
  if (rc != KV_OK) return rc;
  if (!(desc->alpha0 > 0.0f) || !(desc->beta0 > 0.0f)) return KV_ERR_INVALID_ARG;
  const void* need[] = {desc->d_ema, desc->d_decay, desc->d_touch, desc->d_last_epoch, desc->d_pair,
                        desc->d_state, desc->d_tag, desc->d_score, desc->d_hits, desc->d_misses,
                        desc->d_P, desc->d_staging[0], desc->d_staging[1], desc->d_staging[2], desc->d_staging[3],
                        desc->d_workspace,
                        desc->h_workspace};
  for (const void* p : need)
    if (!p || !aligned16(p)) return KV_ERR_INVALID_ARG;
  if (desc->n_tags > 0 && (!desc->d_loc || !aligned16(desc->d_loc))) return KV_ERR_INVALID_ARG;
  if (desc->n_tags >= 0xFFFFFFFFull) return KV_ERR_INVALID_ARG;
  for (int q = 0; q < g.n_parts; ++q) {
    const kv_partition_desc& p = desc->part[q];
    if (!p.d_slab || !aligned16(p.d_slab)) return KV_ERR_INVALID_ARG;
    if (p.ring_slots > 0 && (!p.h_ring || !aligned16(p.h_ring))) return KV_ERR_INVALID_ARG;
    if (p.h_meta && !aligned16(p.h_meta)) return KV_ERR_INVALID_ARG;
    if (desc->staging_bytes < g.entry_bytes[q] + 64) return KV_ERR_INVALID_ARG;
  }
  Layout L;
  make_layout(desc, g, &L);
  if (desc->workspace_bytes < L.dev_total || desc->h_workspace_bytes < L.host_total)
    return KV_ERR_INVALID_ARG;

  kv_pool* p = new (std::nothrow) kv_pool();
  if (!p) return KV_ERR_INVALID_ARG;
  p->desc = *desc;
  p->n_parts = g.n_parts;
  std::memset(&p->stats, 0, sizeof(p->stats));
  std::memset(&p->totals, 0, sizeof(p->totals));
  for (int q = 0; q <= 4; ++q) p->bases[q] = g.bases[q];
  uint8_t* w = static_cast<uint8_t*>(desc->d_workspace);
  p->ws.delta = reinterpret_cast<unsigned long long*>(w + L.delta);
  p->ws.hist = reinterpret_cast<uint32_t*>(w + L.hist);
  p->ws.sel = reinterpret_cast<SelectScalars*>(w + L.sel);
  p->ws.status = reinterpret_cast<uint32_t*>(w + L.status);
  p->ws.blend = reinterpret_cast<BlendState*>(w + L.blend);
  p->ws.block_score = reinterpret_cast<float*>(w + L.block_score);
  p->ws.block_state = w + L.block_state;
  p->ws.block_victims = reinterpret_cast<uint32_t*>(w + L.block_victims);
  p->ws.part_counts = reinterpret_cast<unsigned long long*>(w + L.part_counts);
  p->ws.tile_counts = reinterpret_cast<uint2*>(w + L.tile_counts);
  p->ws.tile_offsets = reinterpret_cast<uint2*>(w + L.tile_offsets);
  p->ws.free_list = reinterpret_cast<uint32_t*>(w + L.free_list);
  for (int b = 0; b < kListBufs; ++b) p->ws.slot_list[b] = reinterpret_cast<uint32_t*>(w + L.slot_list[b]);
  p->ws.n_tiles = L.n_tiles;
  uint8_t* hw = static_cast<uint8_t*>(desc->h_workspace);
  for (int b = 0; b < kListBufs; ++b) p->h_list[b] = reinterpret_cast<uint32_t*>(hw + L.h_list[b]);
  p->h_counts = reinterpret_cast<uint64_t*>(hw + L.h_counts);
  p->h_status = reinterpret_cast<uint32_t*>(hw + L.h_status);
  for (int q = 0; q <= 4; ++q) p->pc.base[q] = g.bases[q];
  p->pc.n_parts = g.n_parts;
  p->pc.d_counts = p->ws.part_counts;
  {
    // kernels write the counts straight into the pinned host workspace where the device can address it
    void* dp = nullptr;
    if (cudaHostGetDevicePointer(&dp, p->h_counts, 0) == cudaSuccess) p->pc.h_counts = static_cast<unsigned long long*>(dp);
    else (void)cudaGetLastError();
    for (int q = 0; q < 4; ++q) p->h_counts[q] = 0;
  }
  p->h_sel_stats = reinterpret_cast<uint32_t*>(hw + L.h_sel_stats);
  p->st = EntryState{desc->d_ema, desc->d_decay, desc->d_touch, desc->d_last_epoch, desc->d_pair,
                     desc->d_state, desc->d_tag, desc->d_score, g.N};

  for (int q = 0; q < g.n_parts; ++q) {
    PartGeom& pg = p->geom[q];
    pg.slab = static_cast<uint8_t*>(desc->part[q].d_slab);
    pg.base = g.bases[q];
    pg.n = g.n[q];
    pg.heads = (uint32_t)g.heads[q];
    pg.n_chunks = (uint32_t)g.n_chunks[q];
    pg.chunk_bytes = (uint32_t)g.chunk_bytes[q];
    pg.entry_bytes = (uint32_t)g.entry_bytes[q];
    pg.ring_slots = (uint32_t)desc->part[q].ring_slots;
    pg.r_tag = reinterpret_cast<uint32_t*>(w + L.ring[q][0]);
    pg.r_last_epoch = reinterpret_cast<uint32_t*>(w + L.ring[q][1]);
    pg.r_ema = reinterpret_cast<float*>(w + L.ring[q][2]);
    pg.r_decay = reinterpret_cast<float*>(w + L.ring[q][3]);
    pg.r_pair = w + L.ring[q][4];
    pg.r_depoch = reinterpret_cast<uint32_t*>(w + L.ring[q][5]);
    pg.epoch_now = 0;
    pg.lazy_decay = 0;
    PartHost& ph = p->host[q];
    ph.variant = g.variant[q];
    ph.n_free = g.n[q];
    ph.live.assign((size_t)desc->part[q].ring_slots, 0);
    ph.h_ring = static_cast<uint8_t*>(desc->part[q].h_ring);
    ph.h_meta = static_cast<uint8_t*>(desc->part[q].h_meta);
    {
      void* dp = nullptr;
      if (ph.h_ring && cudaHostGetDevicePointer(&dp, ph.h_ring, 0) == cudaSuccess) ph.ring_dev = static_cast<const uint8_t*>(dp);
      else (void)cudaGetLastError();
    }
  }
  {
    HeadWeights& hd = p->head;
    hd.imp = reinterpret_cast<float*>(w + L.head_imp);
    hd.mult = reinterpret_cast<float*>(w + L.head_mult);
    hd.w = reinterpret_cast<float*>(w + L.head_w);
    hd.on = 0;
    hd.n_parts = g.n_parts;
    uint32_t io = 0, wo = 0;
    for (int q = 0; q < 4; ++q) {
      const bool in = q < g.n_parts;
      hd.base[q] = g.bases[q];
      hd.heads[q] = in ? (uint32_t)g.heads[q] : 1u;
      hd.q_heads[q] = in ? (uint32_t)g.q_heads[q] : 1u;
      hd.layers[q] = in ? (uint32_t)g.layers[q] : 0u;
      hd.per_layer[q] = in ? (uint32_t)(g.n[q] / g.layers[q]) : 1u;
      hd.imp_off[q] = io;
      hd.w_off[q] = wo;
      if (in) { io += hd.layers[q] * hd.q_heads[q]; wo += hd.layers[q] * hd.heads[q]; }
    }
    hd.base[4] = g.bases[4];
    p->n_head_imp = (uint32_t)g.n_head_imp;
    p->n_head_w = (uint32_t)g.n_head_w;
  }
  {
    PrefetchState& pf = p->prefetch;
    pf.span = reinterpret_cast<float*>(w + L.pf_span);
    pf.win = reinterpret_cast<uint32_t*>(w + L.pf_win);
    pf.chunk_counts = reinterpret_cast<uint32_t*>(w + L.pf_counts);
    uint32_t o = 0;
    for (int q = 0; q < 4; ++q) {
      const bool in = q < g.n_parts;
      pf.off[q] = o;
      pf.layers[q] = in ? (uint32_t)g.layers[q] : 0u;
      pf.heads[q] = in ? (uint32_t)g.heads[q] : 1u;
      pf.block_tokens[q] = in ? (uint32_t)desc->part[q].block_tokens : 1u;
      pf.w_max[q] = kPrefetchWindowCap;
      o += pf.layers[q];
    }
  }
  for (int b = 0; b < 4; ++b) p->staging[b] = static_cast<uint8_t*>(desc->d_staging[b]);
  p->staging_bytes = desc->staging_bytes;
  p->bgeom.n_parts = g.n_parts;
  {
    uint64_t bb = 0;
    for (int q = 0; q < 4; ++q) {
      p->bgeom.block_base[q] = bb;
      if (q < g.n_parts) {
        bb += g.blocks[q];
        p->bgeom.entry_base[q] = g.bases[q];
        p->bgeom.heads[q] = (uint32_t)g.heads[q];
        const int64_t hq = desc->part[q].model.n_q_heads > 0 ? desc->part[q].model.n_q_heads : (int64_t)g.heads[q];
        const int64_t wq = hq / (int64_t)g.heads[q];
        p->bgeom.weight[q] = (float)(wq > 0 ? wq : 1);
      } else {
        p->bgeom.entry_base[q] = g.N;
        p->bgeom.heads[q] = 1;
        p->bgeom.weight[q] = 1.0f;
      }
    }
    p->bgeom.block_base[4] = bb;
    for (int q = g.n_parts; q < 4; ++q) p->bgeom.block_base[q] = bb;
  }
  p->max_promote = desc->max_promote;
  p->stats.n_entries = g.N;
  p->stats.n_free = g.N;

  std::vector<cudaEvent_t*> evs = all_events(p);
  int made = 0;
  cudaError_t e = cudaSuccess;
  for (cudaEvent_t* ev : evs) {
    e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming);
    if (e != cudaSuccess) break;
    ++made;
  }
  if (e == cudaSuccess) {
    p->events_made = true;
    const float p0 = desc->alpha0 / (desc->alpha0 + desc->beta0);
    e = launch_init(p->st, desc->d_hits, desc->d_misses, desc->d_P, p0, desc->d_loc, desc->n_tags,
                    p->geom, p->n_parts, p->ws, S(stream));
    if (e == cudaSuccess) e = launch_head_init(p->head, p->n_head_imp, p->n_head_w, S(stream));
    for (int q = 0; q < g.n_parts && e == cudaSuccess; ++q)
      e = launch_prefetch_window(p->prefetch, q, 1, nullptr, 0.0f, kPrefetchSpanTokens, p->ws, S(stream));
  }
  if (e != cudaSuccess) {
    for (int i = 0; i < made; ++i) cudaEventDestroy(*evs[(size_t)i]);
    delete p;
    return KV_ERR_CUDA;
  }
  *out = p;
  return KV_OK;
}

int32_t kv_pool_destroy(kv_pool* p) {
  if (!p) return KV_ERR_INVALID_ARG;
  (void)drain_pending(p, -1, 0, ~0ull);
  if (p->events_made) {
    std::vector<cudaEvent_t*> evs = all_events(p);
    for (cudaEvent_t* ev : evs) cudaEventDestroy(*ev);
  }
  for (auto& t : p->timed) { cudaEventDestroy(t.a); cudaEventDestroy(t.b); }
  if (p->ws.l2_bytes) {   // the pool's lines in the persisting part of the L2 become ordinary lines again
    (void)cudaCtxResetPersistingL2Cache();
    (void)cudaGetLastError();
  }
  delete p;
  return KV_OK;
}

int32_t kv_epoch_events(kv_pool* p, const uint32_t* d_ev_entry, const uint8_t* d_ev_hit,
                        uint64_t n_events, kv_stream_t stream) {
  if (!p) return KV_ERR_INVALID_ARG;
  KV_SETTLE(p, stream);
  if (n_events > 0 && (!d_ev_entry || !d_ev_hit || !aligned16(d_ev_entry) || !aligned16(d_ev_hit)))
    return KV_ERR_INVALID_ARG;
  KV_CUDA(p, launch_event_reduce(d_ev_entry, d_ev_hit, n_events, p->st, p->ws, S(stream)));
  p->stats.events += n_events;
  return KV_OK;
}

uint64_t* kv_epoch_counts(kv_pool* p) {
  return p ? reinterpret_cast<uint64_t*>(p->ws.delta) : nullptr;
}

int32_t kv_epoch_update(kv_pool* p, uint32_t epoch, kv_stream_t stream) {
  if (!p) return KV_ERR_INVALID_ARG;
  KV_SETTLE(p, stream);
  KV_CUDA(p, launch_entry_update(p->st, p->desc.d_hits, p->desc.d_misses, p->desc.d_P, p->desc.alpha0,
                                 p->desc.beta0, p->ws, epoch, p->score_opt, p->head, S(stream)));
  scoring_pass_enqueued(p, epoch);
  return KV_OK;
}

int32_t kv_epoch_score(kv_pool* p, uint32_t epoch, const uint32_t* d_ev_entry, const uint8_t* d_ev_hit,
                       uint64_t n_events, kv_stream_t stream) {
  const int32_t rc = kv_epoch_events(p, d_ev_entry, d_ev_hit, n_events, stream);
  if (rc != KV_OK) return rc;
  return kv_epoch_update(p, epoch, stream);
}

int32_t kv_head_importance_update(kv_pool* p, int32_t q, const float* d_x, float decay, kv_stream_t stream) {
  if (!p || q < 0 || q >= p->n_parts || !d_x || !aligned16(d_x)) return KV_ERR_INVALID_ARG;
  if (!(decay >= 0.0f) || !(decay <= 1.0f)) return KV_ERR_INVALID_ARG;
  KV_SETTLE(p, stream);
  KV_CUDA(p, launch_head_update(p->head, q, 0, d_x, decay, p->ws, S(stream)));
  p->head.on |= 1u << q;
  return KV_OK;
}

int32_t kv_set_head_multipliers(kv_pool* p, int32_t q, const float* d_mult, kv_stream_t stream) {
  if (!p || q < 0 || q >= p->n_parts || (d_mult && !aligned16(d_mult))) return KV_ERR_INVALID_ARG;
  KV_SETTLE(p, stream);
  KV_CUDA(p, launch_head_update(p->head, q, 1, d_mult, 0.0f, p->ws, S(stream)));
  p->head.on |= 1u << q;
  return KV_OK;
}

const float* kv_head_importance(kv_pool* p, int32_t q) {
  return (p && q >= 0 && q < p->n_parts) ? p->head.imp + p->head.imp_off[q] : nullptr;
}

const float* kv_head_weights(kv_pool* p, int32_t q) {
  return (p && q >= 0 && q < p->n_parts) ? p->head.w + p->head.w_off[q] : nullptr;
}

int32_t kv_prefetch_window_update(kv_pool* p, int32_t q, const float* d_span, float decay, kv_stream_t stream) {
  if (!p || q < 0 || q >= p->n_parts || !d_span) return KV_ERR_INVALID_ARG;
  if (!(decay >= 0.0f) || !(decay <= 1.0f)) return KV_ERR_INVALID_ARG;
  KV_CUDA(p, launch_prefetch_window(p->prefetch, q, 0, d_span, decay, 0.0f, p->ws, S(stream)));
  return KV_OK;
}

int32_t kv_set_prefetch_window(kv_pool* p, int32_t q, float tokens, uint32_t max_blocks, kv_stream_t stream) {
  if (!p || q < 0 || q >= p->n_parts || max_blocks < 1) return KV_ERR_INVALID_ARG;
  if (!(tokens >= 0.0f) || !(tokens <= std::numeric_limits<float>::max())) return KV_ERR_INVALID_ARG;
  p->prefetch.w_max[q] = max_blocks;
  KV_CUDA(p, launch_prefetch_window(p->prefetch, q, 1, nullptr, 0.0f, tokens, p->ws, S(stream)));
  return KV_OK;
}

const float* kv_prefetch_span(kv_pool* p, int32_t q) {
  return (p && q >= 0 && q < p->n_parts) ? p->prefetch.span + p->prefetch.off[q] : nullptr;
}

const uint32_t* kv_prefetch_window(kv_pool* p, int32_t q) {
  return (p && q >= 0 && q < p->n_parts) ? p->prefetch.win + p->prefetch.off[q] : nullptr;
}

int32_t kv_prefetch_list(kv_pool* p, int32_t q, const uint32_t* d_table, uint64_t n_pos, uint64_t pos0,
                         int32_t direction, uint64_t* d_out_slots, uint64_t max_out, uint64_t* d_out_count,
                         kv_stream_t stream) {
  if (!p || q < 0 || q >= p->n_parts || !d_out_count || direction == 0) return KV_ERR_INVALID_ARG;
  if (n_pos > 0 && (!d_table || pos0 >= n_pos)) return KV_ERR_INVALID_ARG;
  if (max_out > 0 && !d_out_slots) return KV_ERR_INVALID_ARG;
  if (n_pos > (1ull << 40) / ((uint64_t)p->prefetch.layers[q] * p->prefetch.heads[q])) return KV_ERR_INVALID_ARG;
  // d_loc is written by demotions (compute stream, at the call) and by promotions (their copy stream)
  const int32_t rc = join_promotions(p, S(stream));
  if (rc != KV_OK) return rc;
  KV_CUDA(p, launch_prefetch_list(p->prefetch, q, d_table, n_pos, pos0, direction, p->desc.d_loc, p->desc.n_tags,
                                  reinterpret_cast<unsigned long long*>(d_out_slots), max_out,
                                  reinterpret_cast<unsigned long long*>(d_out_count), S(stream)));
  return KV_OK;
}

int32_t kv_select_victims(kv_pool* p, uint64_t k, uint32_t* d_victims, kv_stream_t stream) {
  if (!p) return KV_ERR_INVALID_ARG;
  KV_SETTLE(p, stream);
  if (k > p->stats.n_entries - p->stats.n_free) return KV_ERR_K_TOO_LARGE;
  if (k == 0) return KV_OK;
  if (!d_victims || !aligned16(d_victims)) return KV_ERR_INVALID_ARG;
  KV_CUDA(p, launch_select(p->st, k, d_victims, p->ws, S(stream), p->select_variant, &p->pc));
  return counts_to_host(p, S(stream));
}

int32_t kv_epoch_score_select(kv_pool* p, uint32_t epoch, const uint32_t* d_ev_entry,
                              const uint8_t* d_ev_hit, uint64_t n_events, uint64_t k, uint32_t* d_victims,
                              kv_stream_t stream) {
  if (!p) return KV_ERR_INVALID_ARG;
  KV_SETTLE(p, stream);
  if (n_events > 0 && (!d_ev_entry || !d_ev_hit || !aligned16(d_ev_entry) || !aligned16(d_ev_hit)))
    return KV_ERR_INVALID_ARG;
  if (k > p->stats.n_entries - p->stats.n_free) return KV_ERR_K_TOO_LARGE;
  if (k > 0 && (!d_victims || !aligned16(d_victims))) return KV_ERR_INVALID_ARG;
  KV_CUDA(p, launch_event_reduce(d_ev_entry, d_ev_hit, n_events, p->st, p->ws, S(stream)));
  p->stats.events += n_events;
  bool used = false;
  if (k > 0 && p->select_variant != 0) {
    const FusedScore fs{p->desc.d_hits, p->desc.d_misses, p->desc.d_P, p->desc.alpha0,
                        p->desc.beta0,  epoch,            p->score_opt,  p->head};
    KV_CUDA(p, launch_select_persistent(p->st, k, d_victims, p->ws, S(stream), &used, &fs, &p->pc));
  }
  if (used) {
    scoring_pass_enqueued(p, epoch);
    return counts_to_host(p, S(stream));
  }
  const int32_t rc = kv_epoch_update(p, epoch, stream);
  if (rc != KV_OK || k == 0) return rc;
  return kv_select_victims(p, k, d_victims, stream);
}

int32_t kv_select_victim_blocks(kv_pool* p, uint64_t k_blocks, uint32_t* d_victims, uint64_t* h_n_victims,
                                kv_stream_t stream) {
  if (!p) return KV_ERR_INVALID_ARG;
  KV_SETTLE(p, stream);
  if (h_n_victims) *h_n_victims = 0;
  if (k_blocks > p->bgeom.block_base[p->n_parts]) return KV_ERR_K_TOO_LARGE;
  if (k_blocks == 0) return KV_OK;
  if (!d_victims || !aligned16(d_victims)) return KV_ERR_INVALID_ARG;
  KV_CUDA(p, launch_select_blocks(p->st, p->bgeom, k_blocks, d_victims, p->ws, S(stream), p->pc.h_counts));
  if (p->n_parts == 1) {
    if (h_n_victims) *h_n_victims = k_blocks * p->bgeom.heads[0];
    return KV_OK;
  }
  // which partitions the chosen blocks fall in is only known on the device
  if (!p->pc.h_counts) {
    // (the expansion kernel could not write the entry counts to the host itself)
    KV_CUDA(p, cudaMemcpyAsync(p->h_counts, p->ws.part_counts, 4 * sizeof(uint64_t), cudaMemcpyDeviceToHost,
                               S(stream)));
  }
  if (!h_n_victims) return KV_OK;   // the caller reads kv_victim_counts once the stream has run
  KV_CUDA(p, cudaEventRecord(p->ev_counts, S(stream)));
  p->stats.host_waits += 1;
  KV_CUDA(p, cudaEventSynchronize(p->ev_counts));
  uint64_t m = 0;
  for (int q = 0; q < p->n_parts; ++q) {
    if (!p->pc.h_counts) p->h_counts[q] *= p->bgeom.heads[q];   // block counts came over: make them entries
    m += p->h_counts[q];
  }
  *h_n_victims = m;
  return KV_OK;
}

const uint64_t* kv_victim_counts(const kv_pool* p) { return p ? p->h_counts : nullptr; }

uint64_t kv_max_batch_bytes(const kv_pool* p, int32_t q) {
  if (!p || q < 0 || q >= p->n_parts) return 0;
  const uint64_t eb = p->geom[q].entry_bytes;
  return entries_per_batch(p, q, p->staging_bytes) * eb;
}

int32_t kv_demote(kv_pool* p, const uint32_t* d_victims, uint64_t m, uint64_t batch_bytes,
                  kv_stream_t compute_, kv_stream_t copy_) {
  if (!p) return KV_ERR_INVALID_ARG;
  if (p->n_parts == 1 || m == 0) {
    const uint64_t one[4] = {m, 0, 0, 0};
    return kv_demote_counted(p, d_victims, m, one, batch_bytes, compute_, copy_);
  }
  KV_SETTLE(p, compute_);
  if (!d_victims || !aligned16(d_victims) || m > p->stats.n_entries - p->stats.n_free)
    return KV_ERR_INVALID_ARG;
  // Several partitions and no counts from the caller: count on the device (a read-only kernel)
  // and wait for the answer.
  cudaStream_t compute = S(compute_);
  PartCounts pc = p->pc;
  pc.h_counts = nullptr;
  KV_CUDA(p, launch_partition_counts(d_victims, m, pc, compute));
  KV_CUDA(p, cudaMemcpyAsync(p->h_counts, p->ws.part_counts, 4 * sizeof(uint64_t), cudaMemcpyDeviceToHost,
                             compute));
  KV_CUDA(p, cudaEventRecord(p->ev_counts, compute));
  p->stats.host_waits += 1;
  KV_CUDA(p, cudaEventSynchronize(p->ev_counts));
  uint64_t counts[4] = {0, 0, 0, 0}, sum = 0;
  for (int q = 0; q < p->n_parts; ++q) { counts[q] = p->h_counts[q]; sum += counts[q]; }
  if (sum != m) return KV_ERR_INTERNAL;  // ids outside every partition
  return kv_demote_counted(p, d_victims, m, counts, batch_bytes, compute_, copy_);
}

int32_t kv_demote_counted(kv_pool* p, const uint32_t* d_victims, uint64_t m, const uint64_t* counts,
                          uint64_t batch_bytes, kv_stream_t compute_, kv_stream_t copy_) {
  if (!p || (m > 0 && !counts)) return KV_ERR_INVALID_ARG;
  KV_SETTLE(p, compute_);
  if (m == 0) {
    for (int q = 0; q < 4; ++q) p->last_counts[q] = 0;
    return KV_OK;
  }
  if (!d_victims || !aligned16(d_victims) || m > p->stats.n_entries - p->stats.n_free)
    return KV_ERR_INVALID_ARG;
  cudaStream_t compute = S(compute_), copy = S(copy_);
  uint64_t kq[4] = {0, 0, 0, 0}, sum = 0;
  for (int q = 0; q < p->n_parts; ++q) { kq[q] = counts[q]; sum += kq[q]; }
  if (sum != m) return KV_ERR_INVALID_ARG;
  uint64_t per[4] = {0, 0, 0, 0};
  for (int q = 0; q < p->n_parts; ++q) {
    if (kq[q] == 0) continue;
    if (kq[q] > p->geom[q].ring_slots) return KV_ERR_HOST_TIER_TOO_SMALL;
    if (kq[q] > p->geom[q].n - p->host[q].n_free) return KV_ERR_INVALID_ARG;
    if (batch_bytes < p->geom[q].entry_bytes) return KV_ERR_INVALID_ARG;
    per[q] = entries_per_batch(p, q, batch_bytes);
    if (per[q] == 0 || batch_bytes > p->staging_bytes) return KV_ERR_INVALID_ARG;
  }
  // ring slots written below may have been read by the last promotion's H2D copies
  if (p->h2d_valid) KV_CUDA(p, cudaStreamWaitEvent(copy, p->ev_h2d_done, 0));
  kv_pool::Pending& pd = p->pending;
  pd.victims = d_victims;
  pd.compute = compute;
  pd.copy = copy;
  pd.meta_done = p->deferred_packing;
  uint64_t off = 0;
  for (int q = 0; q < 4; ++q) {
    pd.off[q] = off;
    pd.kq[q] = kq[q];
    pd.per[q] = per[q];
    pd.next[q] = 0;
    pd.promoted[q] = 0;
    pd.cursor0[q] = q < p->n_parts ? p->host[q].cursor : 0;
    off += kq[q];
  }
  if (pd.meta_done) {
    // metadata of every victim now (slots become FREE, block table and ring mirror are updated);
    // the payload follows chunk by chunk
    for (int q = 0; q < p->n_parts; ++q)
      KV_CUDA(p, launch_pack_tma(p->geom[q], p->st, p->desc.d_loc, d_victims + pd.off[q], kq[q],
                                 pd.cursor0[q], p->staging[0], ~0ull, p->ws, compute, 1u));
  }
  pd.active = true;
  // host mirror of the rings: slot assignment is fixed here; overwritten live slots are dropped
  for (int q = 0; q < p->n_parts; ++q) {
    PartHost& h = p->host[q];
    const uint64_t eb = p->geom[q].entry_bytes, R = p->geom[q].ring_slots;
    for (uint64_t j = 0; j < kq[q]; ++j) {
      const uint64_t slot = (h.cursor + j) % R;
      if (h.live[slot]) {
        p->stats.bytes_dropped += eb;
      } else {
        h.live[slot] = 1;
        h.n_live += 1;
      }
    }
    if (R) h.cursor = (h.cursor + kq[q]) % R;
    h.n_free += kq[q];
    p->stats.bytes_demoted += kq[q] * eb;
  }
  for (int q = 0; q < 4; ++q) p->last_counts[q] = kq[q];
  p->stats.victims += m;
  p->stats.n_free += m;
  // without deferral everything is enqueued now; with it, the two chunks that need no wait
  return drain_pending(p, -1, 0, pd.meta_done ? 2 : ~0ull);
}

int32_t kv_promote(kv_pool* p, int32_t q, const uint64_t* h_slots, uint64_t m, uint64_t batch_bytes,
                   kv_stream_t compute_, kv_stream_t copy_) {
  if (!p || q < 0 || q >= p->n_parts) return KV_ERR_INVALID_ARG;
  if (m == 0) return KV_OK;
  if (!h_slots || m > p->max_promote) return KV_ERR_INVALID_ARG;
  const PartGeom& g = p->geom[q];
  PartHost& h = p->host[q];
  const uint64_t eb = g.entry_bytes, R = g.ring_slots;
  if (batch_bytes < eb || batch_bytes > p->staging_bytes) return KV_ERR_INVALID_ARG;
  // every listed slot live and distinct: mark with 2 while checking, restore on failure
  uint64_t checked = 0;
  bool ok = true;
  for (; checked < m; ++checked) {
    const uint64_t s = h_slots[checked];
    if (s >= R || h.live[s] != 1) { ok = false; break; }
    h.live[s] = 2;
  }
  if (!ok || m > h.n_free) {
    for (uint64_t j = 0; j < checked; ++j) h.live[h_slots[j]] = 1;
    return ok ? KV_ERR_NO_FREE_SLOT : KV_ERR_BAD_HOST_SLOT;
  }
  cudaStream_t compute = S(compute_), copy = S(copy_);
  {
    // an earlier promotion into this partition may still be scattering: the free list must see its result
    const int32_t rcj = join_promotions(p, compute, q);
    if (rcj != KV_OK) { for (uint64_t j2 = 0; j2 < m; ++j2) h.live[h_slots[j2]] = 1; return rcj; }
  }
  const uint64_t per = batch_bytes / eb;
  const int li = p->list_turn;
  p->list_turn = (p->list_turn + 1) % kListBufs;
  auto restore = [&]() { for (uint64_t j = 0; j < m; ++j) h.live[h_slots[j]] = 1; };
  // the list given kListBufs calls ago must have left this pinned buffer: normally long done
  cudaError_t e = cudaEventQuery(p->ev_list_copied[li]);
  if (e == cudaErrorNotReady) {
    (void)cudaGetLastError();
    p->stats.host_waits += 1;
    e = cudaEventSynchronize(p->ev_list_copied[li]);
  }
  if (e != cudaSuccess) { restore(); return cuda_fail(p, e); }
  // The H2D copies below may run on another stream than the D2H copies that filled the slots, so the
  // copy stream has to wait for the demotion(s) whose slot ranges the list touches.  d2h[q][0] is the
  // newest demotion whose copies are all enqueued; a pending (deferred) demotion is newer still and
  // has no completion event yet.
  const kv_pool::Pending& pd = p->pending;
  const bool q_pending = pd.active && pd.next[q] < pd.kq[q];
  bool hits_pending = false, hits_newest = false;
  for (uint64_t j = 0; j < m; ++j) {
    const uint64_t s = h_slots[j];
    p->h_list[li][j] = (uint32_t)s;
    if (q_pending && (s + R - pd.cursor0[q]) % R < pd.kq[q]) hits_pending = true;
    if (p->d2h[q][0].valid && (s + R - p->d2h[q][0].start) % R < p->d2h[q][0].count) hits_newest = true;
  }
  if (hits_pending) {
    // enqueue all of that demotion's copies for this partition; its record then becomes d2h[q][0]
    const int32_t rc = drain_pending(p, q, pd.kq[q], ~0ull);
    if (rc != KV_OK) { restore(); return rc; }
    hits_newest = true;
  } else if (q_pending) {
    hits_newest = p->d2h[q][0].valid;  // everything older than the pending demotion: wait for the newest recorded
  }
  if (e == cudaSuccess && hits_newest) e = cudaStreamWaitEvent(copy, p->d2h[q][0].ev, 0);
  if (e == cudaSuccess && !hits_newest && p->d2h[q][1].valid)
    e = cudaStreamWaitEvent(copy, p->d2h[q][1].ev, 0);
  if (e == cudaSuccess)
    e = cudaStreamWaitEvent(copy, p->ev_list_free[li], 0);  // older kernels are done reading the device list
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(p->ws.slot_list[li], p->h_list[li], m * 4, cudaMemcpyHostToDevice, copy);
  if (e == cudaSuccess) e = cudaEventRecord(p->ev_list_copied[li], copy);
  // this partition's free slots, ascending, in the partition's own stretch of the list scratch
  if (e == cudaSuccess) e = launch_free_list(p->st, g.base, g.base + g.n, m, p->ws, compute, g.base);
  if (e != cudaSuccess) { restore(); return cuda_fail(p, e); }
  const uint32_t* free_ids = p->ws.free_list + g.base;
  // With P entries promoted into the partition since the pending demotion began, chunk [c0, c0+cnt)
  // fills FREE slots number P+c0 .. P+c0+cnt-1 of the free set as it was right after that demotion.
  // Any of those that the demotion freed is among its first P+c0+cnt victims of the partition (victims
  // and free slots are both in ascending id order), so that much of its payload must have been
  // packed: enqueue it, and let the copy stream wait for it (and for the free list).
  auto ready_for = [&](uint64_t upto) -> int32_t {
    if (p->pending.active) {
      const int32_t rc = drain_pending(p, q, p->pending.promoted[q] + upto, ~0ull);
      if (rc != KV_OK) return rc;
    }
    KV_CUDA(p, cudaEventRecord(p->ev_promote_ready, compute));
    KV_CUDA(p, cudaStreamWaitEvent(copy, p->ev_promote_ready, 0));
    return KV_OK;
  };
  // A list of short runs (a position-ordered prefetch: a block's layers lie far apart in the
  // ring) would cost one DMA set-up per run; the gather kernel fetches such entries itself.
  uint64_t n_runs = 0;
  for (uint64_t j = 0; j < m; ++j) n_runs += (j == 0 || h_slots[j] != h_slots[j - 1] + 1);
  const bool gather = h.ring_dev && m * eb < n_runs * p->gather_run_bytes;
  // The transfers AND the scatter kernels go to the copy stream: the compute stream never waits
  // for the host link, and pack kernels of a demotion keep flowing between them.  Transfers run
  // one chunk ahead of the kernels (two staging buffers).
  auto h2d_chunk = [&](uint64_t c0) -> int32_t {
    const uint64_t cnt = (m - c0 < per) ? m - c0 : per;
    uint8_t* stage = p->staging[2 + ((c0 / per) & 1u)];
    uint64_t j = 0;
    while (j < cnt) {   // runs of consecutive ring slots become single copies
      const uint64_t s0 = h_slots[c0 + j];
      uint64_t len = 1;
      while (j + len < cnt && h_slots[c0 + j + len] == s0 + len) ++len;
      KV_CUDA(p, cudaMemcpyAsync(stage + j * eb, h.h_ring + s0 * eb, len * eb, cudaMemcpyHostToDevice, copy));
      j += len;
    }
    return KV_OK;
  };
  if (!gather) {
    const int32_t rc = h2d_chunk(0);
    if (rc != KV_OK) return rc;
  }
  for (uint64_t c0 = 0; c0 < m; c0 += per) {
    const uint64_t cnt = (m - c0 < per) ? m - c0 : per;
    if (!gather && c0 + per < m) {
      const int32_t rc = h2d_chunk(c0 + per);
      if (rc != KV_OK) return rc;
    }
    const int32_t rc = ready_for(c0 + cnt);
    if (rc != KV_OK) return rc;
    TimedScope ts(p, gather ? 2 : 1, cnt * eb, copy);
    if (gather)
      KV_CUDA(p, launch_gather_promote(g, p->st, p->desc.d_loc, p->ws.slot_list[li] + c0, free_ids + c0, cnt,
                                       h.ring_dev, p->ws, copy));
    else
      KV_CUDA(p, launch_unpack_tma(g, p->st, p->desc.d_loc, p->ws.slot_list[li] + c0, free_ids + c0, cnt,
                                   p->staging[2 + ((c0 / per) & 1u)], p->ws, copy));
  }
  KV_CUDA(p, cudaEventRecord(p->ev_list_free[li], copy));
  KV_CUDA(p, cudaEventRecord(p->ev_h2d_done, copy));
  KV_CUDA(p, cudaEventRecord(p->ev_promoted[q], copy));
  p->promote_open[q] = true;
  p->h2d_valid = true;
  if (gather) p->stats.gathered += m;
  if (p->pending.active) p->pending.promoted[q] += m;
  for (uint64_t j = 0; j < m; ++j) h.live[h_slots[j]] = 0;
  h.n_live -= m;
  h.n_free -= m;
  p->stats.n_free -= m;
  p->stats.promoted += m;
  p->stats.bytes_promoted += m * eb;
  return KV_OK;
}

int32_t kv_admit(kv_pool* p, uint32_t epoch, float decay, const uint8_t* d_new_pairs, uint64_t n_new_pairs,
                 int32_t fill_pattern, uint64_t* n_admitted, kv_stream_t stream) {
  if (!p) return KV_ERR_INVALID_ARG;
  KV_SETTLE(p, stream);
  const uint64_t n_free = p->stats.n_free;
  if (n_admitted) *n_admitted = 0;
  if (n_free == 0) return KV_OK;
  if (!d_new_pairs || n_new_pairs < n_free) return KV_ERR_INVALID_ARG;
  if (p->next_tag + n_free > p->desc.n_tags) return KV_ERR_TAGS_EXHAUSTED;
  KV_CUDA(p, launch_free_list(p->st, 0, p->st.n, n_free, p->ws, S(stream)));
  uint64_t first = 0;
  for (int q = 0; q < p->n_parts; ++q) {
    const uint64_t cnt = p->host[q].n_free;
    KV_CUDA(p, launch_admit(p->geom[q], p->st, p->desc.d_loc, p->ws.free_list, first, cnt, p->next_tag,
                            d_new_pairs, epoch, decay, fill_pattern, p->ws, S(stream)));
    first += cnt;
    p->host[q].n_free = 0;
  }
  p->next_tag += n_free;
  p->stats.admitted += n_free;
  p->stats.n_free = 0;
  if (n_admitted) *n_admitted = n_free;
  return KV_OK;
}

int32_t kv_get_stats(const kv_pool* p, kv_stats* out) {
  if (!p || !out) return KV_ERR_INVALID_ARG;
  *out = p->stats;
  out->kernel_launches = g_kernel_launches.load(std::memory_order_relaxed);
  return KV_OK;
}

int32_t kv_ring_query(const kv_pool* p, int32_t q, uint64_t* cursor, uint64_t* n_live, uint8_t* h_live) {
  if (!p || q < 0 || q >= p->n_parts) return KV_ERR_INVALID_ARG;
  if (cursor) *cursor = p->host[q].cursor;
  if (n_live) *n_live = p->host[q].n_live;
  if (h_live && !p->host[q].live.empty())
    std::memcpy(h_live, p->host[q].live.data(), p->host[q].live.size());
  return KV_OK;
}

int32_t kv_last_demote_counts(const kv_pool* p, uint64_t* counts4) {
  if (!p || !counts4) return KV_ERR_INVALID_ARG;
  for (int q = 0; q < 4; ++q) counts4[q] = p->last_counts[q];
  return KV_OK;
}

int32_t kv_device_status(kv_pool* p, kv_stream_t stream, uint32_t* status_bits) {
  if (!p || !status_bits) return KV_ERR_INVALID_ARG;
  KV_SETTLE(p, stream);
  KV_CUDA(p, cudaMemcpyAsync(p->h_status, p->ws.status, 4, cudaMemcpyDeviceToHost, S(stream)));
  KV_CUDA(p, cudaMemsetAsync(p->ws.status, 0, 4, S(stream)));
  KV_CUDA(p, cudaStreamSynchronize(S(stream)));
  *status_bits = *p->h_status;
  return KV_OK;
}

int32_t kv_hash_entries(kv_pool* p, const uint32_t* d_ids, uint64_t m, uint8_t* d_digests, kv_stream_t stream) {
  if (!p) return KV_ERR_INVALID_ARG;
  KV_SETTLE(p, stream);
  if (m == 0) return KV_OK;
  if (!d_digests || !aligned16(d_digests) || (d_ids && !aligned16(d_ids))) return KV_ERR_INVALID_ARG;
  if (!d_ids && m > p->stats.n_entries) return KV_ERR_INVALID_ARG;
  KV_CUDA(p, launch_hash_entries(p->geom, p->n_parts, d_ids, m, d_digests, p->ws, S(stream)));
  return KV_OK;
}

uint64_t kv_dedup_table_slots(uint64_t m) {
  uint64_t s = 16;
  while (s < 2 * m) s <<= 1;
  return s;
}

int32_t kv_dedup_digests(const uint8_t* d_digests, uint64_t m, uint32_t* d_canon, uint32_t* d_refcount,
                         uint32_t* d_table, uint64_t table_slots, uint32_t* d_n_unique, uint32_t* d_status,
                         kv_stream_t stream) {
  if (m >= 0xFFFFFFFFull) return KV_ERR_INVALID_ARG;
  if (!d_table || !aligned16(d_table) || table_slots < kv_dedup_table_slots(m) ||
      (table_slots & (table_slots - 1)) != 0 || !d_status)
    return KV_ERR_INVALID_ARG;
  if (m > 0 && (!d_digests || !aligned16(d_digests) || !d_canon || !d_refcount)) return KV_ERR_INVALID_ARG;
  const cudaError_t e = launch_dedup(d_digests, m, d_canon, d_refcount, d_table, table_slots, d_n_unique,
                                     d_status, S(stream));
  return e == cudaSuccess ? KV_OK : KV_ERR_CUDA;
}

int32_t kv_set_lazy_decay(kv_pool* p, int32_t on) {
  if (!p) return KV_ERR_INVALID_ARG;
  for (int q = 0; q < p->n_parts; ++q) p->geom[q].lazy_decay = on ? 1u : 0u;
  return KV_OK;
}

int32_t kv_set_policy(kv_pool* p, int32_t policy) {
  if (!p || policy < KV_POLICY_BAYESIAN || policy > KV_POLICY_LRU) return KV_ERR_INVALID_ARG;
  p->score_opt.policy = policy;
  return KV_OK;
}

int32_t kv_set_confidence_blend(kv_pool* p, float kappa, int32_t window, kv_stream_t stream) {
  if (!p || window < 0 || window > (int32_t)kMaxWindow || (window > 0 && !(kappa > 0.0f)))
    return KV_ERR_INVALID_ARG;
  KV_CUDA(p, launch_blend_reset(p->ws, S(stream)));
  p->score_opt.kappa = kappa;
  p->score_opt.window = (uint32_t)window;
  return KV_OK;
}

const float* kv_reuse_estimate(kv_pool* p) { return p ? p->ws.blend->estimate : nullptr; }

int32_t kv_flush(kv_pool* p) {
  if (!p) return KV_ERR_INVALID_ARG;
  KV_DRAIN_ALL(p);
  return KV_OK;
}

int32_t kv_set_gather_threshold(kv_pool* p, uint64_t run_bytes) {
  if (!p) return KV_ERR_INVALID_ARG;
  p->gather_run_bytes = run_bytes;
  return KV_OK;
}

int32_t kv_set_l2_residency(kv_pool* p, uint64_t budget_bytes) {
  if (!p) return KV_ERR_INVALID_ARG;
  int dev = 0, max_persist = 0, max_window = 0;
  KV_CUDA(p, cudaGetDevice(&dev));
  KV_CUDA(p, cudaDeviceGetAttribute(&max_persist, cudaDevAttrMaxPersistingL2CacheSize, dev));
  KV_CUDA(p, cudaDeviceGetAttribute(&max_window, cudaDevAttrMaxAccessPolicyWindowSize, dev));
  if (budget_bytes == 0) {
    if (p->ws.l2_bytes) {
      p->ws.l2_base = nullptr;
      p->ws.l2_bytes = 0;
      p->ws.l2_ratio = 0.0f;
      KV_CUDA(p, cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, 0));
    }
    return KV_OK;
  }
  if (max_persist <= 0 || max_window <= 0) return KV_ERR_UNIMPLEMENTED;
  uint64_t budget = budget_bytes < (uint64_t)max_persist ? budget_bytes : (uint64_t)max_persist;
  const uint64_t touch_bytes = p->st.n * 4, pair_bytes = p->st.n;
  const void* base;
  uint64_t bytes, set_aside;
  if (touch_bytes <= budget && touch_bytes <= (uint64_t)max_window) {   // the touch counts, whole
    base = p->st.touch;
    bytes = set_aside = touch_bytes;
  } else {                                                               // the pair bytes, as far as they fit
    base = p->st.pair;
    bytes = pair_bytes < (uint64_t)max_window ? pair_bytes : (uint64_t)max_window;
    set_aside = bytes < budget ? bytes : budget;
  }
  KV_CUDA(p, cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, (size_t)set_aside));
  p->ws.l2_base = base;
  p->ws.l2_bytes = (size_t)bytes;
  p->ws.l2_ratio = set_aside >= bytes ? 1.0f : (float)((double)set_aside / (double)bytes);
  return KV_OK;
}

int32_t kv_set_deferred_packing(kv_pool* p, int32_t on) {
  if (!p) return KV_ERR_INVALID_ARG;
  KV_DRAIN_ALL(p);
  p->deferred_packing = on != 0;
  return KV_OK;
}

int32_t kv_set_select_variant(kv_pool* p, int32_t variant) {
  if (!p || (variant != 0 && variant != 1)) return KV_ERR_INVALID_ARG;
  p->select_variant = variant;
  return KV_OK;
}

int32_t kv_selection_stats(kv_pool* p, kv_stream_t stream, kv_select_stats* out) {
  if (!p || !out) return KV_ERR_INVALID_ARG;
  KV_SETTLE(p, stream);
  KV_CUDA(p, cudaMemcpyAsync(p->h_sel_stats, &p->ws.sel->n_select, 4 * sizeof(uint32_t), cudaMemcpyDeviceToHost,
                             S(stream)));
  KV_CUDA(p, cudaStreamSynchronize(S(stream)));
  out->selections = p->h_sel_stats[0];
  out->hint_hits = p->h_sel_stats[1];
  out->hint_misses = p->h_sel_stats[2];
  out->reread_ctas = p->h_sel_stats[3];
  return KV_OK;
}

int32_t kv_timing_enable(kv_pool* p, int32_t on) {
  if (!p) return KV_ERR_INVALID_ARG;
  if (on && p->timed.empty()) {
    std::memset(&p->totals, 0, sizeof(p->totals));
    for (int i = 0; i < 256; ++i) {
      kv_pool::Timed t{};
      if (cudaEventCreate(&t.a) != cudaSuccess) return KV_ERR_CUDA;
      if (cudaEventCreate(&t.b) != cudaSuccess) { cudaEventDestroy(t.a); return KV_ERR_CUDA; }
      t.pending = false;
      p->timed.push_back(t);
    }
  }
  p->timing = on != 0;
  return KV_OK;
}

int32_t kv_timing_read(kv_pool* p, kv_timing* out) {
  if (!p || !out) return KV_ERR_INVALID_ARG;
  for (auto& t : p->timed) timing_settle(p, t);
  *out = p->totals;
  std::memset(&p->totals, 0, sizeof(p->totals));
  return KV_OK;
}

int32_t kv_last_cuda_error(const kv_pool* p) { return p ? p->last_cuda_error : 0; }

const char* kv_status_string(int32_t s) {
  switch (s) {
    case KV_OK: return "ok";
    case KV_ERR_INVALID_ARG: return "invalid argument";
    case KV_ERR_UNSUPPORTED_VARIANT: return "unsupported attention variant";
    case KV_ERR_K_TOO_LARGE: return "k exceeds the resident entries";
    case KV_ERR_NO_FREE_SLOT: return "not enough free HBM slots";
    case KV_ERR_BAD_HOST_SLOT: return "dead, duplicate or out-of-range host slot";
    case KV_ERR_HOST_TIER_TOO_SMALL: return "host ring smaller than the victim batch";
    case KV_ERR_CUDA: return "CUDA error";
    case KV_ERR_INTERNAL: return "internal inconsistency";
    case KV_ERR_UNIMPLEMENTED: return "not implemented";
    case KV_ERR_TAGS_EXHAUSTED: return "block handles exhausted";
    default: return "unknown status";
  }
}

const char* kv_version(void) { return "kvtier 0.1 (sm_100a)"; }

}  // extern "C"
