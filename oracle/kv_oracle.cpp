// kv_oracle.cpp -- TEST INFRASTRUCTURE, not product code.
//
// A plain, slow, single-threaded CPU statement of what one epoch of the
// predictive KV-cache manager computes: sizing, event reduction, EMA update,
// Beta posterior, eviction score, k-lowest selection, demotion to a host ring
// and promotion back.  It exists so that the CUDA library can be checked
// against something that a reader can compare with the paper by eye.  It shares
// no code, header, table or helper with the CUDA library and is only ever
// called from tests, the smoke check and the benchmark's CPU-baseline leg.
//
// Which parts are fixed by the paper and which are readings of it:
//   * okv_size_bytes / okv_infer_variant / okv_max_batch follow the sizing
//     section exactly (Eq. "unified", Eq. "total" and the batch formula).
//   * the posterior mean alpha/(alpha+beta) with +1 updates follows the
//     Bayesian-reuse section exactly (Eq. "reuse").
//   * the EMA recurrence, the product score, the per-(layer, head) importance
//     weighting (recurrence, group maximum, multipliers: okv_head_importance_update),
//     the per-layer prefetch window and the position-ordered prefetch list
//     (okv_prefetch_window_update, okv_prefetch_list),
//     the ring organisation of the host
//     tier, the free-slot rule of promotion and the lazy decay of promoted
//     entries (okv_set_lazy_decay) are NOT printed in the paper (it withholds
//     them): they are this build's readings, so their agreement with the paper
//     is "parity unpinned"; their internal consistency (closed forms, brute
//     force, conservation, equality with a resident twin) is what the tests pin.
//   * content hashing (okv_entry_image + SHA-256 in kv_oracle.py) follows the
//     content-addressable deduplication section: the hash is FIPS 180-4's and is
//     pinned to the standard's published digests; what counts as a block's
//     content (the entry image) and the list-order rule of the reference counts
//     are readings, pinned by a hand-built slab and a quadratic brute force.
//
// Floating point is IEEE binary32 with every operation rounded once
// (build with -O2 -ffp-contract=off -fno-fast-math; no flush-to-zero).
//
// Build: see oracle/build.py (g++ -std=c++17 -shared -fPIC).

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <new>
#include <numeric>
#include <vector>

namespace {

// Status values.  They are an interface shared (by value, not by header) with
// the CUDA library so that tests can compare error behaviour.
constexpr int32_t OK = 0;
constexpr int32_t ERR_INVALID_ARG = -1;
constexpr int32_t ERR_UNSUPPORTED_VARIANT = -2;
constexpr int32_t ERR_K_TOO_LARGE = -3;
constexpr int32_t ERR_NO_FREE_SLOT = -4;
constexpr int32_t ERR_BAD_HOST_SLOT = -5;
constexpr int32_t ERR_HOST_TIER_TOO_SMALL = -6;
constexpr int32_t ERR_TAGS_EXHAUSTED = -10;

constexpr int32_t VAR_AUTO = -1, VAR_MHA = 0, VAR_GQA = 1, VAR_MQA = 2, VAR_MLA = 3;

constexpr uint8_t ST_FREE = 0, ST_RESIDENT = 1;
constexpr uint32_t NONE = 0xFFFFFFFFu;      // "no tag" / "not cached"
constexpr uint32_t HOST_BIT = 0x80000000u;  // loc[]: bit 31 set = host tier

struct Model {
  int32_t variant, n_layers, n_q_heads, n_kv_heads, head_dim, d_latent, d_rope, dtype_bits;
};

struct PartDesc {
  Model model;
  int32_t block_tokens;
  int32_t reserved;
  int64_t blocks_per_layer;
  int64_t ring_slots;
};

// Architecture inference of the sizing section: a latent dimension means MLA;
// otherwise the head counts decide.  n_q == n_kv == 1 satisfies both the MHA
// and the MQA rule with the same byte count; MHA is returned.
int32_t infer_variant(const Model& m) {
  if (m.variant != VAR_AUTO) return m.variant;
  if (m.d_latent > 0) return VAR_MLA;
  if (m.n_q_heads <= 0 || m.n_kv_heads <= 0) return ERR_INVALID_ARG;
  if (m.n_kv_heads == m.n_q_heads) return VAR_MHA;
  if (m.n_kv_heads == 1) return VAR_MQA;
  if (m.n_kv_heads > 1 && m.n_kv_heads < m.n_q_heads) return VAR_GQA;
  return ERR_UNSUPPORTED_VARIANT;
}

// Elements of KV state per token per layer (Eq. "unified" without p and n).
int64_t elems_per_token(const Model& m, int32_t variant) {
  switch (variant) {
    case VAR_MHA:
      if (m.n_q_heads <= 0 || m.head_dim <= 0) return ERR_INVALID_ARG;
      return 2LL * m.n_q_heads * m.head_dim;
    case VAR_GQA:
    case VAR_MQA:
      if (m.n_kv_heads <= 0 || m.head_dim <= 0) return ERR_INVALID_ARG;
      if (variant == VAR_MQA && m.n_kv_heads != 1) return ERR_INVALID_ARG;
      return 2LL * m.n_kv_heads * m.head_dim;
    case VAR_MLA:
      if (m.d_latent <= 0 || m.d_rope < 0) return ERR_INVALID_ARG;
      return (int64_t)m.d_latent + m.d_rope;
    default:
      return ERR_UNSUPPORTED_VARIANT;
  }
}

// B(n) of Eq. "unified" (per layer) or L*B(n).  The precision p is carried as
// an integer number of bits so that INT4 (p = 0.5) needs no fractions; a size
// that is not a whole number of bytes is an error.
int64_t size_bytes(const Model& m, int64_t n_tokens, int32_t per_layer) {
  if (n_tokens < 0 || m.dtype_bits <= 0) return ERR_INVALID_ARG;
  if (!per_layer && m.n_layers <= 0) return ERR_INVALID_ARG;
  int32_t v = infer_variant(m);
  if (v < 0) return v;
  int64_t e = elems_per_token(m, v);
  if (e < 0) return e;
  int64_t bits = e * m.dtype_bits * n_tokens;
  if (bits % 8 != 0) return ERR_INVALID_ARG;
  int64_t bytes = bits / 8;
  return per_layer ? bytes : bytes * m.n_layers;
}

// KV heads that a paged block is split into: one entry per KV head, and a
// single entry for MLA (its matrix collapses to [layer][1]).
int64_t heads_of(const Model& m) {
  int32_t v = infer_variant(m);
  if (v < 0) return v;
  if (v == VAR_MLA) return 1;
  if (v == VAR_MHA) return m.n_q_heads;
  return m.n_kv_heads;
}

int64_t entry_bytes_of(const Model& m, int32_t block_tokens) {
  if (block_tokens <= 0) return ERR_INVALID_ARG;
  int64_t b = size_bytes(m, block_tokens, 1);
  if (b < 0) return b;
  int64_t h = heads_of(m);
  if (h <= 0) return ERR_INVALID_ARG;
  if (b % h != 0) return ERR_INVALID_ARG;
  return b / h;
}

struct Part {
  PartDesc d;
  int32_t variant;
  int64_t H, L, NB;
  int64_t base;         // first global entry id
  int64_t n;            // entries
  int64_t entry_bytes;  // bytes of one head-granular entry
  int64_t chunk_bytes;  // one contiguous piece in the slab (K or V; whole MLA entry)
  int32_t n_chunks;     // 2 (K,V) or 1 (MLA)
  int64_t R;            // ring slots
  uint64_t cur;         // ring cursor
  std::vector<uint8_t> slab;  // paged HBM image (payload mode only)
  std::vector<uint8_t> ring;  // host ring image (payload mode only)
  std::vector<uint32_t> r_tag, r_last_epoch;
  std::vector<uint32_t> r_depoch;  // epoch in which the slot's block was demoted
  std::vector<float> r_ema, r_decay;
  std::vector<uint8_t> r_pair, r_live;
  // head-granular importance (see okv_head_importance_update)
  int64_t QH;                   // query heads tracked per layer (1 for MLA)
  bool head_weights;            // scores of this partition are weighted per (layer, KV head)
  std::vector<float> h_imp;     // [L][QH] importance matrix
  std::vector<float> h_mult;    // [L][H] task-transition multipliers
  std::vector<float> h_w;       // [L][H] weight of a KV head: group maximum x multiplier
  // per-layer prefetch window (see okv_prefetch_window_update)
  std::vector<float> pf_span;     // [L] EMA of the observed attention span, in tokens
  std::vector<uint32_t> pf_win;   // [L] window in blocks
  uint32_t pf_max;                // most blocks a window may have
};

struct Stats {
  uint64_t epochs, events, victims, promoted, admitted;
  uint64_t bytes_demoted, bytes_promoted, bytes_dropped;
};

struct Pool {
  int n_parts = 0;
  Part part[4];
  int64_t N = 0;
  int payload = 0;
  float alpha0 = 1.0f, beta0 = 1.0f;
  int policy = 0;                 // 0 Bayesian, 1 EMA only, 2 LRU
  float kappa = 0.0f;             // confidence saturation constant
  int window = 0;                 // epochs in the sliding window; 0 = no blending
  int win_head = 0;
  std::vector<uint64_t> win;      // [window][32] per-epoch counts, index 2*pair + hit
  uint64_t wsum[32] = {0};        // sums over the window
  float estimate[16] = {0};       // reuse estimate used for scoring
  int lazy_decay = 0;             // promotion applies the EMA steps missed on the host
  uint32_t cur_epoch = 0;         // epoch of the last scoring pass
  std::vector<float> ema, decay, score;
  std::vector<uint32_t> touch, last_epoch, tag;
  std::vector<uint8_t> pair, state;
  uint64_t hits[16], misses[16];
  float P[16];
  std::vector<uint32_t> loc;
  uint64_t next_tag = 0;
  Stats st{};
};

int part_of(const Pool& p, int64_t id) {
  for (int q = 0; q < p.n_parts; ++q)
    if (id >= p.part[q].base && id < p.part[q].base + p.part[q].n) return q;
  return -1;
}

// Byte offset, inside the partition slab, of chunk c (0 = K or the MLA chunk,
// 1 = V) of local entry (layer, block, head).  Slab layout:
//   K/V variants: [layer][block][kv][head][token][dim]
//   MLA:          [layer][block][token][d_latent + d_rope]
int64_t chunk_offset(const Part& pt, int64_t local, int c) {
  int64_t head = local % pt.H;
  int64_t lb = local / pt.H;  // layer*NB + block
  if (pt.n_chunks == 1) return lb * pt.chunk_bytes;
  return ((lb * 2 + c) * pt.H + head) * pt.chunk_bytes;
}

void copy_entry_to_image(const Part& pt, int64_t local, uint8_t* image) {
  for (int c = 0; c < pt.n_chunks; ++c)
    std::memcpy(image + c * pt.chunk_bytes, pt.slab.data() + chunk_offset(pt, local, c),
                (size_t)pt.chunk_bytes);
}

void copy_image_to_entry(Part& pt, int64_t local, const uint8_t* image) {
  for (int c = 0; c < pt.n_chunks; ++c)
    std::memcpy(pt.slab.data() + chunk_offset(pt, local, c), image + c * pt.chunk_bytes,
                (size_t)pt.chunk_bytes);
}

// w[l] = min(w_max, max(1, ceil(S[l] / block_tokens))): one IEEE division, the ceiling exact.
void recompute_windows(Part& pt) {
  for (int64_t l = 0; l < pt.L; ++l) {
    const float q = pt.pf_span[(size_t)l] / (float)pt.d.block_tokens;
    double c = std::ceil((double)q);
    if (c < 1.0) c = 1.0;
    if (c > (double)pt.pf_max) c = (double)pt.pf_max;
    pt.pf_win[(size_t)l] = (uint32_t)c;
  }
}

// Weight of KV head (l, h): the maximum importance over the query heads that
// share it (the group of h is query heads h*G .. h*G+G-1, G = QH/H; one head for
// MHA, all of them for MQA, the single column for MLA), times the head's
// task-transition multiplier (head-granular eviction section).
void recompute_head_weights(Part& pt) {
  const int64_t G = pt.QH / pt.H;
  for (int64_t l = 0; l < pt.L; ++l) {
    for (int64_t hh = 0; hh < pt.H; ++hh) {
      float m = pt.h_imp[(size_t)(l * pt.QH + hh * G)];
      for (int64_t g = 1; g < G; ++g) {
        float v = pt.h_imp[(size_t)(l * pt.QH + hh * G + g)];
        if (v > m) m = v;
      }
      pt.h_w[(size_t)(l * pt.H + hh)] = m * pt.h_mult[(size_t)(l * pt.H + hh)];
    }
  }
}

}  // namespace

extern "C" {

int64_t okv_size_bytes(const Model* m, int64_t n_tokens, int32_t per_layer) {
  if (!m) return ERR_INVALID_ARG;
  return size_bytes(*m, n_tokens, per_layer);
}

int32_t okv_infer_variant(const Model* m) {
  if (!m) return ERR_INVALID_ARG;
  return infer_variant(*m);
}

int64_t okv_entry_bytes(const Model* m, int32_t block_tokens) {
  if (!m) return ERR_INVALID_ARG;
  return entry_bytes_of(*m, block_tokens);
}

// Maximum batch of the sizing section: floor(M_target / (L * B(n_max))).
int64_t okv_max_batch(const Model* m, int64_t budget_bytes, int64_t n_max) {
  if (!m || budget_bytes < 0) return ERR_INVALID_ARG;
  int64_t per_seq = size_bytes(*m, n_max, 0);
  if (per_seq <= 0) return per_seq < 0 ? per_seq : ERR_INVALID_ARG;
  return budget_bytes / per_seq;
}

// Creates a pool with every slot FREE and every ring slot dead.
// payload != 0 keeps the paged slabs and host rings as byte images.
void* okv_create(int32_t n_parts, const PartDesc* parts, float alpha0, float beta0,
                 uint64_t n_tags, int32_t payload) {
  if (n_parts < 1 || n_parts > 4 || !parts) return nullptr;
  if (!(alpha0 > 0.0f) || !(beta0 > 0.0f)) return nullptr;
  Pool* p = new (std::nothrow) Pool();
  if (!p) return nullptr;
  p->n_parts = n_parts;
  p->payload = payload;
  p->alpha0 = alpha0;
  p->beta0 = beta0;
  int64_t base = 0;
  for (int q = 0; q < n_parts; ++q) {
    Part& pt = p->part[q];
    pt.d = parts[q];
    pt.variant = infer_variant(pt.d.model);
    int64_t H = heads_of(pt.d.model);
    int64_t eb = entry_bytes_of(pt.d.model, pt.d.block_tokens);
    if (pt.variant < 0 || H <= 0 || eb <= 0 || pt.d.model.n_layers <= 0 ||
        pt.d.blocks_per_layer <= 0 || pt.d.ring_slots < 0) {
      delete p;
      return nullptr;
    }
    pt.H = H;
    pt.L = pt.d.model.n_layers;
    pt.NB = pt.d.blocks_per_layer;
    pt.base = base;
    pt.n = pt.L * pt.NB * pt.H;
    pt.entry_bytes = eb;
    pt.n_chunks = (pt.variant == VAR_MLA) ? 1 : 2;
    pt.chunk_bytes = eb / pt.n_chunks;
    pt.R = pt.d.ring_slots;
    pt.cur = 0;
    if (payload) {
      pt.slab.assign((size_t)(pt.n * eb), 0);
      pt.ring.assign((size_t)(pt.R * eb), 0);
    }
    pt.r_tag.assign((size_t)pt.R, NONE);
    pt.r_last_epoch.assign((size_t)pt.R, 0);
    pt.r_depoch.assign((size_t)pt.R, 0);
    pt.r_ema.assign((size_t)pt.R, 0.0f);
    pt.r_decay.assign((size_t)pt.R, 0.0f);
    pt.r_pair.assign((size_t)pt.R, 0);
    pt.r_live.assign((size_t)pt.R, 0);
    pt.QH = (pt.variant == VAR_MLA) ? 1 : pt.d.model.n_q_heads;
    if (pt.QH < pt.H || pt.QH % pt.H != 0) {  // every KV head serves a whole group of query heads
      delete p;
      return nullptr;
    }
    pt.head_weights = false;
    pt.h_imp.assign((size_t)(pt.L * pt.QH), 1.0f);
    pt.h_mult.assign((size_t)(pt.L * pt.H), 1.0f);
    pt.pf_max = 65535;
    pt.pf_span.assign((size_t)pt.L, 2048.0f);
    pt.pf_win.assign((size_t)pt.L, 0);
    recompute_windows(pt);
    pt.h_w.assign((size_t)(pt.L * pt.H), 1.0f);
    base += pt.n;
  }
  if (base >= (int64_t)HOST_BIT) {  // ids and slots must fit 31 bits
    delete p;
    return nullptr;
  }
  p->N = base;
  size_t N = (size_t)base;
  p->ema.assign(N, 0.0f);
  p->decay.assign(N, 0.0f);
  p->score.assign(N, std::numeric_limits<float>::infinity());
  p->touch.assign(N, 0);
  p->last_epoch.assign(N, 0);
  p->tag.assign(N, NONE);
  p->pair.assign(N, 0);
  p->state.assign(N, ST_FREE);
  for (int i = 0; i < 16; ++i) {
    p->hits[i] = p->misses[i] = 0;
    p->P[i] = alpha0 / (alpha0 + beta0);
    p->estimate[i] = p->P[i];
  }
  p->loc.assign((size_t)n_tags, NONE);
  return p;
}

void okv_destroy(void* h) { delete static_cast<Pool*>(h); }

int64_t okv_num_entries(void* h) { return static_cast<Pool*>(h)->N; }

// Raw views for the Python side (numpy wraps them; nothing is copied).
// which: 0 ema f32, 1 decay f32, 2 touch u32, 3 last_epoch u32, 4 pair u8,
// 5 state u8, 6 tag u32, 7 score f32, 8 hits u64[16], 9 misses u64[16],
// 10 P f32[16], 11 loc u32[n_tags]
void* okv_array(void* h, int32_t which) {
  Pool* p = static_cast<Pool*>(h);
  switch (which) {
    case 0: return p->ema.data();
    case 1: return p->decay.data();
    case 2: return p->touch.data();
    case 3: return p->last_epoch.data();
    case 4: return p->pair.data();
    case 5: return p->state.data();
    case 6: return p->tag.data();
    case 7: return p->score.data();
    case 8: return p->hits;
    case 9: return p->misses;
    case 10: return p->P;
    case 11: return p->loc.data();
    default: return nullptr;
  }
}

// Per-partition views. which: 0 slab u8, 1 ring u8, 2 r_tag u32, 3 r_pair u8,
// 4 r_ema f32, 5 r_decay f32, 6 r_last_epoch u32, 7 r_live u8, 8 r_depoch u32
void* okv_part_array(void* h, int32_t q, int32_t which) {
  Pool* p = static_cast<Pool*>(h);
  if (q < 0 || q >= p->n_parts) return nullptr;
  Part& pt = p->part[q];
  switch (which) {
    case 0: return pt.slab.data();
    case 1: return pt.ring.data();
    case 2: return pt.r_tag.data();
    case 3: return pt.r_pair.data();
    case 4: return pt.r_ema.data();
    case 5: return pt.r_decay.data();
    case 6: return pt.r_last_epoch.data();
    case 7: return pt.r_live.data();
    case 8: return pt.r_depoch.data();
    default: return nullptr;
  }
}

// info: 0 base, 1 n, 2 entry_bytes, 3 chunk_bytes, 4 n_chunks, 5 H, 6 R, 7 cursor
int64_t okv_part_info(void* h, int32_t q, int32_t which) {
  Pool* p = static_cast<Pool*>(h);
  if (q < 0 || q >= p->n_parts) return ERR_INVALID_ARG;
  const Part& pt = p->part[q];
  switch (which) {
    case 0: return pt.base;
    case 1: return pt.n;
    case 2: return pt.entry_bytes;
    case 3: return pt.chunk_bytes;
    case 4: return pt.n_chunks;
    case 5: return pt.H;
    case 6: return pt.R;
    case 7: return (int64_t)pt.cur;
    default: return ERR_INVALID_ARG;
  }
}

void okv_get_stats(void* h, uint64_t* out8) {
  Pool* p = static_cast<Pool*>(h);
  out8[0] = p->st.epochs;
  out8[1] = p->st.events;
  out8[2] = p->st.victims;
  out8[3] = p->st.promoted;
  out8[4] = p->st.admitted;
  out8[5] = p->st.bytes_demoted;
  out8[6] = p->st.bytes_promoted;
  out8[7] = p->st.bytes_dropped;
}

uint64_t okv_next_tag(void* h) { return static_cast<Pool*>(h)->next_tag; }

// The image of entry `id` as the host tier and the content hash see it: K chunk
// then V chunk (or the single MLA chunk).  out holds entry_bytes; returns that
// size, or a negative status (payload mode only).
int64_t okv_entry_image(void* h, uint32_t id, uint8_t* out) {
  Pool* p = static_cast<Pool*>(h);
  if (!p->payload || (int64_t)id >= p->N || !out) return ERR_INVALID_ARG;
  const Part& pt = p->part[part_of(*p, id)];
  copy_entry_to_image(pt, (int64_t)id - pt.base, out);
  return pt.entry_bytes;
}

// Lazy decay of promoted entries: off (default) restores the EMA verbatim.
int32_t okv_set_lazy_decay(void* h, int32_t on) {
  static_cast<Pool*>(h)->lazy_decay = on ? 1 : 0;
  return OK;
}

// Eviction policy: 0 Bayesian (default), 1 EMA only, 2 LRU.
int32_t okv_set_policy(void* h, int32_t policy) {
  if (policy < 0 || policy > 2) return ERR_INVALID_ARG;
  static_cast<Pool*>(h)->policy = policy;
  return OK;
}

// Confidence-weighted blend; window == 0 switches it off.  Resets the window.
int32_t okv_set_confidence_blend(void* h, float kappa, int32_t window) {
  Pool* p = static_cast<Pool*>(h);
  if (window < 0 || window > 64 || (window > 0 && !(kappa > 0.0f))) return ERR_INVALID_ARG;
  p->kappa = kappa;
  p->window = window;
  p->win_head = 0;
  p->win.assign((size_t)window * 32, 0);
  for (int i = 0; i < 32; ++i) p->wsum[i] = 0;
  return OK;
}

// The 16 reuse estimates used by the Bayesian score (the posterior, or its blend).
float* okv_estimate(void* h) { return static_cast<Pool*>(h)->estimate; }

// Head-granular importance (head-granular eviction section).  The paper keeps a
// [layer][head] importance matrix per model, an EMA updated on every attention
// step; for GQA the query heads that share a KV head are grouped and the group's
// maximum is the KV head's score; for MLA the matrix is [layer][1]; and at task
// transitions per-head multipliers bias eviction.  Recurrence and the way the
// matrix enters the eviction score are not printed [reading]:
//   M[l][j] <- d*M[l][j] + (1-d)*x[l][j]      for every query head j (binary32,
//                                              each operation rounded once);
//   W[l][h] = max_{j in group(h)} M[l][j] * mult[l][h];
//   score of entry (l, block, h) = (policy score) * W[l][h]   (Bayesian, EMA only).
// M starts at 1 and multipliers at 1, and a partition's scores are weighted only
// after the first call for it, so a pool that never calls this is unchanged.
// x: QH*L observations (>= 0, finite), row-major [layer][query head].
int32_t okv_head_importance_update(void* h, int32_t q, const float* x, float d) {
  Pool* p = static_cast<Pool*>(h);
  if (q < 0 || q >= p->n_parts || !x || !(d >= 0.0f) || !(d <= 1.0f)) return ERR_INVALID_ARG;
  Part& pt = p->part[q];
  const int64_t n = pt.L * pt.QH;
  for (int64_t i = 0; i < n; ++i)
    if (!(x[i] >= 0.0f) || !(x[i] <= std::numeric_limits<float>::max())) return ERR_INVALID_ARG;
  for (int64_t i = 0; i < n; ++i) {
    float t1 = d * pt.h_imp[(size_t)i];
    float t2 = 1.0f - d;
    float t3 = t2 * x[i];
    pt.h_imp[(size_t)i] = t1 + t3;
  }
  pt.head_weights = true;
  recompute_head_weights(pt);
  return OK;
}

// Task-transition multipliers of partition q: L*H values (>= 0, finite), row-major
// [layer][KV head]; NULL resets them to 1.
int32_t okv_set_head_multipliers(void* h, int32_t q, const float* mult) {
  Pool* p = static_cast<Pool*>(h);
  if (q < 0 || q >= p->n_parts) return ERR_INVALID_ARG;
  Part& pt = p->part[q];
  const int64_t n = pt.L * pt.H;
  if (mult)
    for (int64_t i = 0; i < n; ++i)
      if (!(mult[i] >= 0.0f) || !(mult[i] <= std::numeric_limits<float>::max())) return ERR_INVALID_ARG;
  for (int64_t i = 0; i < n; ++i) pt.h_mult[(size_t)i] = mult ? mult[i] : 1.0f;
  pt.head_weights = true;
  recompute_head_weights(pt);
  return OK;
}

// Per-layer prefetch window (RoPE-aware prefetching section: when a sequence is at
// position n, blocks covering positions [n, n+w] are promoted ahead of use, and the
// window w adapts per layer -- narrow for local-attention layers, wide for
// global-attention layers).  The paper prints neither how w adapts nor its unit
// [reading]:
//   S[l] <- d*S[l] + (1-d)*x[l]      x[l] = attention span observed in layer l this
//                                    step, in tokens (binary32, each operation
//                                    rounded once); S starts at 2,048 tokens;
//   w[l] = min(w_max, max(1, ceil(S[l] / block_tokens)))   blocks.
// x: L observations (>= 0, finite).
int32_t okv_prefetch_window_update(void* h, int32_t q, const float* x, float d) {
  Pool* p = static_cast<Pool*>(h);
  if (q < 0 || q >= p->n_parts || !x || !(d >= 0.0f) || !(d <= 1.0f)) return ERR_INVALID_ARG;
  Part& pt = p->part[q];
  for (int64_t l = 0; l < pt.L; ++l)
    if (!(x[l] >= 0.0f) || !(x[l] <= std::numeric_limits<float>::max())) return ERR_INVALID_ARG;
  for (int64_t l = 0; l < pt.L; ++l) {
    float t1 = d * pt.pf_span[(size_t)l];
    float t2 = 1.0f - d;
    float t3 = t2 * x[l];
    pt.pf_span[(size_t)l] = t1 + t3;
  }
  recompute_windows(pt);
  return OK;
}

// Sets every layer's span to `tokens` (>= 0, finite) and the cap to max_blocks (>= 1).
int32_t okv_set_prefetch_window(void* h, int32_t q, float tokens, uint32_t max_blocks) {
  Pool* p = static_cast<Pool*>(h);
  if (q < 0 || q >= p->n_parts || !(tokens >= 0.0f) || !(tokens <= std::numeric_limits<float>::max()) ||
      max_blocks < 1)
    return ERR_INVALID_ARG;
  Part& pt = p->part[q];
  pt.pf_max = max_blocks;
  for (int64_t l = 0; l < pt.L; ++l) pt.pf_span[(size_t)l] = tokens;
  recompute_windows(pt);
  return OK;
}

// which: 0 spans (float [L]), 1 windows (uint32 [L])
void* okv_prefetch_array(void* h, int32_t q, int32_t which) {
  Pool* p = static_cast<Pool*>(h);
  if (q < 0 || q >= p->n_parts) return nullptr;
  Part& pt = p->part[q];
  return which == 0 ? (void*)pt.pf_span.data() : which == 1 ? (void*)pt.pf_win.data() : nullptr;
}

// The prefetch list of one sequence (same section): table[(pb*L + l)*H + h] is the
// block handle (tag) of the sequence's block at position-block pb, layer l, KV head h,
// for pb in [0, n_pos).  With the sequence at position-block pos0, layer l wants the
// w[l] blocks at distance 0 .. w[l]-1 from pos0: pb = pos0 + dist when dir > 0 (the
// positions [n, n+w] the prefetcher requests), pb = pos0 - dist when dir < 0 (the
// positions [n-w, n] the section names as the likeliest to be read next) [reading: the
// section gives both ranges; the caller picks].  Those blocks that sit in the host tier
// are listed by their ring slot, ordered by (distance, layer, head).  Handles that are
// not cached (dropped, never admitted, >= n_tags) or already in HBM are skipped.
// Writes at most max_out slots; *count receives how many qualified (more than max_out:
// the list was cut).
int32_t okv_prefetch_list(void* h, int32_t q, const uint32_t* table, uint64_t n_pos, uint64_t pos0,
                          int32_t dir, uint64_t* out, uint64_t max_out, uint64_t* count) {
  Pool* p = static_cast<Pool*>(h);
  if (q < 0 || q >= p->n_parts || !count || dir == 0 || (n_pos > 0 && !table)) return ERR_INVALID_ARG;
  if (n_pos > 0 && pos0 >= n_pos) return ERR_INVALID_ARG;
  Part& pt = p->part[q];
  uint64_t n = 0;
  for (uint64_t dist = 0; n_pos > 0; ++dist) {
    if (dir > 0 ? dist >= n_pos - pos0 : dist > pos0) break;  // left the table
    const uint64_t pb = dir > 0 ? pos0 + dist : pos0 - dist;
    bool any = false;   // some layer still wants this distance
    for (int64_t l = 0; l < pt.L; ++l) {
      if (dist >= pt.pf_win[(size_t)l]) continue;
      any = true;
      for (int64_t hd = 0; hd < pt.H; ++hd) {
        const uint32_t t = table[(pb * (uint64_t)pt.L + (uint64_t)l) * (uint64_t)pt.H + (uint64_t)hd];
        if (t >= p->loc.size()) continue;
        const uint32_t where = p->loc[t];
        if (where == NONE || !(where & HOST_BIT)) continue;
        if (n < max_out && out) out[n] = where & ~HOST_BIT;
        ++n;
      }
    }
    if (!any) break;
  }
  *count = n;
  return OK;
}

// which: 0 importance matrix [L][QH], 1 multipliers [L][H], 2 weights [L][H]
float* okv_head_array(void* h, int32_t q, int32_t which) {
  Pool* p = static_cast<Pool*>(h);
  if (q < 0 || q >= p->n_parts) return nullptr;
  Part& pt = p->part[q];
  return which == 0 ? pt.h_imp.data() : which == 1 ? pt.h_mult.data() : which == 2 ? pt.h_w.data() : nullptr;
}

// One epoch of scoring, in the order update-then-decide:
//   1. every observed event adds one to alpha (reuse) or beta (miss) of the
//      entry's (block-type, transition-type) pair, and counts a touch;
//   2. the EMA of every resident entry advances by one step with the epoch's
//      touch count as its input [reading; the paper withholds the recurrence];
//   3. the posterior mean alpha/(alpha+beta) of Eq. "reuse" is formed per pair
//      from the prior plus the counts;
//   4. score = P(pair) * ema for resident entries [reading]; +inf marks
//      non-resident ones, which selection ignores.
int32_t okv_epoch_score(void* h, uint32_t epoch, const uint32_t* ev_entry, const uint8_t* ev_hit,
                        uint64_t n_events) {
  Pool* p = static_cast<Pool*>(h);
  if (n_events > 0 && (!ev_entry || !ev_hit)) return ERR_INVALID_ARG;
  for (uint64_t e = 0; e < n_events; ++e) {
    if ((int64_t)ev_entry[e] >= p->N || p->state[ev_entry[e]] != ST_RESIDENT)
      return ERR_INVALID_ARG;
  }
  p->cur_epoch = epoch;
  // step 1
  uint64_t epoch_hits[16] = {0}, epoch_misses[16] = {0};
  for (uint64_t e = 0; e < n_events; ++e) {
    uint32_t i = ev_entry[e];
    uint8_t pr = p->pair[i];
    if (ev_hit[e]) { p->hits[pr] += 1; epoch_hits[pr] += 1; } else { p->misses[pr] += 1; epoch_misses[pr] += 1; }
    p->touch[i] += 1;
  }
  // step 2
  for (int64_t i = 0; i < p->N; ++i) {
    if (p->state[i] != ST_RESIDENT) continue;
    float d = p->decay[i];
    float x = (float)p->touch[i];
    float t1 = d * p->ema[i];
    float t2 = 1.0f - d;
    float t3 = t2 * x;
    p->ema[i] = t1 + t3;
    if (p->touch[i] > 0) p->last_epoch[i] = epoch;
    p->touch[i] = 0;
  }
  // step 3
  for (int pr = 0; pr < 16; ++pr) {
    float a = p->alpha0 + (float)p->hits[pr];
    float b = p->beta0 + (float)p->misses[pr];
    p->P[pr] = a / (a + b);
  }
  // step 3b (optional): confidence-weighted blend of the posterior with the
  // empirical hit frequency of the last `window` epochs (this one included).
  // The paper describes it in words only (confidence saturates toward 1 with
  // observations; well-observed pairs rely on the posterior, young ones on the
  // windowed frequency) [reading]: c = n/(n+kappa), n = hits+misses;
  // f = window hits / window observations (the posterior itself if the window
  // is empty); estimate = c*P + (1-c)*f.
  if (p->window > 0) {
    uint64_t* slot = &p->win[(size_t)p->win_head * 32];
    for (int pr = 0; pr < 16; ++pr) {
      p->wsum[2 * pr] = p->wsum[2 * pr] - slot[2 * pr] + epoch_misses[pr];
      p->wsum[2 * pr + 1] = p->wsum[2 * pr + 1] - slot[2 * pr + 1] + epoch_hits[pr];
      slot[2 * pr] = epoch_misses[pr];
      slot[2 * pr + 1] = epoch_hits[pr];
    }
    p->win_head = (p->win_head + 1) % p->window;
  }
  for (int pr = 0; pr < 16; ++pr) {
    if (p->window == 0) { p->estimate[pr] = p->P[pr]; continue; }
    float n = (float)(p->hits[pr] + p->misses[pr]);
    float c = n / (n + p->kappa);
    float wh = (float)p->wsum[2 * pr + 1];
    float wn = (float)(p->wsum[2 * pr + 1] + p->wsum[2 * pr]);
    float f = wn > 0.0f ? wh / wn : p->P[pr];
    float t1 = c * p->P[pr];
    float t2 = 1.0f - c;
    float t3 = t2 * f;
    p->estimate[pr] = t1 + t3;
  }
  // step 4: the policy's score.  0 = Bayesian (reuse estimate x EMA importance),
  // 1 = EMA only, 2 = LRU (epoch of the last touch): the paper's three-way
  // comparison of eviction policies.
  for (int64_t i = 0; i < p->N; ++i) {
    if (p->state[i] != ST_RESIDENT) {
      p->score[i] = std::numeric_limits<float>::infinity();
    } else if (p->policy == 2) {
      p->score[i] = (float)p->last_epoch[i];
    } else {
      float sc = (p->policy == 1) ? p->ema[i] : p->estimate[p->pair[i]] * p->ema[i];
      // step 4b (optional): the importance of the entry's (layer, KV head), see
      // okv_head_importance_update; recency-only LRU ignores it
      const Part& pt = p->part[part_of(*p, i)];
      if (pt.head_weights) {
        int64_t local = i - pt.base;
        int64_t layer = local / (pt.NB * pt.H), head = local % pt.H;
        sc = sc * pt.h_w[(size_t)(layer * pt.H + head)];
      }
      p->score[i] = sc;
    }
  }
  p->st.epochs += 1;
  p->st.events += n_events;
  return OK;
}

// The k resident entries that come first in the total order (score, id),
// reported in ascending id order.  This is the definition written out: sort
// everything, cut at k.
int32_t okv_select_victims(void* h, uint64_t k, uint32_t* out_victims) {
  Pool* p = static_cast<Pool*>(h);
  std::vector<uint32_t> ids;
  for (int64_t i = 0; i < p->N; ++i)
    if (p->state[i] == ST_RESIDENT) ids.push_back((uint32_t)i);
  if (k > ids.size()) return ERR_K_TOO_LARGE;
  if (k > 0 && !out_victims) return ERR_INVALID_ARG;
  const std::vector<float>& s = p->score;
  // ids are ascending, and a stable sort keeps that order among equal scores.
  std::stable_sort(ids.begin(), ids.end(), [&s](uint32_t a, uint32_t b) { return s[a] < s[b]; });
  std::vector<uint32_t> v(ids.begin(), ids.begin() + (ptrdiff_t)k);
  std::sort(v.begin(), v.end());
  for (uint64_t j = 0; j < k; ++j) out_victims[j] = v[j];
  return OK;
}

// Block-granular selection (head-granular eviction section: "eviction selects
// the block with the lowest weighted aggregate importance score across heads,
// using architecture-dependent head weights (uniform for MHA, proportional to
// group size for GQA)").  Reading: the aggregate of block (layer, block) is
// w * (s_0 + s_1 + ... + s_{H-1}) over its KV-head entries, summed in head order
// in binary32, with w = query heads per KV-head entry (1 for MHA, the group size
// for GQA, h_q for MQA and MLA), so that blocks of different architectures are
// compared per query head.  A block is a candidate only if all its heads are
// RESIDENT.  The k_blocks candidates first in the order (aggregate, partition,
// layer, block) are chosen; the output lists all their entries, ascending.
// n_out receives the number of entries written.
int32_t okv_select_victim_blocks(void* h, uint64_t k_blocks, uint32_t* out_victims, uint64_t* n_out) {
  Pool* p = static_cast<Pool*>(h);
  struct Blk { float agg; int q; int64_t first; };  // first = id of head 0
  std::vector<Blk> blks;
  for (int q = 0; q < p->n_parts; ++q) {
    const Part& pt = p->part[q];
    int64_t hq = pt.d.model.n_q_heads > 0 ? pt.d.model.n_q_heads : pt.H;
    float w = (float)(hq / pt.H > 0 ? hq / pt.H : 1);
    for (int64_t lb = 0; lb < pt.L * pt.NB; ++lb) {
      int64_t first = pt.base + lb * pt.H;
      bool all = true;
      float sum = 0.0f;
      for (int64_t hd = 0; hd < pt.H; ++hd) {
        if (p->state[first + hd] != ST_RESIDENT) { all = false; break; }
        sum = sum + p->score[first + hd];
      }
      if (all) blks.push_back(Blk{w * sum, q, first});
    }
  }
  if (k_blocks > blks.size()) return ERR_K_TOO_LARGE;
  // blks is in (partition, layer, block) order; a stable sort keeps it among equal aggregates
  std::stable_sort(blks.begin(), blks.end(), [](const Blk& a, const Blk& b) { return a.agg < b.agg; });
  std::vector<uint32_t> v;
  for (uint64_t j = 0; j < k_blocks; ++j)
    for (int64_t hd = 0; hd < p->part[blks[j].q].H; ++hd) v.push_back((uint32_t)(blks[j].first + hd));
  std::sort(v.begin(), v.end());
  if (!v.empty() && !out_victims) return ERR_INVALID_ARG;
  for (size_t j = 0; j < v.size(); ++j) out_victims[j] = v[j];
  if (n_out) *n_out = v.size();
  return OK;
}

// Demotion of a victim list (ascending ids) into the per-partition host rings.
// The j-th victim of a partition goes to ring slot (cursor + j) mod R; a live
// slot that is overwritten is dropped (there is no tier below the host here).
int32_t okv_demote(void* h, const uint32_t* victims, uint64_t m) {
  Pool* p = static_cast<Pool*>(h);
  if (m > 0 && !victims) return ERR_INVALID_ARG;
  uint64_t kq[4] = {0, 0, 0, 0};
  for (uint64_t j = 0; j < m; ++j) {
    uint32_t v = victims[j];
    if ((int64_t)v >= p->N || p->state[v] != ST_RESIDENT) return ERR_INVALID_ARG;
    if (j > 0 && victims[j - 1] >= v) return ERR_INVALID_ARG;  // ascending, distinct
    kq[part_of(*p, v)] += 1;
  }
  for (int q = 0; q < p->n_parts; ++q)
    if (kq[q] > (uint64_t)p->part[q].R) return ERR_HOST_TIER_TOO_SMALL;
  uint64_t jq[4] = {0, 0, 0, 0};
  for (uint64_t j = 0; j < m; ++j) {
    uint32_t v = victims[j];
    int q = part_of(*p, v);
    Part& pt = p->part[q];
    uint64_t slot = (pt.cur + jq[q]) % (uint64_t)pt.R;
    jq[q] += 1;
    if (pt.r_live[slot]) {
      p->loc[pt.r_tag[slot]] = NONE;
      p->st.bytes_dropped += (uint64_t)pt.entry_bytes;
    }
    if (p->payload)
      copy_entry_to_image(pt, (int64_t)v - pt.base, pt.ring.data() + slot * (uint64_t)pt.entry_bytes);
    pt.r_tag[slot] = p->tag[v];
    pt.r_pair[slot] = p->pair[v];
    pt.r_ema[slot] = p->ema[v];
    pt.r_decay[slot] = p->decay[v];
    pt.r_last_epoch[slot] = p->last_epoch[v];
    pt.r_depoch[slot] = p->cur_epoch;
    pt.r_live[slot] = 1;
    p->loc[p->tag[v]] = HOST_BIT | (uint32_t)slot;
    p->state[v] = ST_FREE;
    p->tag[v] = NONE;
    p->st.bytes_demoted += (uint64_t)pt.entry_bytes;
  }
  for (int q = 0; q < p->n_parts; ++q)
    if (p->part[q].R > 0) p->part[q].cur = (p->part[q].cur + kq[q]) % (uint64_t)p->part[q].R;
  p->st.victims += m;
  return OK;
}

// Promotion: the j-th listed host slot goes to the j-th lowest FREE entry of
// the partition; its metadata is restored as it was when demoted.  With lazy
// decay on (okv_set_lazy_decay) the EMA first catches up on the scoring passes
// it missed: a resident entry that nobody touches goes ema <- decay*ema + (1 -
// decay)*0 = decay*ema per pass, so a block demoted in epoch e_d and promoted
// after the pass of epoch e_p takes e_p - e_d such steps, one rounded multiply
// each [reading: the paper does not say what happens to importance while a block
// is in a lower tier].
int32_t okv_promote(void* h, int32_t q, const uint64_t* slots, uint64_t m) {
  Pool* p = static_cast<Pool*>(h);
  if (q < 0 || q >= p->n_parts) return ERR_INVALID_ARG;
  if (m > 0 && !slots) return ERR_INVALID_ARG;
  Part& pt = p->part[q];
  std::vector<uint8_t> seen((size_t)pt.R, 0);
  for (uint64_t j = 0; j < m; ++j) {
    if (slots[j] >= (uint64_t)pt.R || !pt.r_live[slots[j]] || seen[slots[j]]) return ERR_BAD_HOST_SLOT;
    seen[slots[j]] = 1;
  }
  std::vector<int64_t> free_ids;
  for (int64_t i = pt.base; i < pt.base + pt.n; ++i)
    if (p->state[i] == ST_FREE) free_ids.push_back(i);
  if (m > free_ids.size()) return ERR_NO_FREE_SLOT;
  for (uint64_t j = 0; j < m; ++j) {
    uint64_t slot = slots[j];
    int64_t f = free_ids[j];
    if (p->payload)
      copy_image_to_entry(pt, f - pt.base, pt.ring.data() + slot * (uint64_t)pt.entry_bytes);
    p->pair[f] = pt.r_pair[slot];
    p->ema[f] = pt.r_ema[slot];
    if (p->lazy_decay && p->cur_epoch > pt.r_depoch[slot]) {
      // one untouched EMA step per scoring pass the block sat out on the host
      const uint32_t missed = p->cur_epoch - pt.r_depoch[slot];
      for (uint32_t s = 0; s < missed; ++s) p->ema[f] = pt.r_decay[slot] * p->ema[f];
    }
    p->decay[f] = pt.r_decay[slot];
    p->last_epoch[f] = pt.r_last_epoch[slot];
    p->tag[f] = pt.r_tag[slot];
    p->touch[f] = 0;
    p->state[f] = ST_RESIDENT;
    p->loc[pt.r_tag[slot]] = (uint32_t)f;
    pt.r_live[slot] = 0;
    pt.r_tag[slot] = NONE;
    p->st.bytes_promoted += (uint64_t)pt.entry_bytes;
  }
  p->st.promoted += m;
  return OK;
}

// Admission (harness step that keeps the pool full so that eviction pressure
// is real): every FREE entry, ascending, receives a fresh tag, the next pair
// id of new_pairs, a zero EMA and, in payload mode, the next entry image of
// new_payload (entry_bytes each, K chunk then V chunk, back to back in
// admission order).  Returns the number admitted or a negative status.
int64_t okv_admit(void* h, uint32_t epoch, float decay, const uint8_t* new_pairs, uint64_t n_pairs,
                  const uint8_t* new_payload) {
  Pool* p = static_cast<Pool*>(h);
  uint64_t n_free = 0;
  for (int64_t i = 0; i < p->N; ++i) n_free += (p->state[i] == ST_FREE);
  if (n_free > n_pairs) return ERR_INVALID_ARG;
  if (n_free > 0 && !new_pairs) return ERR_INVALID_ARG;
  if (p->next_tag + n_free > p->loc.size()) return ERR_TAGS_EXHAUSTED;
  for (uint64_t t = 0; t < n_free; ++t)
    if (new_pairs[t] > 15) return ERR_INVALID_ARG;
  uint64_t j = 0;
  uint64_t off = 0;
  for (int q = 0; q < p->n_parts; ++q) {
    Part& pt = p->part[q];
    for (int64_t i = pt.base; i < pt.base + pt.n; ++i) {
      if (p->state[i] != ST_FREE) continue;
      uint32_t t = (uint32_t)p->next_tag++;
      p->tag[i] = t;
      p->pair[i] = new_pairs[j];
      p->ema[i] = 0.0f;
      p->decay[i] = decay;
      p->last_epoch[i] = epoch;
      p->touch[i] = 0;
      p->state[i] = ST_RESIDENT;
      p->loc[t] = (uint32_t)i;
      if (p->payload && new_payload) copy_image_to_entry(pt, i - pt.base, new_payload + off);
      off += (uint64_t)pt.entry_bytes;
      ++j;
    }
  }
  p->st.admitted += j;
  return (int64_t)j;
}

}  // extern "C"
