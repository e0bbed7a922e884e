// Internal declarations shared by the kvtier translation units.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "kvtier.h"

namespace kvt {

constexpr int kThreads = 256;
constexpr uint32_t kRadixBits1 = 11, kRadixBits2 = 11, kRadixBits3 = 10;
constexpr uint32_t kHistBins = 2048;  // bins of the widest digit
constexpr uint32_t kTileEntries = 2048;  // entries per compaction tile (256 threads x 8)
// Bit 7 of an entry's pair byte is set while the entry is FREE, so that the event
// reduction learns both the pair and the state from one gathered byte.
constexpr uint32_t kPairFree = 0x80u;

// Kernels launched by this library in this process (all pools).
extern std::atomic<uint64_t> g_kernel_launches;
inline void count_launches(uint64_t n) { g_kernel_launches.fetch_add(n, std::memory_order_relaxed); }

// Streaming multiprocessors of the current device (148 on a B200); grids are sized in
// multiples of it.  Asked of the runtime at every launch: the answer belongs to the
// device that is current, not to the process.
inline int sm_count() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
    (void)cudaGetLastError();
    return 1;
  }
  return n;
}

// Geometry of one partition, as the kernels need it.
struct PartGeom {
  uint8_t* slab;         // device
  uint64_t base;         // first global id
  uint64_t n;            // entries
  uint32_t heads;        // KV heads per block (1 for MLA)
  uint32_t n_chunks;     // 2 (K, V) or 1 (MLA)
  uint32_t chunk_bytes;  // bytes of one contiguous chunk in the slab
  uint32_t entry_bytes;  // n_chunks * chunk_bytes
  uint32_t ring_slots;
  // device mirror of per-ring-slot metadata
  uint32_t* r_tag;
  uint32_t* r_last_epoch;
  float* r_ema;
  float* r_decay;
  uint8_t* r_pair;
  uint32_t* r_depoch;    // epoch in which the slot's block was demoted
  uint32_t epoch_now;    // epoch of the pool's last scoring pass (set by the host before a launch)
  uint32_t lazy_decay;   // promotion applies the EMA steps missed on the host
};

// EMA of a block that sat out `missed` scoring passes untouched: every pass is
// ema <- decay*ema + (1 - decay)*0 = decay*ema, one rounded multiply.  Stops early
// at a fixed point (0, decay 1, or a denormal that no longer shrinks), where
// further steps change nothing.
__device__ __forceinline__ float ema_catch_up(float ema, float decay, uint32_t missed) {
  for (uint32_t s = 0; s < missed; ++s) {
    const float nx = __fmul_rn(decay, ema);
    if (nx == ema) break;
    ema = nx;
  }
  return ema;
}

// Per-entry state arrays.
//
struct EntryState {
  float* ema;
  float* decay;
  uint32_t* touch;
  uint32_t* last_epoch;
  uint8_t* pair;
  uint8_t* state;
  uint32_t* tag;
  float* score;
  uint64_t n;
};

// Small block of device scalars used by selection and compaction.
struct SelectScalars {
  uint32_t prefix;        // key bits fixed so far
  uint32_t tau;           // key of the k-th smallest entry
  unsigned long long k_rem;    // rank still to resolve inside the current bucket
  unsigned long long need_eq;  // how many entries with key == tau are taken
  unsigned int bar_arrive;     // grid barrier of the persistent selection: arrivals
  unsigned int bar_done;       // ... and CTAs that have left (the last one resets both)
  unsigned int update_ticket;  // blocks of the entry pass that have finished (the last one commits)
  unsigned int hint_valid;     // the persistent selection left a usable hint
  uint32_t hint_tau;           // where the next persistent selection centres its bracket ...
  uint32_t hint_last;          // (tau of the last one)
  unsigned long long hint_n;   // ... and the number of keys it ran over
  unsigned long long below;    // keys below the bracket (accumulated per launch, cleared inside it)
  unsigned long long phase_ns[16]; // %globaltimer at the phase boundaries of the last persistent selection (CTA 0)
  // how the persistent selections went so far (kv_selection_stats)
  unsigned int n_select;       // selections run
  unsigned int n_hint_hit;     // ... whose hint's bracket held rank k
  unsigned int n_hint_miss;    // ... whose hint's bracket did not
  unsigned int n_reread;       // CTAs (over all selections) that had to re-read their keys although the hint held
  // persistent selection on a pool of several partitions: (below tau, equal to tau) counts of
  // the entries before partition boundary q + 1 inside the slice of the CTA that holds it
  uint2 bsplit[3];
  // width of the next selection's bracket: its 2,048 bins are 2^hint_shift keys wide (7..11);
  // hint_resid is a slowly decaying maximum of how far tau landed from where the hint put it
  uint32_t hint_shift;
  uint32_t hint_resid;
};

// Sliding window of per-epoch (pair, hit) counts for the confidence-weighted
// blend of the reuse estimate, and the estimates themselves.
constexpr uint32_t kMaxWindow = 64;
struct BlendState {
  unsigned long long wsum[32];              // sums over the window, index 2*pair + hit
  unsigned long long win[kMaxWindow * 32];  // ring of per-epoch counts
  float estimate[16];                       // reuse estimate used by the Bayesian score
  uint32_t head;                            // ring slot the next epoch overwrites
  uint32_t pad;
};

// Host-chosen options of the scoring pass.
struct ScoreOptions {
  int policy = 0;       // 0 Bayesian, 1 EMA only, 2 LRU
  float kappa = 0.0f;   // confidence saturation constant
  uint32_t window = 0;  // epochs in the sliding window; 0 = no blending
};

// Paged blocks (layer, block) of all partitions in one index space, for
// block-granular selection.
struct BlockGeom {
  uint64_t block_base[5];   // first global block index of each partition; [n_parts] = total
  uint64_t entry_base[4];   // first global entry id of each partition
  uint32_t heads[4];        // KV-head entries per block
  float weight[4];          // query heads per KV-head entry
  int n_parts;
};

// Head-granular importance (head-granular eviction section): per partition a
// [layer][query head] importance matrix, [layer][KV head] multipliers and the
// resulting [layer][KV head] score weights, each partition's block at its offset.
struct HeadWeights {
  float* imp;              // importance matrices, partition q at imp_off[q]
  float* mult;             // multipliers, partition q at w_off[q]
  float* w;                // weights, partition q at w_off[q]
  uint64_t base[5];        // first global entry id of each partition; [n_parts] = N
  uint32_t per_layer[4];   // entries per layer: blocks per layer x KV heads
  uint32_t heads[4];       // KV heads (1 for MLA)
  uint32_t q_heads[4];     // tracked query heads per layer (1 for MLA)
  uint32_t layers[4];
  uint32_t imp_off[4], w_off[4];
  uint32_t on;             // bit q: scores of partition q are weighted
  int n_parts;
};

// Per-layer prefetch windows (RoPE-aware prefetching section): per partition the EMA of
// the observed attention span in tokens and the window in blocks derived from it.
constexpr uint32_t kPrefetchChunks = 1024;   // most blocks of one prefetch-list launch
struct PrefetchState {
  float* span;             // [layers] per partition, partition q at off[q]
  uint32_t* win;           // same layout
  uint32_t* chunk_counts;  // [kPrefetchChunks] scratch of the list kernels
  uint32_t off[4], layers[4], heads[4];
  uint32_t block_tokens[4];
  uint32_t w_max[4];       // cap on the window, blocks
};

struct Workspace {
  BlendState* blend;
  float* block_score;       // [blocks] aggregate score per paged block
  uint8_t* block_state;     // [blocks] RESIDENT iff every head of the block is
  uint32_t* block_victims;  // [blocks] selected global block indices
  unsigned long long* delta;   // [32] per-epoch (pair, hit) counts: index pair*2+hit
  uint32_t* hist;              // [3][kHistBins]
  SelectScalars* sel;
  uint32_t* status;            // device status word
  uint2* tile_counts;          // [n_tiles] (less, equal) or (free, 0)
  uint2* tile_offsets;         // [n_tiles] exclusive prefix of tile_counts
  uint32_t* free_list;         // [max(N, ..)] ascending ids of FREE entries
  uint32_t* slot_list[8];      // [max_promote] promote lists (ring slots), used in turn
  unsigned long long* part_counts;  // [4] victims per partition
  uint32_t n_tiles;
  // One of the state arrays kept in the persisting part of the L2 (kv_set_l2_residency):
  // the scoring kernels are launched with this access-policy window.  bytes == 0: none.
  const void* l2_base = nullptr;
  size_t l2_bytes = 0;
  float l2_ratio = 0.0f;
};

// Launches fn (kernel taking the arguments in args) with the workspace's L2 window, if it has
// one, as a launch attribute; cooperative launches carry that attribute too.
inline cudaError_t launch_scoring_kernel(const void* fn, dim3 grid, dim3 block, void** args, size_t smem,
                                         cudaStream_t s, bool cooperative, const Workspace& ws) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  unsigned n = 0;
  if (cooperative) {
    attr[n].id = cudaLaunchAttributeCooperative;
    attr[n].val.cooperative = 1;
    ++n;
  }
  if (ws.l2_bytes) {
    attr[n].id = cudaLaunchAttributeAccessPolicyWindow;
    attr[n].val.accessPolicyWindow.base_ptr = const_cast<void*>(ws.l2_base);
    attr[n].val.accessPolicyWindow.num_bytes = ws.l2_bytes;
    attr[n].val.accessPolicyWindow.hitRatio = ws.l2_ratio;
    attr[n].val.accessPolicyWindow.hitProp = cudaAccessPropertyPersisting;
    attr[n].val.accessPolicyWindow.missProp = cudaAccessPropertyNormal;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelExC(&cfg, fn, args);
}

// ---- kv_score.cu ----
cudaError_t launch_event_reduce(const uint32_t* ev_entry, const uint8_t* ev_hit, uint64_t n_events,
                                const EntryState& st, const Workspace& ws, cudaStream_t s);
// posterior (from hits/misses plus the epoch counters in ws.delta) + EMA + score in one launch;
// folds ws.delta into hits/misses, clears it and writes P
cudaError_t launch_entry_update(const EntryState& st, uint64_t* hits, uint64_t* misses, float* P,
                                float alpha0, float beta0, const Workspace& ws, uint32_t epoch,
                                const ScoreOptions& opt, const HeadWeights& hw, cudaStream_t s);
// kv_heads.cu: mode 0 = EMA step of partition q's importance matrix with observations
// src [L][QH]; mode 1 = multipliers of q from src [L][H] (nullptr: all 1).  Both then
// recompute q's weights.  Values that are negative or not finite are skipped and flagged.
cudaError_t launch_head_update(const HeadWeights& hw, int q, int mode, const float* src, float decay,
                               const Workspace& ws, cudaStream_t s);
cudaError_t launch_head_init(const HeadWeights& hw, uint32_t n_imp, uint32_t n_w, cudaStream_t s);
// kv_prefetch.cu: mode 0 = EMA step of partition q's per-layer span with observations x [L]
// (any negative or non-finite value: nothing changes, flagged); mode 1 = every span = tokens.
// Both recompute the windows.
cudaError_t launch_prefetch_window(const PrefetchState& pf, int q, int mode, const float* x, float decay,
                                   float tokens, const Workspace& ws, cudaStream_t s);
// ring slots of the host-tier blocks of table [n_pos][L][H] inside the windows around
// position-block pos0, ordered by (distance, layer, head); *count = how many qualified
cudaError_t launch_prefetch_list(const PrefetchState& pf, int q, const uint32_t* table, uint64_t n_pos,
                                 uint64_t pos0, int dir, const uint32_t* loc, uint64_t n_tags,
                                 unsigned long long* out, uint64_t max_out, unsigned long long* count,
                                 cudaStream_t s);
// empties the sliding window of the blend (the estimates stay as they are)
cudaError_t launch_blend_reset(const Workspace& ws, cudaStream_t s);

// ---- kv_select.cu ----
// Where the victims of a selection fall: partition bases (global entry ids; [n_parts] = N),
// and where the per-partition victim counts go (device, and host memory the device can
// write, or nullptr).
struct PartCounts {
  unsigned long long base[5] = {0, 0, 0, 0, 0};
  int n_parts = 1;
  unsigned long long* d_counts = nullptr;   // [4]
  unsigned long long* h_counts = nullptr;   // [4] device-visible address of pinned host memory
};
// variant 1 = one persistent cooperative launch (falls back to 0 where the device cannot run
// it or the slices are too long), 0 = one launch per phase of the radix select
cudaError_t launch_select(const EntryState& st, uint64_t k, uint32_t* d_victims, const Workspace& ws,
                          cudaStream_t s, int variant = 1, const PartCounts* pc = nullptr);
// kv_select_persist.cu: the same selection as one cooperative launch; *used tells
// whether it was launched (false: the device cannot co-schedule it, nothing was enqueued)
// With fs the launch also does the entry pass first (posterior, EMA, score; the
// epoch's events have been reduced by an earlier launch).
struct FusedScore {
  uint64_t* hits;
  uint64_t* misses;
  float* P;
  float alpha0, beta0;
  uint32_t epoch;
  ScoreOptions opt;
  HeadWeights hw;
};
cudaError_t launch_select_persistent(const EntryState& st, uint64_t k, uint32_t* d_victims,
                                     const Workspace& ws, cudaStream_t s, bool* used,
                                     const FusedScore* fs = nullptr, const PartCounts* pc = nullptr);
// kv_blocks.cu: k_blocks lowest blocks by weighted aggregate score; writes all their entries
// (ascending) to d_victims, the per-partition block counts to ws.part_counts and the
// per-partition ENTRY counts to h_entry_counts (host memory the device can write; may be nullptr)
cudaError_t launch_select_blocks(const EntryState& st, const BlockGeom& bg, uint64_t k_blocks,
                                 uint32_t* d_victims, const Workspace& ws, cudaStream_t s,
                                 unsigned long long* h_entry_counts);
// ascending ids of FREE entries in [lo, hi), at most `limit` of them, into ws.free_list + out_offset
cudaError_t launch_free_list(const EntryState& st, uint64_t lo, uint64_t hi, uint64_t limit,
                             const Workspace& ws, cudaStream_t s, uint64_t out_offset = 0);
// victims per partition of an ascending list into pc.d_counts (and pc.h_counts)
cudaError_t launch_partition_counts(const uint32_t* d_victims, uint64_t m, const PartCounts& pc,
                                    cudaStream_t s);

// ---- kv_dedup.cu ----
// SHA-256 of the images of entries ids[0..m) (ids == nullptr: entries 0..m-1), 32 bytes each
cudaError_t launch_hash_entries(const PartGeom* parts, int n_parts, const uint32_t* ids, uint64_t m,
                                uint8_t* digests, const Workspace& ws, cudaStream_t s);
// first position per digest and reference counts; table_slots is a power of two >= 2*m
cudaError_t launch_dedup(const uint8_t* digests, uint64_t m, uint32_t* canon, uint32_t* refcount,
                         uint32_t* table, uint64_t table_slots, uint32_t* n_unique, uint32_t* status,
                         cudaStream_t s);

// ---- kv_move.cu ----
cudaError_t launch_init(const EntryState& st, uint64_t* hits, uint64_t* misses, float* P, float p0,
                        uint32_t* loc, uint64_t n_tags, const PartGeom* parts, int n_parts,
                        const Workspace& ws, cudaStream_t s);
// ---- kv_move_tma.cu: gather (demotion) and scatter (promotion) on the bulk asynchronous copy engine ----
// pack: victims[0 .. count) of one partition into staging (images back to back) followed, at
// meta_offset, by kv_slot_meta records; also moves the metadata.
// mode: 0 = metadata and payload, 1 = metadata only (staging unused), 2 = payload only
// (the metadata moved earlier; host-mirror records are rebuilt from the ring mirror)
cudaError_t launch_pack_tma(const PartGeom& g, const EntryState& st, uint32_t* loc, const uint32_t* victims,
                            uint64_t count, uint64_t ring_start, uint8_t* staging, uint64_t meta_offset,
                            const Workspace& ws, cudaStream_t s, uint32_t mode = 0);
// unpack: staging images [0, count) into the listed free slots of the partition
cudaError_t launch_unpack_tma(const PartGeom& g, const EntryState& st, uint32_t* loc, const uint32_t* slots,
                              const uint32_t* free_ids, uint64_t count, const uint8_t* staging,
                              const Workspace& ws, cudaStream_t s);
// the same scatter with the entries fetched by the kernel itself from the pinned ring (ring_dev:
// the address at which the device sees it): for lists of short runs
cudaError_t launch_gather_promote(const PartGeom& g, const EntryState& st, uint32_t* loc, const uint32_t* slots,
                                  const uint32_t* free_ids, uint64_t count, const uint8_t* ring_dev,
                                  const Workspace& ws, cudaStream_t s);
// admits free_list[first .. first+count) of one partition
cudaError_t launch_admit(const PartGeom& g, const EntryState& st, uint32_t* loc, const uint32_t* free_ids,
                         uint64_t first, uint64_t count, uint64_t first_tag, const uint8_t* new_pairs,
                         uint32_t epoch, float decay, int fill_pattern, const Workspace& ws,
                         cudaStream_t s);

}  // namespace kvt
