/* kvtier.h -- C ABI of the per-epoch hot path of a predictive two-tier KV-cache
 * manager (paged HBM pool above a pinned-host ring), for NVIDIA B200 (sm_100a).
 *
 * Operations and where the paper defines them:
 *   kv_size_bytes      sizing section, Eq. "unified" (B(n) per attention
 *                      variant) and Eq. "total" (L * B(n))
 *   kv_epoch_score     Bayesian reuse section, Eq. "reuse" (Beta posterior mean
 *                      with +1 updates per reuse/miss) and head-granular
 *                      eviction section (EMA importance per (layer, head))
 *   kv_select_victims  head-granular eviction section ("lowest ... score")
 *   kv_demote          six-tier hierarchy section, Tier 1 (pinned host memory,
 *                      asynchronous DMA on CUDA streams)
 *   kv_promote         RoPE-aware prefetching section (asynchronous promotion
 *                      requests from lower tiers)
 *   kv_prefetch_list   same section (the blocks covering the next positions of a
 *                      sequence, inside a window that adapts per layer)
 * The paper withholds the EMA recurrence, the way the reuse probability and the
 * importance are combined, and the organisation of the host tier; the
 * definitions used here are stated at each function.
 *
 * Conventions
 *   - plain C; every pointer is marked (device), (pinned host) or (host);
 *   - the caller allocates ALL memory (device, pinned host) and the streams;
 *     the library allocates no device memory and never synchronises the device;
 *     GPU work is enqueued on the given streams and results are valid once the
 *     caller has synchronised them.  Use ONE compute stream for every call on a
 *     pool.  kv_demote and kv_promote each take a copy stream; give kv_promote a
 *     different one than kv_demote and the H2D copies of a promotion overlap the
 *     D2H copies of the demotion before it (the library orders the two streams
 *     wherever a promotion reads ring slots that a demotion is still writing,
 *     and the other way round); keep each call's copy stream the same over time;
 *   - device and pinned pointers must be 16-byte aligned;
 *   - functions return KV_OK (0) or a negative kv_status; on a negative status
 *     detected by the host no state has changed and nothing that changes state has
 *     been enqueued;
 *   - an entry is one head-granular KV block: physical slot (layer, block, head)
 *     of a partition, local id (layer*blocks_per_layer + block)*heads + head,
 *     global id = partition base + local id (partitions are laid end to end in
 *     the order given).  MLA partitions have heads = 1.
 */
#ifndef KVTIER_H
#define KVTIER_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef void* kv_stream_t; /* a cudaStream_t */
typedef struct kv_pool kv_pool;

typedef enum {
  KV_OK = 0,
  KV_ERR_INVALID_ARG = -1,
  KV_ERR_UNSUPPORTED_VARIANT = -2,
  KV_ERR_K_TOO_LARGE = -3,         /* k exceeds the number of resident entries */
  KV_ERR_NO_FREE_SLOT = -4,        /* fewer free HBM slots than entries to promote */
  KV_ERR_BAD_HOST_SLOT = -5,       /* promote list names a dead, duplicate or out-of-range slot */
  KV_ERR_HOST_TIER_TOO_SMALL = -6, /* more victims in one call than ring slots */
  KV_ERR_CUDA = -7,                /* a CUDA call failed; see kv_last_cuda_error */
  KV_ERR_INTERNAL = -8,            /* a kernel reported an inconsistency (kv_device_status) */
  KV_ERR_UNIMPLEMENTED = -9,
  KV_ERR_TAGS_EXHAUSTED = -10      /* admission would exceed n_tags */
} kv_status;

typedef enum { KV_AUTO = -1, KV_MHA = 0, KV_GQA = 1, KV_MQA = 2, KV_MLA = 3 } kv_variant_t;

/* Entry states and block-table encoding. */
#define KV_STATE_FREE 0u
#define KV_STATE_RESIDENT 1u
#define KV_NONE 0xFFFFFFFFu     /* no tag / block not cached */
#define KV_LOC_HOST 0x80000000u /* d_loc[tag]: bit 31 set = host ring slot in bits 0..30 */

/* Bits of the device status word (kv_device_status). */
#define KV_DEV_EVENT_BAD_ID 1u       /* an event named an id >= N */
#define KV_DEV_EVENT_NOT_RESIDENT 2u /* an event named a FREE entry (event skipped) */
#define KV_DEV_SELECT_MISMATCH 4u    /* selection wrote a count other than k */
#define KV_DEV_VICTIM_NOT_RESIDENT 8u
#define KV_DEV_BAD_INDEX 16u         /* an index was out of range and the access was skipped */
#define KV_DEV_WAIT_EXPIRED 32u      /* a bounded wait inside a kernel gave up */
#define KV_DEV_BAD_HEAD_VALUE 64u    /* a head observation or multiplier was negative or not finite */
#define KV_DEV_BAD_SPAN_VALUE 128u   /* an attention-span observation was negative or not finite */

typedef struct {
  int32_t variant;    /* kv_variant_t; KV_AUTO infers it from the fields below */
  int32_t n_layers;   /* L */
  int32_t n_q_heads;  /* h (h_q) */
  int32_t n_kv_heads; /* h_kv */
  int32_t head_dim;   /* d */
  int32_t d_latent;   /* MLA latent dimension (0 = not MLA) */
  int32_t d_rope;     /* MLA RoPE dimension */
  int32_t dtype_bits; /* precision p in bits: 16 = BF16, 8 = INT8, 4 = INT4 (p = 0.5) */
} kv_model_desc;

/* Bytes of KV cache for n_tokens tokens (sizing section, Eq. "unified"):
 *   MHA 2*h*d*p*n, GQA/MQA 2*h_kv*d*p*n, MLA (d_latent+d_rope)*p*n   per layer;
 * per_layer == 0 multiplies by n_layers (one sequence of Eq. "total").
 * KV_AUTO: a latent dimension selects MLA, else h_q == h_kv is MHA, h_kv == 1 is
 * MQA, 1 < h_kv < h_q is GQA (h_q == h_kv == 1 reports MHA; same bytes).
 * Returns bytes, or a negative kv_status (fields inconsistent with the variant,
 * or a size that is not a whole number of bytes).  Host only; no CUDA. */
int64_t kv_size_bytes(const kv_model_desc* model, int64_t n_tokens, int32_t per_layer);

/* The variant kv_size_bytes would use, or a negative kv_status. */
int32_t kv_infer_variant(const kv_model_desc* model);

/* Bytes of one entry: B(block_tokens) / kv heads (one head's K and V), or
 * B(block_tokens) for MLA, whose importance matrix collapses to one column.
 * Must come out a multiple of 16. */
int64_t kv_entry_bytes(const kv_model_desc* model, int32_t block_tokens);

/* Slab layout of a partition (PagedAttention-style paging, head-major inside a
 * block so that one head's K and V of a block are each one contiguous chunk):
 *   MHA/GQA/MQA: [layer][block][K,V][head][token][dim]   two chunks per entry
 *   MLA:         [layer][block][token][d_latent+d_rope]  one chunk per entry
 * Ring / staging image of an entry: K chunk then V chunk (or the MLA chunk),
 * entry_bytes long, entries back to back. */
typedef struct {
  kv_model_desc model;
  int32_t block_tokens;
  int32_t reserved;
  int64_t blocks_per_layer;
  void* d_slab;        /* (device) n_layers*blocks_per_layer*heads*entry_bytes */
  void* h_ring;        /* (pinned host) ring_slots*entry_bytes */
  uint64_t ring_slots; /* < 2^31 */
  void* h_meta;        /* (pinned host, optional, may be NULL) ring_slots records of
                          kv_slot_meta: metadata of the block last demoted into each slot */
} kv_partition_desc;

typedef struct {
  uint32_t tag;
  uint32_t last_epoch;
  float ema;
  float decay;
  uint32_t pair;
  uint32_t demote_epoch; /* epoch of the pool's last scoring pass when the block was demoted */
} kv_slot_meta; /* 24 bytes */

typedef struct {
  int32_t n_partitions; /* 1..4 */
  int32_t reserved;
  kv_partition_desc part[4];
  /* per-entry state, struct of arrays of length N in global id order (device) */
  float* d_ema;           /* EMA access score */
  float* d_decay;         /* EMA decay per entry */
  uint32_t* d_touch;      /* touches seen in the current epoch */
  uint32_t* d_last_epoch; /* epoch of the last touch */
  uint8_t* d_pair;        /* 4*block_type + transition_type, 0..15; the library sets bit 7
                             while the entry is FREE (the value is then meaningless) */
  uint8_t* d_state;       /* KV_STATE_* */
  uint32_t* d_tag;        /* logical handle of the block in the slot, KV_NONE if FREE */
  float* d_score;         /* eviction score, +inf for FREE entries */
  /* predictor (device) */
  uint64_t* d_hits;   /* [16] reuse events per pair  (alpha - alpha0) */
  uint64_t* d_misses; /* [16] miss events per pair   (beta - beta0) */
  float* d_P;         /* [16] posterior reuse probability */
  float alpha0, beta0; /* Beta prior, both > 0 */
  /* block table (device): d_loc[tag] = entry id, KV_LOC_HOST|ring slot, or KV_NONE */
  uint32_t* d_loc;
  uint64_t n_tags;
  /* four device staging buffers of staging_bytes each: [0],[1] double-buffer the
   * demotions, [2],[3] the promotions */
  void* d_staging[4];
  uint64_t staging_bytes;
  uint64_t max_promote; /* longest promote list this pool will be given */
  /* scratch of the sizes kv_workspace_bytes reports */
  void* d_workspace;
  uint64_t workspace_bytes;
  void* h_workspace; /* (pinned host) */
  uint64_t h_workspace_bytes;
} kv_pool_desc;

/* Scratch sizes for a pool description (pointer fields are ignored). */
int32_t kv_workspace_bytes(const kv_pool_desc* desc, uint64_t* dev_bytes, uint64_t* host_bytes);

/* Validates and copies the description, creates the library's CUDA events, and
 * enqueues on `stream` the initialisation of all state: every entry FREE, every
 * ring slot dead, counters zero, d_P = alpha0/(alpha0+beta0), d_loc = KV_NONE.
 * The pool must be destroyed before the caller frees the memory it was given. */
int32_t kv_pool_create(const kv_pool_desc* desc, kv_stream_t stream, kv_pool** out);
int32_t kv_pool_destroy(kv_pool* pool);

/* One epoch of scoring over every entry, update-then-decide:
 *  1. each event e (entry id d_ev_entry[e], flag d_ev_hit[e]) adds one to the
 *     reuse count (flag != 0) or the miss count of the entry's pair -- the
 *     alpha += 1 / beta += 1 update of the Bayesian reuse section -- and one to
 *     the entry's touch count;
 *  2. EMA step of every RESIDENT entry, in binary32 with each operation rounded
 *     once:  ema = decay*ema + (1-decay)*float(touch);  last_epoch = epoch if
 *     touched;  touch = 0.  [The paper names an EMA importance per (layer, head)
 *     but withholds its recurrence; this is the standard one.]
 *  3. P[p] = (alpha0+hits[p]) / (alpha0+hits[p] + beta0+misses[p])   (Eq. "reuse");
 *  4. score = P[pair]*ema for RESIDENT entries, +inf for FREE ones.  [The paper
 *     says in words that placement weighs reuse probability and importance; the
 *     product is this library's reading.]
 * d_ev_entry (device, u32[n_events]) and d_ev_hit (device, u8[n_events]) may be
 * NULL when n_events == 0.  An event on an id >= N or on a FREE entry is
 * skipped and sets a bit of the device status word. */
int32_t kv_epoch_score(kv_pool* pool, uint32_t epoch, const uint32_t* d_ev_entry,
                       const uint8_t* d_ev_hit, uint64_t n_events, kv_stream_t stream);

/* kv_epoch_score in two halves, for pools sharded over several GPUs (each GPU
 * holds its own entries; only the 16 pair counters are shared, since the
 * predictor keeps one Beta distribution per pair for the whole system):
 *   kv_epoch_events  step 1 only: adds this GPU's events to the epoch counters;
 *   kv_epoch_counts  device address of the 32 epoch counters (u64, index
 *                    2*pair + hit), to be summed over GPUs in place by the
 *                    caller's collective (e.g. one NCCL all-reduce of 256 bytes);
 *   kv_epoch_update  folds the epoch counters into d_hits/d_misses, clears them,
 *                    and runs steps 2-4.
 * kv_epoch_score(pool, ...) == kv_epoch_events(...) then kv_epoch_update(...). */
int32_t kv_epoch_events(kv_pool* pool, const uint32_t* d_ev_entry, const uint8_t* d_ev_hit,
                        uint64_t n_events, kv_stream_t stream);
uint64_t* kv_epoch_counts(kv_pool* pool);
int32_t kv_epoch_update(kv_pool* pool, uint32_t epoch, kv_stream_t stream);

/* Eviction policy used by step 4 of kv_epoch_score from the next call on: the
 * three policies the paper compares in its table of cache hit rates.
 *   KV_POLICY_BAYESIAN  score = reuse estimate of the pair x EMA importance (default)
 *   KV_POLICY_EMA       score = EMA importance alone ("pattern-aware")
 *   KV_POLICY_LRU       score = epoch of the last touch ("reactive") */
typedef enum { KV_POLICY_BAYESIAN = 0, KV_POLICY_EMA = 1, KV_POLICY_LRU = 2 } kv_policy_t;
int32_t kv_set_policy(kv_pool* pool, int32_t policy);

/* Confidence-weighted reuse estimate (Bayesian reuse section: a confidence score
 * that saturates toward 1 as observations accumulate weighs the posterior
 * against an empirical frequency over a sliding window of recent observations;
 * the paper gives no formula, the one used here is):
 *   n = hits + misses of the pair,  c = n / (n + kappa),
 *   f = hits / observations of the pair over the last `window` epochs (this
 *       epoch included; the posterior itself while the window is empty),
 *   estimate = c * P + (1 - c) * f          (binary32, each operation rounded once)
 * and the Bayesian score uses `estimate` in place of P.  window is 1..64 epochs;
 * window = 0 switches the blend off (default; estimate = P).  The call empties
 * the window (enqueued on `stream`) and takes effect from the next
 * kv_epoch_score.  d_P keeps holding the plain posterior of Eq. "reuse". */
int32_t kv_set_confidence_blend(kv_pool* pool, float kappa, int32_t window, kv_stream_t stream);

/* Device address of the 16 reuse estimates (f32) the Bayesian score used last. */
const float* kv_reuse_estimate(kv_pool* pool);

/* Head-granular importance (head-granular eviction section).  The paper keeps,
 * per model, a [layer][head] importance matrix as an exponential moving average
 * updated on every attention step; for GQA the query heads that share a KV head
 * form a group whose maximum is the KV head's score; for MLA the matrix is
 * [layer][1]; at task transitions per-head multipliers bias eviction.  It prints
 * no formula; the form used here, per partition q (one model):
 *   M[l][j] <- decay*M[l][j] + (1-decay)*x[l][j]     every query head j
 *                                 (binary32, each operation rounded once; M starts at 1)
 *   W[l][h] = max{ M[l][j] : j in group(h) } * mult[l][h]
 *             group(h) = query heads h*G .. h*G+G-1, G = n_q_heads / KV heads
 *             (G = 1 for MHA; MLA tracks one column per layer)
 *   score of entry (l, block, h) = policy score * W[l][h]   for KV_POLICY_BAYESIAN
 *             and KV_POLICY_EMA; KV_POLICY_LRU, pure recency, ignores the matrix.
 * A partition's scores are weighted from its first call of either function on;
 * a pool that never calls them computes exactly what it did before.
 *   kv_head_importance_update  d_x: device f32 [n_layers][n_q_heads] ([n_layers][1]
 *                              for MLA), observations >= 0; 0 <= decay <= 1.
 *   kv_set_head_multipliers    d_mult: device f32 [n_layers][KV heads], >= 0; NULL
 *                              resets all multipliers of the partition to 1.
 * Both are enqueued on `stream` and take effect for kernels enqueued after them
 * (use the stream of kv_epoch_score).  A value that is negative, NaN or infinite
 * is skipped (the element keeps its old value) and sets KV_DEV_BAD_HEAD_VALUE.
 * kv_head_importance / kv_head_weights: device addresses of M ([L][query heads])
 * and W ([L][KV heads]) of partition q. */
int32_t kv_head_importance_update(kv_pool* pool, int32_t q, const float* d_x, float decay,
                                  kv_stream_t stream);
int32_t kv_set_head_multipliers(kv_pool* pool, int32_t q, const float* d_mult, kv_stream_t stream);
const float* kv_head_importance(kv_pool* pool, int32_t q);
const float* kv_head_weights(kv_pool* pool, int32_t q);

/* Writes to d_victims (device, u32[k]) the k RESIDENT entries that come first in
 * the total order (score, global id), in ascending id order: the k lowest
 * scores, ties broken by lowest (partition, layer, block, head).
 * KV_ERR_K_TOO_LARGE if k exceeds the resident count (tracked on the host). */
int32_t kv_select_victims(kv_pool* pool, uint64_t k, uint32_t* d_victims, kv_stream_t stream);

/* kv_epoch_score followed by kv_select_victims with the per-entry pass and the
 * selection in ONE kernel: steps 2-4 of kv_epoch_score (Bayesian reuse section,
 * Eq. "reuse") hand every fresh score straight to the k-lowest selection, so the
 * scores are written once for the caller and never read back, and a launch
 * boundary disappears (two launches in all: the event reduction, then the rest).
 * State, d_victims and the device status word end up exactly as after the two
 * calls.  All arguments are checked before anything is enqueued: on an error
 * (including KV_ERR_K_TOO_LARGE) the epoch has NOT been scored.  k == 0 scores
 * only.  Where the device cannot keep the kernel's whole grid resident at once,
 * the separate kernels run one after the other instead. */
int32_t kv_epoch_score_select(kv_pool* pool, uint32_t epoch, const uint32_t* d_ev_entry,
                              const uint8_t* d_ev_hit, uint64_t n_events, uint64_t k,
                              uint32_t* d_victims, kv_stream_t stream);

/* Demotes the m entries listed in d_victims (device, ascending distinct ids of
 * RESIDENT entries, as kv_select_victims writes them): packs their K/V (or MLA)
 * chunks into the staging buffers in chunks of at most batch_bytes on `compute`,
 * and copies each chunk to the partition's host ring on `copy`.  The j-th victim
 * of a partition takes ring slot (cursor + j) mod ring_slots; a live slot that
 * is overwritten is dropped (d_loc of its tag becomes KV_NONE).  Each victim's
 * slot becomes FREE, its tag KV_NONE, and d_loc[tag] = KV_LOC_HOST | slot.
 * With more than one partition the host has to know how many victims fall in
 * each (ring slots are assigned on the host): kv_demote counts them with a small
 * read-only kernel and WAITS for the 32-byte answer (everything enqueued before it
 * on `compute` finishes first; the wait is counted in kv_stats.host_waits).
 * kv_demote_counted takes the counts from the caller and never waits: every
 * selection call of a pool with several partitions leaves them in pinned host
 * memory (kv_victim_counts), valid once the selection's stream has run -- a caller
 * that synchronises there anyway passes them on.  Single-partition pools never wait.
 * batch_bytes must be in [entry_bytes, staging_bytes - metadata room]; see
 * kv_max_batch_bytes. */
int32_t kv_demote(kv_pool* pool, const uint32_t* d_victims, uint64_t m, uint64_t batch_bytes,
                  kv_stream_t compute, kv_stream_t copy);
/* h_counts (host, 4 values): victims per partition, in partition order; their sum must be m. */
int32_t kv_demote_counted(kv_pool* pool, const uint32_t* d_victims, uint64_t m, const uint64_t* h_counts,
                          uint64_t batch_bytes, kv_stream_t compute, kv_stream_t copy);
/* Pinned host memory (4 values) that receives the victims per partition of the pool's
 * last kv_select_victims / kv_epoch_score_select / kv_select_victim_blocks (entries, not
 * blocks); written by the device, valid once that call's stream has run.  Only pools
 * with several partitions fill it. */
const uint64_t* kv_victim_counts(const kv_pool* pool);

/* Promotes the m host ring slots listed in h_host_slots (host, read during the
 * call; all live and distinct) into partition `partition`: runs of consecutive
 * slots are copied to staging on `copy`, and the j-th listed entry is scattered
 * into the j-th lowest FREE slot of the partition on `compute`, with the pair,
 * EMA, decay, last epoch and tag it had when demoted (the EMA decayed for the
 * passes it missed if kv_set_lazy_decay is on); the host slot dies. */
int32_t kv_promote(kv_pool* pool, int32_t partition, const uint64_t* h_host_slots, uint64_t m,
                   uint64_t batch_bytes, kv_stream_t compute, kv_stream_t copy);

/* Per-layer prefetch window and the prefetch list of a sequence (RoPE-aware
 * prefetching section).  The section states that with a sequence at position n the
 * prefetcher requests promotion of the blocks covering positions [n, n+w] (it also
 * names [n-w, n] as the range likeliest to be read next), and that the window w
 * adapts to the observed attention patterns: narrow for local-attention (early)
 * layers, wide for global-attention (later) layers.  It prints no formula; the form
 * used here, per partition q (one model):
 *   S[l] <- decay*S[l] + (1-decay)*x[l]    x[l] = attention span observed in layer l,
 *                                  in tokens (binary32, each operation rounded once;
 *                                  S starts at 2,048 tokens)
 *   w[l] = min(w_max, max(1, ceil(S[l] / block_tokens)))   blocks (w_max starts at 65,535)
 *   kv_prefetch_window_update  d_span: device f32 [n_layers], observations >= 0 and
 *                              finite; 0 <= decay <= 1.  If any observation is
 *                              negative, NaN or infinite the partition keeps all its
 *                              spans and KV_DEV_BAD_SPAN_VALUE is set.
 *   kv_set_prefetch_window     every span of the partition = tokens (>= 0, finite),
 *                              w_max = max_blocks (>= 1).
 *   kv_prefetch_span / kv_prefetch_window: device addresses of S (f32 [n_layers]) and
 *                              w (u32 [n_layers]) of partition q.
 * kv_prefetch_list: d_table (device, u32 [n_pos][n_layers][KV heads]; one column for
 * MLA) holds the block handles (tags) of one sequence, position-block by
 * position-block.  With the sequence at position-block pos0 (< n_pos), layer l wants
 * the w[l] blocks at distance 0 .. w[l]-1 from pos0, toward higher positions when
 * direction > 0 and toward lower ones when direction < 0, as far as the table reaches.
 * Of those, the blocks that sit in the host tier (d_loc[tag] has KV_LOC_HOST) are
 * written to d_out_slots (device-accessible u64 [max_out]) as ring slots, ordered by
 * (distance, layer, head): a list kv_promote accepts once it has been brought to the
 * host.  Handles >= n_tags, dropped or never admitted, and blocks already in HBM are
 * skipped.  *d_out_count (device-accessible u64) receives how many qualified; if that
 * exceeds max_out only the first max_out were written.  n_pos == 0 gives count 0.
 * Two small launches on `stream`, which first joins the pool's promotions in flight
 * (they write d_loc); call it on the pool's compute stream.  Calls of one pool share a
 * scratch array: do not run two of them concurrently on different streams. */
int32_t kv_prefetch_window_update(kv_pool* pool, int32_t q, const float* d_span, float decay,
                                  kv_stream_t stream);
int32_t kv_set_prefetch_window(kv_pool* pool, int32_t q, float tokens, uint32_t max_blocks,
                               kv_stream_t stream);
const float* kv_prefetch_span(kv_pool* pool, int32_t q);
const uint32_t* kv_prefetch_window(kv_pool* pool, int32_t q);
int32_t kv_prefetch_list(kv_pool* pool, int32_t q, const uint32_t* d_table, uint64_t n_pos,
                         uint64_t pos0, int32_t direction, uint64_t* d_out_slots, uint64_t max_out,
                         uint64_t* d_out_count, kv_stream_t stream);

/* How kv_promote moves the bytes.  Runs of consecutive ring slots in the list become
 * one DMA transfer each into a staging buffer, which the unpack kernel scatters; that
 * is right for long runs.  A list ordered by token position (RoPE-aware prefetching
 * section: blocks covering the next positions of a sequence, every layer of a block
 * in turn) names slots that lie far apart -- only a block's heads are neighbours in a
 * ring filled in (layer, block, head) order -- and breaks into runs of a few slots.
 * For a list whose runs average less than run_bytes the entries are instead fetched
 * by a kernel on the copy stream, through the device's view of the pinned ring, and
 * written straight into their slots.  Default 1 MiB (measured: a transfer per run costs
 * about 12 us on top of its bytes, the kernel fetches at about 28 GB/s, so they break
 * even near 0.8 MB per run); 0 = always per-run transfers. */
int32_t kv_set_gather_threshold(kv_pool* pool, uint64_t run_bytes);

/* L2 residency of a state array (off by default).  The event reduction scatters atomics
 * over the touch counts and gathers pair bytes, and the entry pass then streams both
 * arrays once more; between the two, and from one epoch to the next, the gigabytes that
 * the block movement sends through the L2 evict them.  With a budget > 0 the scoring
 * kernels (event reduction, entry pass, fused selection) are launched with an access-policy
 * window that keeps ONE array in the persisting part of the L2: the touch counts (4 B per
 * entry) when they fit the budget whole, else the pair bytes (1 B per entry), a fraction
 * of them if even those do not fit.  Measured on a B200 (126 MB L2): 47 MB of touch counts
 * resident take 20 us off a 150 us pass; 75 MB resident leave too little L2 for the
 * streaming entry pass and cost more than they save, hence the rule.  A budget of 3/8 of
 * the L2 is a good choice.  Results are bit for bit the same.
 * The call sets the persisting-L2 set-aside of the CUDA context (cudaLimitPersistingL2CacheSize)
 * to what it uses, a setting of the calling process's context, shared by everything in it;
 * budget_bytes == 0 switches the window off and sets the set-aside to 0.  Nothing is
 * enqueued; it takes effect for calls made after it.  kv_pool_destroy of a pool with a window
 * turns the context's persisting lines back into ordinary ones (the set-aside stays as it
 * is).  KV_ERR_UNIMPLEMENTED on devices without a persisting L2. */
int32_t kv_set_l2_residency(kv_pool* pool, uint64_t budget_bytes);

/* Lazy decay of promoted entries (off by default).  The head-granular eviction
 * section updates importance on every step for blocks in HBM; the paper does not
 * say what a block's importance is when it returns from a lower tier.  Off, the
 * EMA comes back exactly as it left.  On, kv_promote first applies the EMA steps
 * the block missed: a resident entry that nobody touches goes
 *   ema <- decay*ema + (1-decay)*0 = decay*ema
 * per scoring pass, so a block demoted after the pass of epoch e_d and promoted
 * after the pass of epoch e_p takes e_p - e_d such steps (binary32, one rounded
 * multiply each) and ends with exactly the EMA of an entry that stayed resident
 * and untouched.  "Epoch" is the one given to the pool's last kv_epoch_score /
 * kv_epoch_update / kv_epoch_score_select; each ring slot remembers it
 * (kv_slot_meta.demote_epoch).  Takes effect for promotions enqueued after the call. */
int32_t kv_set_lazy_decay(kv_pool* pool, int32_t on);

/* Content hashing (content-addressable deduplication section: blocks are indexed
 * by the SHA-256 hash of their content).  Writes to d_digests (device, 32 bytes
 * per entry, in the byte order the standard prints) the SHA-256 digest (FIPS
 * 180-4) of the image of each of the m entries listed in d_ids (device, u32 global
 * ids; NULL = entries 0..m-1): the entry's K chunk followed by its V chunk, or its
 * single MLA chunk, exactly the bytes kv_demote would send to the host ring.  The
 * entries need not be RESIDENT (a FREE slot's bytes are whatever was left there).
 * An id >= N sets KV_DEV_BAD_INDEX and leaves its digest unwritten. */
int32_t kv_hash_entries(kv_pool* pool, const uint32_t* d_ids, uint64_t m, uint8_t* d_digests,
                        kv_stream_t stream);

/* Deduplication by content hash (same section: when a new block's hash is already
 * in the store, a reference count is incremented instead of duplicating the block;
 * the paper keeps the store in a radix tree on the CPU, here it is an
 * open-addressing table on the GPU).  The m digests are taken as a list of blocks
 * entering the store in list order, so the first block with a given digest is the
 * stored copy:
 *   d_canon[j]    (device, u32[m]) position of the stored copy that block j refers
 *                 to; j itself if block j is the stored copy
 *   d_refcount[i] (device, u32[m]) references to stored copy i, itself included; 0
 *                 for blocks that are not stored
 *   d_n_unique    (device, optional) one u32: number of stored copies; the bytes
 *                 saved are (m - n_unique) * entry_bytes
 * The result does not depend on thread scheduling (the smallest position wins).
 * d_table (device) is scratch of table_slots u32, table_slots a power of two >=
 * kv_dedup_table_slots(m) = 2*m rounded up; d_status (device, one u32 the caller
 * zeroes) receives KV_DEV_* bits if the table was found inconsistent.  m < 2^32-1.
 * Pointers 16-byte aligned.  Needs no pool. */
uint64_t kv_dedup_table_slots(uint64_t m);
int32_t kv_dedup_digests(const uint8_t* d_digests, uint64_t m, uint32_t* d_canon, uint32_t* d_refcount,
                         uint32_t* d_table, uint64_t table_slots, uint32_t* d_n_unique,
                         uint32_t* d_status, kv_stream_t stream);

/* Block-granular selection (head-granular eviction section: eviction takes the
 * block with the lowest weighted aggregate importance across heads, with head
 * weights uniform for MHA and proportional to the group size for GQA).  The
 * aggregate of a paged block (layer, block) is w * (s_0 + ... + s_{H-1}) over the
 * scores of its H KV-head entries, added in head order in binary32, with w = query
 * heads per KV-head entry (1 for MHA, h_q/h_kv for GQA, h_q for MQA and MLA), so
 * that blocks of different architectures in one pool compare per query head.
 * Only blocks whose heads are all RESIDENT are candidates.  The k_blocks
 * candidates first in the order (aggregate, partition, layer, block) are chosen
 * and ALL their entries are written to d_victims (device, u32, room for
 * k_blocks x the largest head count), in ascending id order, ready for kv_demote.
 * *h_n_victims (host) receives the number of entries: known without waiting for
 * a single-partition pool; a pool with several partitions waits on the host for a
 * 32-byte readback (everything enqueued on `stream` before it finishes first) --
 * unless h_n_victims is NULL: then the call returns at once, and the entries per
 * partition are in kv_victim_counts once `stream` has run.
 * If k_blocks exceeds the number of candidate blocks (not known to the host) the
 * device status word gets KV_DEV_SELECT_MISMATCH. */
int32_t kv_select_victim_blocks(kv_pool* pool, uint64_t k_blocks, uint32_t* d_victims,
                                uint64_t* h_n_victims, kv_stream_t stream);

/* Selection for callers that cannot allocate (the paper has no counterpart; it
 * is a packaging of kv_select_victims, not another method).  A serving engine
 * that has given all device memory to its own pools, or code that runs where
 * cudaMalloc is off limits, has no workspace to hand to kv_pool_create.  This
 * call needs none: it takes the score and state arrays directly and keeps its
 * scratch (histograms, scalars, per-tile counts; about 58 KB) in a fixed array
 * inside the library, which every GPU that loads the library holds until the
 * process exits.  It calls no allocating routine.
 *   d_score  (device) f32[n]  eviction scores, as kv_epoch_score writes them
 *   d_state  (device) u8[n]   KV_STATE_*; only RESIDENT entries are candidates
 *   d_victims (device) u32[k] receives the k lowest (score, id) entries, ascending id
 *   d_status (device, optional) one u32 that receives KV_DEV_SELECT_MISMATCH if k
 *            exceeded the number of RESIDENT entries (the host cannot know that
 *            count here, so the caller must keep k within it); the caller zeroes it
 * Limits and rules:
 *   - n <= 4,194,304 entries; larger n returns KV_ERR_INVALID_ARG, k > n returns
 *     KV_ERR_K_TOO_LARGE; pointers must be 16-byte aligned;
 *   - the first call on each device looks up the array's device address (with
 *     that device current); make that first call before any stream capture;
 *   - all calls on a device share the one array, which is cleared at the start of
 *     each call: two calls whose GPU work overlaps (different streams, no
 *     ordering between them) race and give wrong results.  Order them. */
int32_t kv_select_victims_static(const float* d_score, const uint8_t* d_state, uint64_t n,
                                 uint64_t k, uint32_t* d_victims, uint32_t* d_status,
                                 kv_stream_t stream);

/* Deferred packing (off by default).  A demotion larger than two staging buffers
 * keeps the compute stream waiting for its own D2H copies, and a promotion
 * enqueued after it would only start unpacking when the demotion is nearly over.
 * With deferred packing on, kv_demote moves the metadata of ALL victims at once
 * (their slots become FREE immediately) and enqueues only the first two payload
 * chunks; the remaining chunks are enqueued by the NEXT call on the pool:
 * kv_promote interleaves them with its own chunks (a promoted entry only ever
 * lands in a freed slot whose payload has already been packed, because victims
 * and free slots are both taken in ascending id order), any other call enqueues
 * all that is left first.  Results are the same as without it.  The price is a
 * contract: d_victims must stay valid, and the caller's own kernels must not
 * write into the freed slots, until a later call on the pool has returned and its
 * work on `compute` has run. */
int32_t kv_set_deferred_packing(kv_pool* pool, int32_t on);

/* Enqueues (on the streams the demotion was given) whatever deferred packing still
 * holds back.  After it returns, synchronising those streams completes the
 * demotion, and d_victims may be reused once they have run.  A no-op otherwise. */
int32_t kv_flush(kv_pool* pool);

/* Largest batch_bytes the staging buffers allow for a partition. */
uint64_t kv_max_batch_bytes(const kv_pool* pool, int32_t partition);

/* Harness step, not part of the paper's method: fills every FREE slot, in
 * ascending id order, with a fresh block: tag = next unused handle, pair =
 * d_new_pairs[j] for the j-th admitted (device, u8, at least as many as there
 * are FREE slots), ema 0, the given decay, last_epoch = epoch, touch 0.  With
 * fill_pattern != 0 the block's bytes are set so that 8-byte word j of the entry
 * image holds SplitMix64(tag * 2^20 + j).  *n_admitted (host, optional)
 * receives the count, which the host knows without reading the device. */
int32_t kv_admit(kv_pool* pool, uint32_t epoch, float decay, const uint8_t* d_new_pairs,
                 uint64_t n_new_pairs, int32_t fill_pattern, uint64_t* n_admitted,
                 kv_stream_t stream);

typedef struct {
  uint64_t epochs, events, victims, promoted, admitted;
  uint64_t bytes_demoted, bytes_promoted, bytes_dropped;
  uint64_t n_entries, n_free;
  uint64_t kernel_launches; /* kernels launched by the library in this process so far */
  uint64_t host_waits;      /* times kv_demote, kv_promote or kv_select_victim_blocks blocked the host */
  uint64_t gathered;        /* entries promoted by the gather kernel instead of per-run transfers */
} kv_stats;

/* Host-side counters, kept eagerly at call time. */
int32_t kv_get_stats(const kv_pool* pool, kv_stats* out);

/* Host-side view of a partition's ring: cursor, and (optional) one byte per ring
 * slot, 1 = live.  h_live (host) must hold ring_slots bytes if not NULL. */
int32_t kv_ring_query(const kv_pool* pool, int32_t partition, uint64_t* cursor, uint64_t* n_live,
                      uint8_t* h_live);

/* Number of victims per partition of the last kv_demote (host, 4 values). */
int32_t kv_last_demote_counts(const kv_pool* pool, uint64_t* counts4);

/* Reads and clears the device status word (KV_DEV_* bits).  This one call
 * blocks the host until `stream` has drained. */
int32_t kv_device_status(kv_pool* pool, kv_stream_t stream, uint32_t* status_bits);

/* Measurement aid (no counterpart in the paper): when enabled, every pack and
 * unpack kernel launch is bracketed by two timing events on the stream it is
 * launched on.  kv_timing_read waits for the recorded launches to finish, adds
 * their durations up, reports the totals since the last read and resets them. */
typedef struct {
  double pack_ms, unpack_ms;            /* summed kernel durations */
  uint64_t pack_launches, unpack_launches;
  uint64_t pack_bytes, unpack_bytes;    /* payload bytes moved (read + written counted once each) */
  double gather_ms;                     /* the same for the gather kernel of kv_promote, which reads */
  uint64_t gather_launches, gather_bytes; /* the host ring itself: its time is the host link's */
} kv_timing;
int32_t kv_timing_enable(kv_pool* pool, int32_t on);
int32_t kv_timing_read(kv_pool* pool, kv_timing* out);

/* Measurement aid: how this pool's selections run from now on: 1 = one persistent
 * cooperative launch (default; falls back to 0 where the device cannot co-schedule it
 * or the pool has more than 262,144 entries per SM), 0 = one launch per phase of the
 * radix select. */
int32_t kv_set_select_variant(kv_pool* pool, int32_t variant);

/* Measurement aid: how the pool's persistent selections went so far.  Each starts from
 * a hint (the threshold of the selection before it): a hit means one short pass after
 * the scoring pass finished it, a miss that the keys were read again (two or three
 * passes); reread_ctas counts thread blocks that read their keys again although the
 * hint held (more keys near the threshold than they could note).  Blocks the host
 * until `stream` has drained. */
typedef struct {
  uint64_t selections, hint_hits, hint_misses, reread_ctas;
} kv_select_stats;
int32_t kv_selection_stats(kv_pool* pool, kv_stream_t stream, kv_select_stats* out);

/* The last CUDA error code seen by a call on this pool (0 = none). */
int32_t kv_last_cuda_error(const kv_pool* pool);

const char* kv_status_string(int32_t status);
const char* kv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* KVTIER_H */
