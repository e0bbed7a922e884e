// k-lowest selection as ONE cooperative, persistent launch.
//
// The multi-launch selection in kv_select.cu spends most of its time between
// kernels when the pool has a few million entries: ten dependent launches of
// 3-10 us each.  Here one CTA per SM stays resident for the whole selection.
// CTA g owns the chunks g, g + G, g + 2G, ... of the pool (4,096 entries each): a
// region of the pool that costs more than others -- many touched entries, many
// keys near the threshold -- is spread over all CTAs, and the one barrier that
// ends a phase waits for no overloaded CTA.  Bitmaps and notes index the CTA's
// entries by (local chunk, offset).  The phases of the selection are separated by
// grid-wide barriers instead of kernel boundaries:
//
//   A  every score becomes an order-preserving key (fused form: the entry pass
//      itself produces it) and enters the first histogram.  With a hint -- tau of
//      the previous selection -- the histogram covers a bracket of 2^18 .. 2^22 keys
//      around it (2,048 bins; the width follows how far tau moved lately); the
//      pass also leaves in shared memory a bitmap "key below the
//      bracket", and every thread notes the keys it saw inside the bracket
//      (typically 5-10 % of the slice) in a few private slots: no vote, no atomic.
//   B  the remaining histograms of the radix select.  When rank k falls inside
//      the bracket, ONE more histogram (the single keys of the bracket bin
//      that holds rank k, at most 2^11) finishes it, and it is built from the
//      noted keys alone: no second pass over the scores.  Otherwise (no hint, a miss, a thread that
//      ran out of slots) the keys are re-read from the score array, which then
//      sits mostly in L2, and the last histogram of that path leaves the bitmaps
//      "key below the final range" and "key inside the final range".
//   C  tau picked: the keys of the final range are sorted into "below tau" and
//      "equal to tau" -- from the notes, or, on the other path, by fetching just
//      the keys inside the range (not even those when the CTA's own histogram
//      shows that all of them equal tau: a tie, the usual case when few distinct
//      scores exist).
//   D  per-chunk counts = population counts of the two bitmaps, kept in a
//      pool-wide table; after the last barrier every CTA sums the table's rows
//      and knows how many victims precede each of its chunks; it writes its own
//      victims, chunk by chunk in ascending id order, straight from the bitmaps.
//
// The grid barrier is a counter in global memory that every CTA increments and
// then polls.  A cooperative launch guarantees that all CTAs are resident, so
// the wait ends; it is nevertheless bounded, and a CTA that gives up sets
// KV_DEV_WAIT_EXPIRED and leaves (every other CTA then runs into the same limit).
//
// The same kernel also exists fused with the per-entry scoring pass (FUSED =
// true): every CTA first updates the entries of its own chunks (posterior, EMA,
// score), their inputs streamed through shared-memory stages by asynchronous
// copies, and turns the fresh scores straight into keys -- a kernel boundary
// disappears.  The event reduction stays a launch of its own ahead of it: its
// scattered gathers and atomics ran 2.5x slower inside this kernel when that was
// tried, and a grid barrier costs about what the launch boundary does.
#include <mutex>
#include <type_traits>

#include "kv_score_device.cuh"

namespace kvt {

constexpr uint32_t kPThreads = 1024;
constexpr uint32_t kPChunk = kPThreads * 4;             // 4096 entries: one 16-byte vector per thread
constexpr uint32_t kPHistBins = 2048;
constexpr uint32_t kExcluded = 0xFFFFFFFFu;             // key of a non-candidate (FREE) entry
constexpr uint32_t kBarrierSpins = 1u << 22;
constexpr uint32_t kBracketShiftMax = 11;               // a bracket bin is at most 2^11 keys wide: the 2,048 bins then
                                                        // reach 2^21 keys to either side of the hint ...
constexpr uint32_t kBracketShiftMin = 7;                // ... and at least 2^7 (2^17 keys to either side)
constexpr uint32_t kPIdxBits = 18;                      // index of an entry inside its slice
constexpr uint32_t kPMaxSlice = 1u << kPIdxBits;        // entries per CTA the bitmaps are sized for (2 x 32 KB)
constexpr uint32_t kPMaxChunks = kPMaxSlice / kPChunk;  // chunks per CTA
// Fused form: the entry pass's inputs of one chunk in shared memory -- ema, decay and touch
// (4,096 words each), pair and state bytes (1,024 words each)
constexpr uint32_t kEntryStageWords = 3u * kPChunk + 2u * kPThreads;
constexpr uint32_t kEntryStages = 2;                    // chunks in flight ahead of the one being finished
constexpr uint32_t kPSlotsMin = 10;
constexpr uint32_t kPSlotsMax = 32;                     // bracket keys a thread can note (its private slots)


__device__ __forceinline__ uint32_t p_score_key(float s) {
  uint32_t b = __float_as_uint(s);
  if (b == 0x80000000u) b = 0u;  // -0.0 orders with +0.0
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Adds one to s_hist[bin] for every active lane.  When the warp agrees on the bin
// (the common case while many scores are equal) the addition is not even issued:
// the warp carries a pending (bin, count) pair, identical in all its lanes, and
// only a change of bin sends the count to shared memory.  Atomics of different
// warps on one hot address serialise at ~18 cycles each, which is what a pass
// over a heavily tied slice used to spend its time on.
struct WarpHist {
  uint32_t bin = 0, cnt = 0;
  // m = the warp's vote on `active` (every lane calls, with the same m)
  __device__ __forceinline__ void add_voted(uint32_t* s_hist, unsigned m, bool active, uint32_t b) {
    if (m == 0) return;
    const int leader = __ffs(m) - 1;
    const uint32_t b0 = __shfl_sync(0xFFFFFFFFu, b, leader);
    const bool same = !active || b == b0;
    if (__all_sync(0xFFFFFFFFu, same)) {
      if (b0 != bin) {
        flush(s_hist);
        bin = b0;
      }
      cnt += (uint32_t)__popc(m);
    } else if (active) {
      atomicAdd(&s_hist[b], 1u);
    }
  }
  __device__ __forceinline__ void add(uint32_t* s_hist, bool active, uint32_t b) {
    add_voted(s_hist, __ballot_sync(0xFFFFFFFFu, active), active, b);
  }
  __device__ __forceinline__ void flush(uint32_t* s_hist) {
    if (cnt && (threadIdx.x & 31u) == 0) atomicAdd(&s_hist[bin], cnt);
    cnt = 0;
  }
};

struct PArgs {
  const float* score;
  const uint8_t* state;
  unsigned long long n;
  unsigned long long k;
  uint32_t* victims;
  uint32_t* hist;         // [3][2048], zero on entry, zero again on exit
  SelectScalars* sel;
  uint2* chunk_counts;    // [total_chunks] (below tau, equal to tau) per chunk of the pool
  uint32_t total_chunks;  // chunks of 4,096 entries in the pool
  uint32_t* status;
  unsigned long long per; // most entries of a CTA: whole chunks, at most kPMaxSlice
  uint32_t words;         // 32-bit words of one bitmap of a slice (a multiple of 4)
  uint32_t slots;         // private slots per thread for keys inside the bracket (at least 10)
  uint32_t entry_stages;  // fused form: stages of the entry pass's inputs behind the slots (0: direct loads)
  PartCounts pc;          // partitions of the pool (the victims per partition are a by-product)
  uint32_t* spill;        // [n] global scratch for the notes a thread's slots cannot hold (nullptr: none)
  // the scoring pass of the fused form
  EntryState st;
  Predictor pd;
  HeadWeights hw;
  uint32_t epoch;
};

// Bounded grid-wide barrier; false if the wait ran out.
__device__ __forceinline__ bool grid_barrier(unsigned int* counter, unsigned int target) {
  __shared__ int s_ok;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(counter, 1u);
    int ok = 0;
    for (uint32_t it = 0; it < kBarrierSpins; ++it) {
      unsigned int v;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
      if (v >= target) { ok = 1; break; }
      __nanosleep(32);
    }
    s_ok = ok;
    __threadfence();
  }
  __syncthreads();
  return s_ok != 0;
}

// Block-wide exclusive scan over the 1024 threads; also returns the block total.
__device__ __forceinline__ uint32_t block_scan_excl(uint32_t v, uint32_t* s_warp, uint32_t& total) {
  const uint32_t t = threadIdx.x;
  uint32_t incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if ((t & 31u) >= (uint32_t)o) incl += y;
  }
  __syncthreads();  // s_warp may still be read by the previous call's consumers
  if ((t & 31u) == 31u) s_warp[t >> 5] = incl;
  __syncthreads();
  if (t < 32) {
    uint32_t w = s_warp[t];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, w, o);
      if (t >= (uint32_t)o) w += y;
    }
    s_warp[t] = w;
  }
  __syncthreads();
  total = s_warp[31];
  return incl - v + ((t >> 5) ? s_warp[(t >> 5) - 1] : 0u);
}

// Finds the bin of a global histogram (nbins <= 2048) that contains rank k_rem
// (1-based) and returns (bin, ranks before the bin) to every thread; bin is
// 0xFFFFFFFF when k_rem exceeds the histogram's total.
__device__ __forceinline__ void pick_bin(const uint32_t* __restrict__ hist, uint32_t nbins,
                                         unsigned long long k_rem, uint32_t* s_warp, uint32_t* s_pick,
                                         uint32_t& bin, uint32_t& before_bin) {
  const uint32_t t = threadIdx.x;
  const uint32_t b0 = 2 * t, b1 = 2 * t + 1;
  const uint32_t c0 = b0 < nbins ? __ldcg(&hist[b0]) : 0u;
  const uint32_t c1 = b1 < nbins ? __ldcg(&hist[b1]) : 0u;
  if (t == 0) { s_pick[0] = 0xFFFFFFFFu; s_pick[1] = 0; }
  uint32_t total;
  const uint32_t before = block_scan_excl(c0 + c1, s_warp, total);  // contains block barriers
  if (c0 && (unsigned long long)before < k_rem && k_rem <= (unsigned long long)before + c0) {
    s_pick[0] = b0; s_pick[1] = before;
  }
  const uint32_t before1 = before + c0;
  if (c1 && (unsigned long long)before1 < k_rem && k_rem <= (unsigned long long)before1 + c1) {
    s_pick[0] = b1; s_pick[1] = before1;
  }
  __syncthreads();
  bin = s_pick[0];
  before_bin = s_pick[1];
  __syncthreads();
}

// PLAIN (fused form only): the policy is the Bayesian product and no partition is weighted.
template <bool FUSED, bool PLAIN>
__global__ void __launch_bounds__(kPThreads, 1) select_persistent_kernel(const PArgs a) {
  extern __shared__ __align__(16) uint32_t s_dyn[];
  uint32_t* const s_bit_l = s_dyn;                    // bit j: key of local entry j is below tau
  uint32_t* const s_bit_e = s_bit_l + a.words;        // bit j: key of local entry j equals tau
  // [slot][thread]: (key - base0) | position in the vector << 22 | chunk << 24; later the
  // staging buffer of the ordered write
  uint32_t* const s_note = s_bit_e + a.words;
  // behind the slots: the stages of the fused entry pass; once phase A is over both together
  // are scratch (stages of the re-reading passes, staging of the ordered write)
  uint32_t* const s_entry = s_note + a.slots * kPThreads;
  const uint32_t scratch_words = a.slots * kPThreads + a.entry_stages * kEntryStageWords;
  __shared__ uint32_t s_hist[kPHistBins];
  __shared__ uint32_t s_warp[32];
  __shared__ uint32_t s_pick[2];
  __shared__ uint2 s_cex[kPMaxChunks + 1];    // (below, equal) counts the CTA holds before each of its chunks
  __shared__ uint2 s_cpre[kPMaxChunks];       // ... and the pool holds before them
  __shared__ uint32_t s_gstart[kPMaxChunks];  // where a chunk's victims start in the output
  __shared__ uint32_t s_lstart[kPMaxChunks + 1];  // ... and in the stage of the ordered write
  __shared__ uint2 s_rowtot[kPMaxChunks];     // totals of the rows of the chunk table, then the sums before each row
  __shared__ uint2 s_all;                     // the table's total
  __shared__ uint2 s_bnd[3];   // last CTA: (below tau, equal to tau) over the CTAs before each partition boundary's CTA
  __shared__ float sP[16];
  const uint32_t t = threadIdx.x;
  const uint32_t lane = t & 31u;
  unsigned int* bar = &a.sel->bar_arrive;
  const unsigned int G = gridDim.x;
  // The CTA's entries: chunks blockIdx.x, blockIdx.x + G, ... of the pool (4,096 entries each),
  // so that regions of the pool that cost more -- many touched entries, many keys near the
  // threshold -- are spread over all CTAs.  Local chunk c is pool chunk c * G + blockIdx.x; the
  // bitmaps and notes index entries by local position (chunk c, offset o) -> c * 4096 + o.
  const uint32_t n_chunks = a.total_chunks > blockIdx.x ? (a.total_chunks - blockIdx.x + G - 1u) / G : 0u;
  auto chunk_base = [&](uint32_t c) { return ((unsigned long long)c * G + blockIdx.x) * kPChunk; };
  // pool id of local entry j
  auto pool_id = [&](uint32_t j) { return chunk_base(j / kPChunk) + (j % kPChunk); };
  bool ok = true;
  // Phase boundaries of CTA 0 for timing studies (compiled in with -DKV_PHASE_STAMPS only: a
  // read of the global timer stalls the thread for a few hundred nanoseconds).
  auto stamp = [&](int i) {
#ifdef KV_PHASE_STAMPS
    if (blockIdx.x == 0 && t == 0) {
      unsigned long long ns;
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(ns));
      a.sel->phase_ns[i] = ns;
    }
#else
    (void)i;
#endif
  };
  stamp(0);

  // keys of the thread's vector (4 entries) of chunk c, computed from the arrays;
  // entries past the slice or not RESIDENT give kExcluded
  auto keys_from_arrays = [&](uint32_t c, uint32_t key[4]) {
    const unsigned long long i0 = chunk_base(c) + 4u * t;
    if (i0 + 4 <= a.n) {
      const float4 sc = __ldcg(reinterpret_cast<const float4*>(a.score + i0));
      const uchar4 st = __ldcg(reinterpret_cast<const uchar4*>(a.state + i0));
      key[0] = st.x == KV_STATE_RESIDENT ? p_score_key(sc.x) : kExcluded;
      key[1] = st.y == KV_STATE_RESIDENT ? p_score_key(sc.y) : kExcluded;
      key[2] = st.z == KV_STATE_RESIDENT ? p_score_key(sc.z) : kExcluded;
      key[3] = st.w == KV_STATE_RESIDENT ? p_score_key(sc.w) : kExcluded;
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j)
        key[j] = (i0 + j < a.n && a.state[i0 + j] == KV_STATE_RESIDENT) ? p_score_key(a.score[i0 + j])
                                                                        : kExcluded;
    }
  };
  // A pass over the slice's keys, re-read from the arrays: body(c, key) sees the thread's
  // four keys of every chunk c, last chunk first (the end of the slice is what the cache
  // hierarchy saw last), all threads in lock step (body may vote across the warp).  The
  // loads of kAhead chunks are issued before the first of them is used.
  constexpr uint32_t kAhead = 2;
  auto for_chunks = [&](auto body) {
    uint32_t c = n_chunks;
    while (c > 0) {
      const uint32_t nb = c < kAhead ? c : kAhead;
      float4 sc[kAhead];
      uchar4 st[kAhead];
#pragma unroll
      for (uint32_t u = 0; u < kAhead; ++u) {
        const unsigned long long i0 = u < nb ? chunk_base(c - 1u - u) + 4u * t : a.n;
        if (i0 + 4 <= a.n) {
          sc[u] = __ldcg(reinterpret_cast<const float4*>(a.score + i0));
          st[u] = __ldcg(reinterpret_cast<const uchar4*>(a.state + i0));
        }
      }
#pragma unroll
      for (uint32_t u = 0; u < kAhead; ++u) {
        if (u < nb) {
          const uint32_t cc = c - 1u - u;
          uint32_t key[4];
          if (chunk_base(cc) + 4u * t + 4 <= a.n) {
            key[0] = st[u].x == KV_STATE_RESIDENT ? p_score_key(sc[u].x) : kExcluded;
            key[1] = st[u].y == KV_STATE_RESIDENT ? p_score_key(sc[u].y) : kExcluded;
            key[2] = st[u].z == KV_STATE_RESIDENT ? p_score_key(sc[u].z) : kExcluded;
            key[3] = st[u].w == KV_STATE_RESIDENT ? p_score_key(sc[u].w) : kExcluded;
          } else {
            keys_from_arrays(cc, key);   // the ragged end of the slice
          }
          body(cc, key);
        }
      }
      c -= nb;
    }
  };
  // The same pass for the re-reads of phase B, where the threads' notes are dead: their
  // space becomes a ring of stages that asynchronous copies (global -> shared, no registers
  // in between) keep filled several chunks ahead.  A thread reads back only what it copied
  // itself, so waiting for its own copy groups is all the synchronisation there is.
  auto for_chunks_staged = [&](auto body) {
    constexpr uint32_t kStageWords = kPChunk + kPThreads;   // 4096 scores + 1024 state words
    const uint32_t n_stages = scratch_words / kStageWords;   // at least 2 (slots >= 10)
    const uint32_t depth = n_stages < 8u ? n_stages : 8u;
    auto issue = [&](uint32_t c, uint32_t stage) {
      const unsigned long long i0 = chunk_base(c) + 4u * t;
      if (i0 + 4 <= a.n) {
        uint32_t* dst = s_note + stage * kStageWords;
        const uint32_t d_sc = (uint32_t)__cvta_generic_to_shared(dst + 4u * t);
        const uint32_t d_st = (uint32_t)__cvta_generic_to_shared(dst + kPChunk + t);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d_sc), "l"(a.score + i0) : "memory");
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(d_st), "l"(a.state + i0) : "memory");
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    // chunks go last to first; chunk number n_chunks-1-i uses stage i % depth
    for (uint32_t i = 0; i < depth; ++i) {
      if (i < n_chunks) issue(n_chunks - 1u - i, i);
      else asm volatile("cp.async.commit_group;" ::: "memory");
    }
    for (uint32_t i = 0; i < n_chunks; ++i) {
      // all but the newest depth-1 groups are complete: the oldest one is chunk i's
      switch (depth) {
        case 2: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
        case 3: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
        case 4: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
        case 5: asm volatile("cp.async.wait_group 4;" ::: "memory"); break;
        case 6: asm volatile("cp.async.wait_group 5;" ::: "memory"); break;
        case 7: asm volatile("cp.async.wait_group 6;" ::: "memory"); break;
        default: asm volatile("cp.async.wait_group 7;" ::: "memory"); break;
      }
      const uint32_t c = n_chunks - 1u - i, stage = i % depth;
      uint32_t key[4];
      if (chunk_base(c) + 4u * t + 4 <= a.n) {
        const uint32_t* src = s_note + stage * kStageWords;
        const float4 sc = *reinterpret_cast<const float4*>(src + 4u * t);
        const uint32_t st4 = src[kPChunk + t];
        key[0] = (st4 & 0xFFu) == KV_STATE_RESIDENT ? p_score_key(sc.x) : kExcluded;
        key[1] = ((st4 >> 8) & 0xFFu) == KV_STATE_RESIDENT ? p_score_key(sc.y) : kExcluded;
        key[2] = ((st4 >> 16) & 0xFFu) == KV_STATE_RESIDENT ? p_score_key(sc.z) : kExcluded;
        key[3] = (st4 >> 24) == KV_STATE_RESIDENT ? p_score_key(sc.w) : kExcluded;
      } else {
        keys_from_arrays(c, key);   // the ragged end of the slice
      }
      // refill the stage with the chunk `depth` further on (an empty group keeps the count)
      if (i + depth < n_chunks) issue(n_chunks - 1u - (i + depth), stage);
      else asm volatile("cp.async.commit_group;" ::: "memory");
      body(c, key);
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
  };
  // Eight lanes x four bits (a lane holds 4 consecutive entries) -> the bitmap word of
  // the 32 entries starting at j0 of the lane with (lane & 7) == 0, which stores it.
  auto store_word = [&](uint32_t* bits, uint32_t nib, uint32_t j0) {
    uint32_t v = nib << (4u * (lane & 7u));
    v |= __shfl_xor_sync(0xFFFFFFFFu, v, 1);
    v |= __shfl_xor_sync(0xFFFFFFFFu, v, 2);
    v |= __shfl_xor_sync(0xFFFFFFFFu, v, 4);
    if ((lane & 7u) == 0 && (j0 >> 5) < a.words) bits[j0 >> 5] = v;
  };
  auto clear_hist = [&]() {
    for (uint32_t b = t; b < kPHistBins; b += kPThreads) s_hist[b] = 0;
    __syncthreads();
  };
  auto flush_hist = [&](uint32_t* g_hist, uint32_t nbins) {
    __syncthreads();
    for (uint32_t b = t; b < nbins; b += kPThreads) {
      const uint32_t c = s_hist[b];
      if (c) atomicAdd(&g_hist[b], c);
    }
  };
  // every thread owns a contiguous run of bitmap words inside one chunk (a chunk has 128 words;
  // the run is 1, 2, 4 or 8 words long)
  uint32_t wpt = 1;
  while (wpt * kPThreads < a.words) wpt <<= 1;
  const uint32_t w0 = t * wpt < a.words ? t * wpt : a.words;
  const uint32_t w1 = w0 + wpt < a.words ? w0 + wpt : a.words;

  if constexpr (FUSED) {
    // reuse estimates from the totals plus this epoch's counts (final: the event
    // reduction is an earlier launch)
    if (t < 16) {
      unsigned long long h, m, wh, wm;
      const float P = posterior(a.pd, t, h, m);
      sP[t] = reuse_estimate(a.pd, t, P, h, m, wh, wm);
    }
  }
  for (uint32_t w = t; w < 2 * a.words; w += kPThreads) s_bit_l[w] = 0;   // both bitmaps

  // ---- phase A: keys and the first histogram ----
  // Without a hint the first histogram is digit 0 of a plain radix select (bits
  // 31..21 of every key).  With a hint it covers only the bracket [base0, base0 +
  // 2,048 << bshift) around the hinted tau in 2,048 bins of 2^bshift keys (bshift 7..11); keys below base0 set
  // their bit in s_bit_l (and are counted), keys inside are noted: scores move
  // little from one epoch to the next, so the k-th key is almost always inside,
  // and then only the notes are looked at again.
  const bool hint = a.sel->hint_valid != 0 && a.sel->hint_n == a.n;
  const uint32_t hint_tau = a.sel->hint_tau;
  // The bracket's width follows how well the hints have been doing: 2,048 bins of 2^bshift keys.
  uint32_t bshift = a.sel->hint_shift;
  bshift = bshift < kBracketShiftMin ? kBracketShiftMin : (bshift > kBracketShiftMax ? kBracketShiftMax : bshift);
  const uint32_t bbits = bshift + 11u;                  // log2 of the bracket's width in keys
  const uint32_t bhalf = 1u << (bbits - 1u);
  // (the bracket [base0, base0 + 2^bbits) must end below the excluded key 0xFFFFFFFF)
  const uint32_t base_max = 0xFFFFFFFFu - (1u << bbits);
  const uint32_t base_c = hint_tau > bhalf ? hint_tau - bhalf : 0u;
  const uint32_t base0 = hint ? (base_c < base_max ? base_c : base_max) : 0u;
  const uint32_t shift0 = hint ? bshift : 21u;
  bool hint_hit = false;
  WarpHist wh;
  uint32_t n_noted = 0;   // keys of this thread inside the bracket
  uint32_t a_bin = 0, a_cnt = 0;   // ... and its pending count for one bin of the bracket's histogram
  // notes beyond the thread's slots: the CTA's stretch of the global scratch, laid out like the slots
  // (row r of 1,024 notes lives in the stretch of the scratch that belongs to local chunk r / 4:
  // a thread has noted at most four keys per chunk, so that chunk is already the CTA's own)
  uint32_t* const spill = a.spill;
  auto spill_at = [&](uint32_t r) { return spill + chunk_base(r >> 2) + (r & 3u) * kPThreads + t; };
  // body(v) for every note of the thread: the slots first, then the spilled ones, whose loads
  // (L2) are issued eight at a time before the first of them is used.  body may rewrite the
  // list in place at positions up to the note it has been given.
  auto for_notes = [&](auto body) {
    const uint32_t in_slots = n_noted < a.slots ? n_noted : a.slots;
    for (uint32_t i = 0; i < in_slots; ++i) body(s_note[i * kPThreads + t]);   // (read before body may overwrite slot <= i)
    const uint32_t n_all = n_noted;   // (body may shorten the list behind the note it is given)
    for (uint32_t r = 0; a.slots + r < n_all; r += 8u) {
      uint32_t v[8];
#pragma unroll
      for (uint32_t u = 0; u < 8u; ++u) v[u] = (a.slots + r + u < n_all) ? __ldcg(spill_at(r + u)) : 0xFFFFFFFFu;
#pragma unroll
      for (uint32_t u = 0; u < 8u; ++u)
        if (a.slots + r + u < n_all) body(v[u]);
    }
  };
  auto phase_a = [&](uint32_t c, const uint32_t key[4]) {
    if (!hint) {
#pragma unroll
      for (int q = 0; q < 4; ++q) wh.add(s_hist, key[q] != kExcluded, key[q] >> 21);
      return;
    }
    // A key lies inside the bracket iff (key - base0) >> bbits == 0: a key below base0 wraps
    // around to a large difference, and the bracket ends below the excluded key (base0 is
    // kept that far down).  The thread's in-bracket keys -- usually none or one of the four --
    // are then handled one after the other, so that a warp runs the body as often as its
    // busiest lane has such keys and not once per position.
    uint32_t nib_l = 0, in = 0;
    uint32_t d[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      d[q] = key[q] - base0;
      nib_l |= (uint32_t)(key[q] < base0) << q;
      in |= (uint32_t)((d[q] >> bbits) == 0u) << q;
    }
    while (in) {
      const uint32_t q = (in & 1u) ? 0u : (in & 2u) ? 1u : (in & 4u) ? 2u : 3u;
      in &= in - 1u;
      const uint32_t dq = q == 0u ? d[0] : q == 1u ? d[1] : q == 2u ? d[2] : d[3];
      // the histogram count waits in the thread while the bin stays the same (entries with
      // equal scores come in runs, and atomics of many threads on one hot bin serialise)
      const uint32_t bq = dq >> bshift;
      if (bq != a_bin) {
        if (a_cnt) atomicAdd(&s_hist[a_bin], a_cnt);
        a_bin = bq;
        a_cnt = 0;
      }
      ++a_cnt;
      const uint32_t note = dq | (q << 22) | (c << 24);
      if (n_noted < a.slots) s_note[n_noted * kPThreads + t] = note;
      else if (spill) *spill_at(n_noted - a.slots) = note;   // (a dense slice: the rest goes to L2)
      ++n_noted;
    }
    store_word(s_bit_l, nib_l, c * kPChunk + 4u * t);
  };
  clear_hist();
  if constexpr (FUSED) {
    // the slice's entries go through the EMA and score update on the way
    const int policy = PLAIN ? 0 : a.pd.policy;
    const uint32_t jt = 4u * t;
    // finishes the thread's vector of chunk c (entries j0 .. j0+3 of the slice, loaded into cur
    // when the whole vector lies inside the slice) and hands its keys to phase A
    auto finish_chunk = [&](uint32_t c, EntryVec& cur) {
      const unsigned long long i0 = chunk_base(c) + jt;
      uint32_t key[4] = {kExcluded, kExcluded, kExcluded, kExcluded};
      if (i0 + 4 <= a.n) {
        float4 sc;
        entry_finish4<PLAIN>(a.st, i0 / 4, cur, sP, policy, a.epoch, a.hw, sc);
        key[0] = cur.st.x == KV_STATE_RESIDENT ? p_score_key(sc.x) : kExcluded;
        key[1] = cur.st.y == KV_STATE_RESIDENT ? p_score_key(sc.y) : kExcluded;
        key[2] = cur.st.z == KV_STATE_RESIDENT ? p_score_key(sc.z) : kExcluded;
        key[3] = cur.st.w == KV_STATE_RESIDENT ? p_score_key(sc.w) : kExcluded;
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (i0 + j < a.n) {
            float sc;
            uint32_t s1;
            entry_update1(a.st, i0 + j, sP, policy, a.epoch, a.hw, sc, s1);
            if (s1 == KV_STATE_RESIDENT) key[j] = p_score_key(sc);
          }
        }
      }
      phase_a(c, key);
    };
    // Full chunks stream through shared-memory stages filled by asynchronous copies, two
    // chunks ahead of the one being finished: no registers hold data in flight, and the
    // thread reads back only what it copied itself, so its own copy groups are all it
    // waits for.  (The LRU policy also reads last_epoch, for which the stages have no
    // room: it takes the direct loads, like the ragged last chunk.)
    // (all of the CTA's chunks are full but the pool's last one, which may be ragged)
    const uint32_t n_full = (n_chunks && chunk_base(n_chunks - 1u) + kPChunk > a.n) ? n_chunks - 1u : n_chunks;
    const uint32_t n_staged = (a.entry_stages == kEntryStages && policy != 2) ? n_full : 0u;
    if (n_staged) {
      auto issue = [&](uint32_t c, uint32_t stage) {
        uint32_t* dst = s_entry + stage * kEntryStageWords;
        const unsigned long long i0 = chunk_base(c) + jt;
        const uint32_t d0 = (uint32_t)__cvta_generic_to_shared(dst + jt);
        const uint32_t d1 = (uint32_t)__cvta_generic_to_shared(dst + 3u * kPChunk + t);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d0), "l"(a.st.ema + i0) : "memory");
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d0 + 4u * kPChunk), "l"(a.st.decay + i0) : "memory");
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d0 + 8u * kPChunk), "l"(a.st.touch + i0) : "memory");
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(d1), "l"(a.st.pair + i0) : "memory");
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(d1 + 4u * kPThreads), "l"(a.st.state + i0) : "memory");
        asm volatile("cp.async.commit_group;" ::: "memory");
      };
      for (uint32_t i = 0; i < kEntryStages; ++i) {
        if (i < n_staged) issue(i, i);
        else asm volatile("cp.async.commit_group;" ::: "memory");
      }
      for (uint32_t c = 0; c < n_staged; ++c) {
        asm volatile("cp.async.wait_group 1;" ::: "memory");   // kEntryStages - 1 newer groups may be pending
        const uint32_t stage = c % kEntryStages;
        const uint32_t* src = s_entry + stage * kEntryStageWords;
        EntryVec cur;
        cur.e = *reinterpret_cast<const float4*>(src + jt);
        cur.d = *reinterpret_cast<const float4*>(src + kPChunk + jt);
        cur.t = *reinterpret_cast<const uint4*>(src + 2u * kPChunk + jt);
        cur.pr = *reinterpret_cast<const uchar4*>(src + 3u * kPChunk + t);
        cur.st = *reinterpret_cast<const uchar4*>(src + 3u * kPChunk + kPThreads + t);
        cur.le = make_uint4(0, 0, 0, 0);
        if (c + kEntryStages < n_staged) issue(c + kEntryStages, stage);
        else asm volatile("cp.async.commit_group;" ::: "memory");
        finish_chunk(c, cur);
      }
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    EntryVec cur;
    if (n_staged < n_chunks && chunk_base(n_staged) + jt + 4 <= a.n)
      cur = entry_load4(a.st, (chunk_base(n_staged) + jt) / 4, policy);
    for (uint32_t c = n_staged; c < n_chunks; ++c) {
      // the next chunk's loads fly while this one is finished
      EntryVec nxt;
      const unsigned long long i1 = c + 1 < n_chunks ? chunk_base(c + 1u) + jt : a.n;
      if (i1 + 4 <= a.n) nxt = entry_load4(a.st, i1 / 4, policy);
      finish_chunk(c, cur);
      cur = nxt;
    }
  } else {
    for_chunks(phase_a);
  }
  wh.flush(s_hist);
  // pending bracket counts: one atomic per bin value and warp
  for (;;) {
    const unsigned m = __ballot_sync(0xFFFFFFFFu, a_cnt != 0u);
    if (m == 0) break;
    const int leader = __ffs(m) - 1;
    const uint32_t b0 = __shfl_sync(0xFFFFFFFFu, a_bin, leader);
    const bool mine = a_cnt != 0u && a_bin == b0;
    uint32_t sum = mine ? a_cnt : 0u;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
    if ((int)lane == leader) atomicAdd(&s_hist[b0], sum);
    if (mine) a_cnt = 0;
  }
  flush_hist(a.hist, kPHistBins);   // (begins with a block barrier: the bitmap words are all written)
  if (hint) {
    uint32_t below = 0, cta_below0;
    for (uint32_t w = w0; w < w1; ++w) below += (uint32_t)__popc(s_bit_l[w]);
    (void)block_scan_excl(below, s_warp, cta_below0);
    if (t == 0 && cta_below0) atomicAdd(&a.sel->below, (unsigned long long)cta_below0);
  }
  // without the global scratch a thread that ran out of slots sends the whole CTA the long way
  // (its keys are re-read)
  const bool notes_complete = spill != nullptr || __syncthreads_or(n_noted > a.slots) == 0;
  if (!spill && n_noted > a.slots) n_noted = a.slots;
  stamp(1);
  ok = grid_barrier(bar, G);
  stamp(2);
  if (!ok) goto fail;
  if constexpr (FUSED) {
    // every CTA has formed its estimates: the epoch's counts can be folded in
    if (blockIdx.x == 0 && t < 16) commit_predictor(a.pd, t);
  }

  {
    // ---- phase B: narrow [base, base + 2^shift) around rank k, one histogram per step ----
    // The current histogram is a.hist[h]; it was built over [base, base + 2048 << shift).
    // Every CTA reads the same global data, so all of them take the same path.
    uint32_t h = 0, nbar = 1, base = base0, shift = shift0;
    unsigned long long k_rem = a.k;
    uint32_t bin, before;
    bool found = true;
    bool clear_below = hint;
    bool use_notes = false;   // rank k is inside the hint's bracket and this CTA noted all its bracket keys
    auto hist_pass = [&](uint32_t width_log2, uint32_t new_shift, uint32_t h_new) {
      // histogram of ((key - base) >> new_shift) over the keys in [base, base + 2^width_log2)
      clear_hist();
      const uint32_t top = width_log2 - new_shift;  // log2 of the number of bins
      WarpHist w2;
      if (new_shift != 0) {
        for_chunks_staged([&](uint32_t, const uint32_t key[4]) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint32_t d = key[q] - base;
            w2.add(s_hist, key[q] != kExcluded && key[q] >= base && ((d >> new_shift) >> top) == 0u,
                   d >> new_shift);
          }
        });
      } else if (use_notes) {
        // the last histogram (single keys of the bracket bin that holds rank k) from the
        // notes; noted keys of earlier bins are below the final range: their bit joins s_bit_l
        const uint32_t bin_k = (base - base0) >> bshift;
        uint32_t p_bin = 0, p_cnt = 0;   // the thread's pending count for one key value
        // the notes of bin_k are all that phase C looks at again: they move to the front of the
        // thread's list (never ahead of the note being read) and the list shrinks to them
        uint32_t n_kept = 0;
        for_notes([&](uint32_t v) {
          const uint32_t d = v & ((1u << 22) - 1u), b = d >> bshift;
          if (b < bin_k) {
            const uint32_t j = (v >> 24) * kPChunk + 4u * t + ((v >> 22) & 3u);
            atomicOr(&s_bit_l[j >> 5], 1u << (j & 31u));
          } else if (b == bin_k) {
            const uint32_t low = d & ((1u << bshift) - 1u);
            if (low != p_bin) {
              if (p_cnt) atomicAdd(&s_hist[p_bin], p_cnt);
              p_bin = low;
              p_cnt = 0;
            }
            ++p_cnt;
            if (n_kept < a.slots) s_note[n_kept * kPThreads + t] = v;
            else *spill_at(n_kept - a.slots) = v;
            ++n_kept;
          }
        });
        n_noted = n_kept;
        // pending counts: one atomic per key value and warp
        for (;;) {
          const unsigned m = __ballot_sync(0xFFFFFFFFu, p_cnt != 0u);
          if (m == 0) break;
          const int leader = __ffs(m) - 1;
          const uint32_t b0 = __shfl_sync(0xFFFFFFFFu, p_bin, leader);
          const bool mine = p_cnt != 0u && p_bin == b0;
          uint32_t sum = mine ? p_cnt : 0u;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
          if ((int)lane == leader) atomicAdd(&s_hist[b0], sum);
          if (mine) p_cnt = 0;
        }
        stamp(8);
      } else {
        // the last histogram (single keys) from the arrays; it also leaves the bitmaps "key
        // below the range" in s_bit_l and "key inside the range" in s_bit_e
        for_chunks_staged([&](uint32_t c, const uint32_t key[4]) {
          uint32_t nl = 0, ne = 0;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint32_t d = key[q] - base;
            const bool in = key[q] != kExcluded && key[q] >= base && (d >> top) == 0u;
            nl |= (uint32_t)(key[q] < base) << q;
            ne |= (uint32_t)in << q;
            w2.add(s_hist, in, d);
          }
          store_word(s_bit_l, nl, c * kPChunk + 4u * t);
          store_word(s_bit_e, ne, c * kPChunk + 4u * t);
        });
      }
      w2.flush(s_hist);
      flush_hist(a.hist + h_new * kPHistBins, 1u << top);
      stamp(9);
    };
    auto retire = [&](uint32_t h_old) {   // after a barrier: nobody reads histogram h_old any more
      if (blockIdx.x == 0) {
        for (uint32_t b = t; b < kPHistBins; b += kPThreads) a.hist[h_old * kPHistBins + b] = 0;
        if (clear_below && t == 0) a.sel->below = 0;
      }
      clear_below = false;
    };
    if (hint) {
      const unsigned long long below = __ldcg(&a.sel->below);
      const bool above = a.k > below;
      pick_bin(a.hist, kPHistBins, above ? a.k - below : 1ull, s_warp, s_pick, bin, before);
      if (above && bin != 0xFFFFFFFFu) {
        k_rem = a.k - below;
        hint_hit = true;
        use_notes = notes_complete;
        if (t == 0) {
          if (blockIdx.x == 0) atomicAdd(&a.sel->n_hint_hit, 1u);
          if (!notes_complete) atomicAdd(&a.sel->n_reread, 1u);
        }
      } else {
        // rank k is outside the bracket: digit 0 of the plain radix select
        if (blockIdx.x == 0 && t == 0) atomicAdd(&a.sel->n_hint_miss, 1u);
        base = 0;
        shift = 21;
        hist_pass(32, 21, 1);
        ok = grid_barrier(bar, ++nbar * G);
        if (!ok) goto fail;
        retire(0);
        h = 1;
        pick_bin(a.hist + kPHistBins, kPHistBins, k_rem, s_warp, s_pick, bin, before);
      }
    } else {
      pick_bin(a.hist, kPHistBins, k_rem, s_warp, s_pick, bin, before);
    }
    for (int step = 0;; ++step) {
      found = found && bin != 0xFFFFFFFFu;
      k_rem -= before;
      base += (bin & (kPHistBins - 1u)) << shift;   // rank k lies in [base, base + 2^shift)
      const uint32_t new_shift = shift > 11u ? shift - 11u : 0u;
      const uint32_t h_new = (h + 1u) % 3u;
      hist_pass(shift, new_shift, h_new);
      ok = grid_barrier(bar, ++nbar * G);
      if (step < 2) stamp(3 + step);
      if (!ok) goto fail;
      retire(h);
      pick_bin(a.hist + h_new * kPHistBins, 1u << (shift - new_shift), k_rem, s_warp, s_pick, bin, before);
      h = h_new;
      if (new_shift == 0) break;   // bin is tau's offset inside the final range [base, base + 2^shift)
      shift = new_shift;
    }
    found = found && bin != 0xFFFFFFFFu;
    k_rem -= before;

    // ---- phases C, D: tau is known; complete the bitmaps and count ----
    const uint32_t tau_low = found ? bin : 0u;          // tau - base
    const uint32_t tau = base + tau_low;
    const unsigned long long need_eq = k_rem;
    uint32_t c_l = 0, c_e = 0;
    if (use_notes) {
      const uint32_t bin_k = (base - base0) >> bshift;
      for_notes([&](uint32_t v) {
        const uint32_t d = v & ((1u << 22) - 1u);
        if ((d >> bshift) != bin_k) return;
        const uint32_t low = d & ((1u << bshift) - 1u);
        const uint32_t j = (v >> 24) * kPChunk + 4u * t + ((v >> 22) & 3u);
        if (low < tau_low) atomicOr(&s_bit_l[j >> 5], 1u << (j & 31u));
        else if (low == tau_low) atomicOr(&s_bit_e[j >> 5], 1u << (j & 31u));
      });
      __syncthreads();
      stamp(10);
      for (uint32_t w = w0; w < w1; ++w) {
        c_l += (uint32_t)__popc(s_bit_l[w]);
        c_e += (uint32_t)__popc(s_bit_e[w]);
      }
    } else {
      // s_bit_e holds the keys inside the final range; the ones below tau move to s_bit_l,
      // the ones above tau drop out.  The CTA's own last histogram is still in s_hist: when
      // all its keys of the range equal tau nothing has to be looked at again, otherwise
      // only the keys inside the range are fetched.
      uint32_t in_range = 0, cta_in_range;
      for (uint32_t w = w0; w < w1; ++w) in_range += (uint32_t)__popc(s_bit_e[w]);
      (void)block_scan_excl(in_range, s_warp, cta_in_range);
      const bool all_tau = s_hist[tau_low] == cta_in_range;
      for (uint32_t w = w0; w < w1; ++w) {
        uint32_t bl = s_bit_l[w], be = s_bit_e[w];
        if (!all_tau) {
          uint32_t bits = be;
          while (bits) {
            const uint32_t b = (uint32_t)__ffs(bits) - 1u;
            bits &= bits - 1u;
            const uint32_t key = p_score_key(__ldcg(a.score + pool_id(32u * w + b)));
            if (key != tau) be &= ~(1u << b);
            if (key < tau) bl |= 1u << b;
          }
          s_bit_l[w] = bl;
          s_bit_e[w] = be;
        }
        c_l += (uint32_t)__popc(bl);
        c_e += (uint32_t)__popc(be);
      }
    }
    uint32_t tot_l, tot_e;
    const uint32_t ex_l = block_scan_excl(c_l, s_warp, tot_l);
    const uint32_t ex_e = block_scan_excl(c_e, s_warp, tot_e);
    // The counts of every chunk go to the pool-wide table (pool order = chunk order): the scan's
    // value at a chunk's first thread is what the CTA holds before that chunk.
    const uint32_t tpc = 128u / wpt;   // threads per chunk
    const uint32_t my_c = t / tpc;     // local chunk of this thread's words
    if (t % tpc == 0u && my_c < n_chunks) s_cex[my_c] = make_uint2(ex_l, ex_e);
    if (t == 0) s_cex[n_chunks] = make_uint2(tot_l, tot_e);
    __syncthreads();
    if (t < n_chunks) {
      const uint2 c0 = s_cex[t], c1 = s_cex[t + 1u];
      a.chunk_counts[t * G + blockIdx.x] = make_uint2(c1.x - c0.x, c1.y - c0.y);
    }
    stamp(11);
    // a partition boundary strictly inside one of this CTA's chunks: how many of the chunk's
    // marked entries lie before it
    for (int q = 1; q < a.pc.n_parts; ++q) {   // (the condition is the same for the whole CTA)
      const unsigned long long bq = a.pc.base[q];
      if (bq >= a.n || (bq % kPChunk) == 0u || (bq / kPChunk) % G != blockIdx.x) continue;
      const uint32_t lc = (uint32_t)((bq / kPChunk) / G);
      const uint32_t jb = lc * kPChunk + (uint32_t)(bq % kPChunk);   // first local entry of partition q
      uint32_t bl = 0, be = 0;
      for (uint32_t w = lc * 128u + t; w <= (jb >> 5); w += kPThreads) {
        const uint32_t m = w < (jb >> 5) ? 0xFFFFFFFFu : ((1u << (jb & 31u)) - 1u);
        bl += (uint32_t)__popc(s_bit_l[w] & m);
        be += (uint32_t)__popc(s_bit_e[w] & m);
      }
      uint32_t sl, se;
      (void)block_scan_excl(bl, s_warp, sl);
      (void)block_scan_excl(be, s_warp, se);
      if (t == 0) a.sel->bsplit[q - 1] = make_uint2(sl, se);
    }
    stamp(5);
    ok = grid_barrier(bar, ++nbar * G);
    stamp(6);
    if (!ok) goto fail;
    retire(h);

    // The table read as rows of G chunks (row r = every CTA's local chunk r): what the pool holds
    // before this CTA's chunk of row r is the rows before r plus the row's columns before the
    // CTA's own.  A warp sums a row -- all of it and the part before the CTA -- with its loads
    // in flight together; one warp then scans the row totals.
    uint32_t all_l, all_e;
    {
      const uint32_t n_rows = (a.total_chunks + G - 1u) / G;   // at most kPMaxChunks
      const uint32_t warp = t >> 5;
      for (uint32_t r = warp; r < n_rows; r += kPThreads / 32u) {
        uint32_t tl = 0, te = 0, pl = 0, pe = 0;
        for (uint32_t g0 = 0; g0 < G; g0 += 128u) {
          uint2 cc[4];
#pragma unroll
          for (uint32_t u = 0; u < 4u; ++u) {
            const uint32_t gg = g0 + 32u * u + lane, cid = r * G + gg;
            cc[u] = (gg < G && cid < a.total_chunks) ? __ldcg(&a.chunk_counts[cid]) : make_uint2(0u, 0u);
          }
#pragma unroll
          for (uint32_t u = 0; u < 4u; ++u) {
            tl += cc[u].x; te += cc[u].y;
            if (g0 + 32u * u + lane < blockIdx.x) { pl += cc[u].x; pe += cc[u].y; }
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          tl += __shfl_xor_sync(0xFFFFFFFFu, tl, o); te += __shfl_xor_sync(0xFFFFFFFFu, te, o);
          pl += __shfl_xor_sync(0xFFFFFFFFu, pl, o); pe += __shfl_xor_sync(0xFFFFFFFFu, pe, o);
        }
        if (lane == 0) { s_rowtot[r] = make_uint2(tl, te); s_cpre[r] = make_uint2(pl, pe); }
      }
      __syncthreads();
      if (t < 32u) {
        // exclusive scan of the row totals (two rows per lane); s_rowtot becomes "before row r"
        const uint2 v0 = lane < n_rows ? s_rowtot[lane] : make_uint2(0u, 0u);
        const uint2 v1 = lane + 32u < n_rows ? s_rowtot[lane + 32u] : make_uint2(0u, 0u);
        uint32_t l0 = v0.x, e0 = v0.y, l1 = v1.x, e1 = v1.y;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t a0 = __shfl_up_sync(0xFFFFFFFFu, l0, o), b0 = __shfl_up_sync(0xFFFFFFFFu, e0, o);
          const uint32_t a1 = __shfl_up_sync(0xFFFFFFFFu, l1, o), b1 = __shfl_up_sync(0xFFFFFFFFu, e1, o);
          if (lane >= (uint32_t)o) { l0 += a0; e0 += b0; l1 += a1; e1 += b1; }
        }
        const uint32_t tl0 = __shfl_sync(0xFFFFFFFFu, l0, 31), te0 = __shfl_sync(0xFFFFFFFFu, e0, 31);
        s_rowtot[lane] = make_uint2(l0 - v0.x, e0 - v0.y);
        s_rowtot[lane + 32u] = make_uint2(tl0 + l1 - v1.x, te0 + e1 - v1.y);
        if (lane == 31u) s_all = make_uint2(tl0 + l1, te0 + e1);
      }
      __syncthreads();
      if (t < n_rows) {
        const uint2 rp = s_rowtot[t], cp = s_cpre[t];
        s_cpre[t] = make_uint2(rp.x + cp.x, rp.y + cp.y);
      }
      all_l = s_all.x; all_e = s_all.y;
      // the last CTA also reports the victims per partition: warp q - 1 sums what lies in front of
      // partition q's first chunk
      if (blockIdx.x == G - 1 && (int)warp + 1 < a.pc.n_parts && a.pc.base[warp + 1u] < a.n) {
        const uint32_t cb = (uint32_t)(a.pc.base[warp + 1u] / kPChunk), r = cb / G, gq = cb % G;
        uint32_t pl = 0, pe = 0;
        for (uint32_t gg = lane; gg < gq; gg += 32u) {
          const uint2 cc = __ldcg(&a.chunk_counts[r * G + gg]);
          pl += cc.x; pe += cc.y;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          pl += __shfl_xor_sync(0xFFFFFFFFu, pl, o); pe += __shfl_xor_sync(0xFFFFFFFFu, pe, o);
        }
        if (lane == 0) s_bnd[warp] = make_uint2(s_rowtot[r].x + pl, s_rowtot[r].y + pe);
      }
      __syncthreads();
      stamp(12);
    }
    if (found) {
      // Position of a victim.  With L entries below tau and E entries equal to tau before it
      // in id order, an entry below tau goes to L + min(E, need_eq) and an entry equal to tau,
      // taken while E < need_eq, to L + E.  The victims of a chunk form one contiguous piece of
      // the output.  Every thread walks the set bits of its own words and puts the ids in
      // order in shared memory (the notes' space, free by now), the CTA's chunks one after the
      // other; from there they leave as full-line stores, a stage-full per round.
      const uint32_t eq_room = need_eq > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)need_eq;
      auto taken = [&](uint32_t e) { return e < eq_room ? e : eq_room; };
      if (t < 32u) {
        // where each chunk's piece starts: in the output (s_gstart) and in the stage (s_lstart)
        uint32_t v[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const uint32_t lc = lane + 32u * u;
          v[u] = 0;
          if (lc < n_chunks) {
            const uint2 c0 = s_cex[lc], c1 = s_cex[lc + 1u], pre = s_cpre[lc];
            v[u] = (c1.x - c0.x) + (taken(pre.y + (c1.y - c0.y)) - taken(pre.y));
            s_gstart[lc] = pre.x + taken(pre.y);
          }
        }
        uint32_t i0 = v[0], i1 = v[1];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t y0 = __shfl_up_sync(0xFFFFFFFFu, i0, o), y1 = __shfl_up_sync(0xFFFFFFFFu, i1, o);
          if (lane >= (uint32_t)o) { i0 += y0; i1 += y1; }
        }
        const uint32_t tot0 = __shfl_sync(0xFFFFFFFFu, i0, 31);
        s_lstart[lane] = i0 - v[0];
        s_lstart[lane + 32u] = tot0 + i1 - v[1];
        if (lane == 31u) s_lstart[64] = tot0 + i1;
      }
      __syncthreads();
      stamp(14);
      const uint32_t cta_total = s_lstart[64];
      uint32_t* const s_stage = s_note;
      const uint32_t stage_cap = scratch_words;
      // A thread whose words are full writes positions 32 * wpt apart from its neighbour's: the
      // stage is indexed with the bank bits folded over by that stride, which keeps those writes
      // and the consecutive reads of the copy-out both free of bank conflicts.
      const uint32_t fold = 5u + (uint32_t)__ffs(wpt) - 1u;
      auto stage_at = [&](uint32_t p) { return p ^ ((p >> fold) & 31u); };
      // entries below / equal to tau in front of this thread's words, in the whole pool
      const uint32_t mc = my_c < n_chunks ? my_c : 0u;   // (threads past the last chunk hold nothing)
      const uint32_t Lg = s_cpre[mc].x + (ex_l - s_cex[mc].x), Eg = s_cpre[mc].y + (ex_e - s_cex[mc].y);
      // from a position in the output to one in the stage (modulo 2^32)
      const uint32_t to_stage = s_lstart[mc] - s_gstart[mc];
      // the thread's own victims are the consecutive stage positions [p_first, p_first + p_count)
      const uint32_t p_first = Lg + taken(Eg) + to_stage, p_count = c_l + (taken(Eg + c_e) - taken(Eg));
      __syncthreads();   // every thread is done with the notes
      stamp(13);
      for (uint32_t r0 = 0; r0 < cta_total; r0 += stage_cap) {
        if (p_count != 0 && p_first < r0 + stage_cap && p_first + p_count > r0) {
          // entries below tau before the current word (shifted into stage positions), entries at tau
          uint32_t n_l = Lg + to_stage, n_e = Eg;
          for (uint32_t w = w0; w < w1; ++w) {
            const uint32_t bl = s_bit_l[w], be = s_bit_e[w];
            const uint32_t id0 = (uint32_t)pool_id(32u * w);   // (ids fit 32 bits)
            const uint32_t ce = (uint32_t)__popc(be);
            if (be == 0u || n_e >= eq_room || n_e + ce <= eq_room) {
              // no entry at tau in this word, none of them taken any more, or all of them taken:
              // the word's victims take consecutive positions
              const uint32_t vb = (be == 0u || n_e >= eq_room) ? bl : (bl | be);
              uint32_t pos = n_l + (n_e < eq_room ? n_e : eq_room) - r0;   // (wraps below r0: skipped)
              uint32_t bits = vb;
              while (bits) {
                const uint32_t b = (uint32_t)__ffs(bits) - 1u;
                bits &= bits - 1u;
                if (pos < stage_cap) s_stage[stage_at(pos)] = id0 + b;
                ++pos;
              }
              n_l += (uint32_t)__popc(bl);
              n_e += ce;
              continue;
            }
            uint32_t bits = bl | be;
            while (bits) {
              const uint32_t b = (uint32_t)__ffs(bits) - 1u;
              bits &= bits - 1u;
              uint32_t pos = 0xFFFFFFFFu;
              if ((bl >> b) & 1u) {
                pos = n_l + (n_e < eq_room ? n_e : eq_room);
                ++n_l;
              } else {
                if (n_e < eq_room) pos = n_l + n_e;
                ++n_e;
              }
              if (pos >= r0 && pos - r0 < stage_cap) s_stage[stage_at(pos - r0)] = id0 + b;
            }
          }
        }
        __syncthreads();
        stamp(4);
        const uint32_t r1 = cta_total - r0 < stage_cap ? cta_total : r0 + stage_cap;
        {
          // stage position i belongs to the chunk lc with s_lstart[lc] <= i < s_lstart[lc + 1]; a
          // thread's positions ascend, so its chunk only moves forward
          uint32_t lc = 0, le = s_lstart[1];
          for (uint32_t i = r0 + t; i < r1; i += kPThreads) {
            while (i >= le) { ++lc; le = s_lstart[lc + 1u]; }
            const unsigned long long g = (unsigned long long)s_gstart[lc] + (i - s_lstart[lc]);
            if (g < a.k) a.victims[g] = s_stage[stage_at(i - r0)];
          }
        }
        stamp(15);
        __syncthreads();
      }
    }
    if (blockIdx.x == G - 1) __syncthreads();   // s_bnd
    if (blockIdx.x == G - 1 && t == 0) {
      // every entry has been counted: the selection must hold exactly k ids
      const unsigned long long tl = all_l, te = all_e;
      const unsigned long long got = tl + (te < need_eq ? te : need_eq);
      if (!found || got != a.k) atomicOr(a.status, KV_DEV_SELECT_MISMATCH);
      if (a.pc.n_parts > 1 && a.pc.d_counts) {
        // victims before each partition boundary = entries below tau before it + the taken
        // ones among the entries equal to tau before it
        unsigned long long before[5] = {0, 0, 0, 0, 0};
        for (int q = 1; q <= a.pc.n_parts; ++q) {
          if (q == a.pc.n_parts || a.pc.base[q] >= a.n) { before[q] = got; continue; }
          unsigned long long l = s_bnd[q - 1].x, e = s_bnd[q - 1].y;     // sums over the chunks before the boundary's
          if (a.pc.base[q] % kPChunk) {                                   // strictly inside that chunk
            const uint2 sp = __ldcg(&a.sel->bsplit[q - 1]);
            l += sp.x; e += sp.y;
          }
          before[q] = l + (e < need_eq ? e : need_eq);
        }
        for (int q = 0; q < 4; ++q) {
          const unsigned long long c = q < a.pc.n_parts ? before[q + 1] - before[q] : 0ull;
          a.pc.d_counts[q] = c;
          if (a.pc.h_counts) a.pc.h_counts[q] = c;
        }
      }
      a.sel->tau = tau;
      a.sel->need_eq = need_eq;
      a.sel->n_select += 1;
      // hint for the next selection over the same keys: this tau moved on by as much as it
      // moved since the selection before (while a pool warms up its scores grow epoch after
      // epoch, and the trend is a better centre for the bracket than the last value)
      const bool had = a.sel->hint_valid != 0 && a.sel->hint_n == a.n;
      const long long step = had ? (long long)tau - (long long)a.sel->hint_last : 0ll;
      long long guess = (long long)tau + step;
      if (guess < 0) guess = 0;
      if (guess > 0xFFFFFFFEll) guess = 0xFFFFFFFEll;
      // ... and the bracket is as wide as the hints have been off lately: eight times a slowly
      // decaying maximum of |tau - hinted tau|, full width again after a miss (a narrow
      // bracket means fewer keys to note; a miss costs two more passes over the keys)
      uint32_t resid = a.sel->hint_resid, new_shift = kBracketShiftMax;
      if (hint_hit) {
        const uint32_t off = tau > hint_tau ? tau - hint_tau : hint_tau - tau;
        resid -= resid >> 2;
        if (off > resid) resid = off;
        new_shift = kBracketShiftMin;
        while (new_shift < kBracketShiftMax && (1ull << (new_shift + 10u)) < 8ull * resid) ++new_shift;
      } else {
        resid = 1u << 18;
      }
      a.sel->hint_resid = resid;
      a.sel->hint_shift = new_shift;
      a.sel->hint_last = tau;
      a.sel->hint_tau = (uint32_t)guess;
      a.sel->hint_n = a.n;
      a.sel->hint_valid = (found && got == a.k) ? 1u : 0u;
    }
  }
  stamp(7);
  goto done;

fail:
  if (t == 0) atomicOr(a.status, KV_DEV_WAIT_EXPIRED);
done:
  // the last CTA to leave resets the barrier for the next launch
  __syncthreads();
  if (t == 0) {
    __threadfence();
    const unsigned int old = atomicAdd(&a.sel->bar_done, 1u);
    if (old == G - 1) {
      a.sel->bar_arrive = 0;
      a.sel->bar_done = 0;
      __threadfence();
    }
  }
}

// What one device can do with the persistent kernels, probed once per device
// (with that device current) under a lock.
namespace {
struct PersistDevice {
  int state = 0;   // 0 = not probed, 1 = usable, -1 = not usable
  int n_sm = 0;
  size_t smem_max = 0;   // dynamic shared memory the kernels were opted in for
};
constexpr int kPMaxDevices = 64;
std::mutex g_persist_mutex;
PersistDevice g_persist[kPMaxDevices];

// Dynamic shared memory of a launch: two bitmaps and the threads' private slots (which the
// ordered write reuses as its staging buffer).
inline size_t persist_smem(uint32_t words, uint32_t slots, uint32_t entry_stages = 0) {
  return (size_t)words * 8u + (size_t)slots * kPThreads * 4u + (size_t)entry_stages * kEntryStageWords * 4u;
}
}  // namespace

// Launches the persistent selection (fused with the entry pass when fs is given)
// if the device can hold one CTA per SM of it co-resident and the slices fit the
// bitmaps; *used = false (and nothing launched) otherwise.
cudaError_t launch_select_persistent(const EntryState& st, uint64_t k, uint32_t* d_victims,
                                     const Workspace& ws, cudaStream_t s, bool* used, const FusedScore* fs,
                                     const PartCounts* pc) {
  *used = false;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return cudaGetLastError();
  if (dev < 0 || dev >= kPMaxDevices) return cudaSuccess;
  PersistDevice pd;
  {
    std::lock_guard<std::mutex> lock(g_persist_mutex);
    PersistDevice& d = g_persist[dev];
    if (d.state == 0) {
      int coop = 0, blocks = 0, blocks_f = 0, optin = 0;
      cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
      cudaDeviceGetAttribute(&d.n_sm, cudaDevAttrMultiProcessorCount, dev);
      cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
      void* fns[3] = {(void*)select_persistent_kernel<false, false>, (void*)select_persistent_kernel<true, false>,
                      (void*)select_persistent_kernel<true, true>};
      cudaError_t e = cudaSuccess;
      size_t fixed = 0;
      for (void* fn : fns) {
        cudaFuncAttributes fa{};
        if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa, fn);
        if (fa.sharedSizeBytes > fixed) fixed = fa.sharedSizeBytes;
      }
      // the most a launch may ask for: everything a block can opt in to beyond the kernels' static
      // share; the least that must fit: the largest bitmaps, the fewest slots, the entry stages
      const size_t want = (size_t)optin > fixed ? ((size_t)optin - fixed) / 1024 * 1024 : 0;
      if (want < persist_smem(kPMaxSlice / 32, kPSlotsMin, kEntryStages)) e = cudaErrorInvalidValue;
      d.smem_max = want;
      blocks = 1;
      for (void* fn : fns) {
        int b = 0;
        if (e == cudaSuccess) e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)want);
        if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, fn, (int)kPThreads, want);
        if (b < blocks) blocks = b;
      }
      blocks_f = blocks;
      d.state = (e == cudaSuccess && coop && blocks >= 1 && blocks_f >= 1 && d.n_sm > 0) ? 1 : -1;
      (void)cudaGetLastError();
    }
    pd = d;
  }
  if (pd.state != 1) return cudaSuccess;
  unsigned int G = (unsigned int)pd.n_sm;
  if (G > kPThreads) G = kPThreads;
  const uint64_t total_chunks = (st.n + kPChunk - 1) / kPChunk;
  if (total_chunks < G) G = (unsigned int)total_chunks;   // tiny pools: not more CTAs than chunks
  if (G == 0) G = 1;
  if (total_chunks + 2 > ws.n_tiles) return cudaSuccess;  // the per-chunk counts live in the tile-count scratch
  PArgs a;
  a.score = st.score;
  a.state = st.state;
  a.n = st.n;
  a.k = k;
  a.victims = d_victims;
  a.hist = ws.hist;
  a.sel = ws.sel;
  a.chunk_counts = ws.tile_counts;
  a.total_chunks = (uint32_t)total_chunks;
  a.status = ws.status;
  a.per = (total_chunks + G - 1) / G * kPChunk;   // the most entries a CTA holds: its chunks, whole
  if (a.per > kPMaxSlice) return cudaSuccess;  // more than the bitmaps hold: the multi-launch selection runs
  a.words = (uint32_t)(a.per / 32);
  // The hint's bracket typically holds 5-10 % of a slice's keys, but slices differ (blocks of one
  // history sit together), and a thread that runs out of slots sends its CTA the long way.  What this kernel does not take
  // of the shared memory stays with the L1, whose lines hold the loads in flight of the streaming
  // entry pass.
  uint64_t slots = (a.per + kPThreads - 1) / kPThreads;   // as many as the thread sees keys, up to the maximum
  if (slots < kPSlotsMin) slots = kPSlotsMin;   // (two stages of the re-reading passes fit)
  if (slots > kPSlotsMax) slots = kPSlotsMax;
  // the fused form streams its entries through stages behind the slots; the slots give way
  // (a thread's notes beyond them go to the global scratch)
  a.entry_stages = fs ? kEntryStages : 0u;
  while (slots > kPSlotsMin && persist_smem(a.words, (uint32_t)slots, a.entry_stages) > pd.smem_max) --slots;
  a.slots = (uint32_t)slots;
  const size_t smem = persist_smem(a.words, a.slots, a.entry_stages);
  if (smem > pd.smem_max) return cudaSuccess;
  a.pc = pc ? *pc : PartCounts{};
  a.spill = ws.free_list;   // (scratch of promotions and admissions: idle while a selection runs)
  a.st = st;
  a.pd = Predictor{};
  a.hw = HeadWeights{};
  a.epoch = 0;
  if (fs) {
    a.pd = Predictor{fs->hits,       fs->misses,    fs->P,          fs->alpha0, fs->beta0, ws.delta, nullptr,
                     fs->opt.policy, fs->opt.kappa, fs->opt.window, ws.blend};
    a.hw = fs->hw;
    a.epoch = fs->epoch;
  }
  void* args[] = {&a};
  const bool plain = fs && fs->opt.policy == 0 && fs->hw.on == 0;
  void* fn = !fs ? (void*)select_persistent_kernel<false, false>
                 : plain ? (void*)select_persistent_kernel<true, true> : (void*)select_persistent_kernel<true, false>;
  cudaError_t e = launch_scoring_kernel(fn, dim3(G), dim3(kPThreads), args, smem, s, true, ws);
  if (e != cudaSuccess) return e;
  count_launches(1);
  *used = true;
  return cudaSuccess;
}

}  // namespace kvt
