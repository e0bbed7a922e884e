// k-lowest selection as ONE cooperative, persistent launch.
//
// The multi-launch selection in kv_select.cu spends most of its time between
// kernels when the pool has a few million entries: ten dependent launches of
// 3-10 us each.  Here one CTA per SM stays resident for the whole selection.
// Each CTA owns a contiguous slice of the entries; the phases of the selection
// are separated by grid-wide barriers instead of kernel boundaries:
//
//   A  every score becomes an order-preserving key (fused form: the entry pass
//      itself produces it) and enters the first histogram.  With a hint -- tau of
//      the previous selection -- the histogram covers a bracket of 2^22 keys
//      around it, and the pass also leaves in shared memory a bitmap "key below
//      the bracket" and a list of the keys inside the bracket (index in the
//      slice, bracket bin, low bits): typically 5-10 % of the slice.
//   B  the remaining histograms of the radix select.  When rank k falls inside
//      the bracket, ONE more histogram (the 2^11 single keys of the bracket bin
//      that holds rank k) finishes it, and it is built from the list alone: no
//      second pass over the scores.  Otherwise (no hint, a miss, a list that
//      overflowed) the keys are re-read from the score array, which then sits
//      mostly in L2; the last histogram of that path leaves the bitmaps "key
//      below the final range" and "key inside the final range".
//   C  tau picked: the keys of the final range are sorted into "below tau" and
//      "equal to tau" -- from the list, or, on the other path, by fetching just
//      the keys inside the range (not even those when the CTA's own histogram
//      shows that all of them equal tau: a tie, the usual case when few distinct
//      scores exist).
//   D  per-CTA counts = population counts of the two bitmaps; after the last
//      barrier every CTA knows how many victims precede its slice and writes its
//      own victims in ascending id order straight from the bitmaps.
//
// The grid barrier is a counter in global memory that every CTA increments and
// then polls.  A cooperative launch guarantees that all CTAs are resident, so
// the wait ends; it is nevertheless bounded, and a CTA that gives up sets
// KV_DEV_WAIT_EXPIRED and leaves (every other CTA then runs into the same limit).
//
// The same kernel also exists fused with the per-entry scoring pass (FUSED =
// true): every CTA first updates the entries of its own slice (posterior, EMA,
// score) and turns the fresh scores straight into keys -- a kernel boundary
// disappears.  The event reduction stays a launch of its own ahead of it: its
// scattered gathers and atomics ran 2.5x slower inside this kernel when that was
// tried, and a grid barrier costs about what the launch boundary does.
#include <cstdlib>
#include <mutex>
#include <type_traits>

#include "kv_score_device.cuh"

namespace kvt {

constexpr uint32_t kPThreads = 1024;
constexpr uint32_t kPChunk = kPThreads * 4;             // 4096 entries: one 16-byte vector per thread
constexpr uint32_t kPHistBins = 2048;
constexpr uint32_t kExcluded = 0xFFFFFFFFu;             // key of a non-candidate (FREE) entry
constexpr uint32_t kBarrierSpins = 1u << 22;
constexpr uint32_t kBracketShift = 11;                  // a bracket bin is 2^11 keys wide ...
constexpr uint32_t kBracketHalf = 1u << 21;             // ... and the 2,048 bins reach 2^21 keys to either side of the hint
constexpr uint32_t kBracketBits = 22;                   // log2 of the bracket's width in keys
constexpr uint32_t kPIdxBits = 18;                      // index of an entry inside its slice
constexpr uint32_t kPMaxSlice = 1u << kPIdxBits;        // entries per CTA the bitmaps are sized for (2 x 32 KB)
constexpr uint32_t kPListCapMax = 16384;                // bracket keys remembered per CTA (6 bytes each)

static_assert(kPIdxBits + kBracketBits - kBracketShift <= 32, "index and bracket bin share one word");

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
  uint2* cta_counts;      // [gridDim.x]
  uint32_t* status;
  unsigned long long per; // entries per CTA slice (multiple of 4, at most kPMaxSlice)
  uint32_t words;         // 32-bit words of one bitmap of a slice (a multiple of 4)
  uint32_t list_cap;      // entries of the bracket list (a multiple of 8)
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

template <bool FUSED>
__global__ void __launch_bounds__(kPThreads, 1) select_persistent_kernel(const PArgs a) {
  extern __shared__ __align__(16) uint32_t s_dyn[];
  uint32_t* const s_bit_l = s_dyn;                    // bit j: key of local entry j is below tau
  uint32_t* const s_bit_e = s_bit_l + a.words;        // bit j: key of local entry j equals tau
  uint32_t* const s_list_jb = s_bit_e + a.words;      // bracket list: index in slice | bracket bin << kPIdxBits
  uint16_t* const s_list_low = reinterpret_cast<uint16_t*>(s_list_jb + a.list_cap);  // ... and key bits below the bin
  __shared__ uint32_t s_hist[kPHistBins];
  __shared__ uint32_t s_warp[32];
  __shared__ uint32_t s_pick[2];
  __shared__ uint32_t s_list_n;
  __shared__ float sP[16];
  const uint32_t t = threadIdx.x;
  const uint32_t lane = t & 31u;
  unsigned int* bar = &a.sel->bar_arrive;
  const unsigned int G = gridDim.x;
  const unsigned long long s0 = (unsigned long long)blockIdx.x * a.per;
  const unsigned long long s1 = (s0 + a.per < a.n) ? s0 + a.per : a.n;
  const uint32_t len = s1 > s0 ? (uint32_t)(s1 - s0) : 0u;
  const uint32_t n_chunks = (len + kPChunk - 1) / kPChunk;
  bool ok = true;
  auto stamp = [&](int i) {
    if (blockIdx.x == 0 && t == 0) {
      unsigned long long ns;
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(ns));
      a.sel->phase_ns[i] = ns;
    }
  };
  stamp(0);

  // keys of the thread's vector (4 entries) of chunk c, computed from the arrays;
  // entries past the slice or not RESIDENT give kExcluded
  auto keys_from_arrays = [&](uint32_t c, uint32_t key[4]) {
    const uint32_t j0 = c * kPChunk + 4u * t;
    const unsigned long long i0 = s0 + j0;
    if (j0 + 4 <= len) {
      const float4 sc = __ldcg(reinterpret_cast<const float4*>(a.score + i0));
      const uchar4 st = __ldcg(reinterpret_cast<const uchar4*>(a.state + i0));
      key[0] = st.x == KV_STATE_RESIDENT ? p_score_key(sc.x) : kExcluded;
      key[1] = st.y == KV_STATE_RESIDENT ? p_score_key(sc.y) : kExcluded;
      key[2] = st.z == KV_STATE_RESIDENT ? p_score_key(sc.z) : kExcluded;
      key[3] = st.w == KV_STATE_RESIDENT ? p_score_key(sc.w) : kExcluded;
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j)
        key[j] = (j0 + j < len && a.state[i0 + j] == KV_STATE_RESIDENT) ? p_score_key(a.score[i0 + j])
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
        const uint32_t j0 = (c - 1u - u) * kPChunk + 4u * t;
        if (u < nb && j0 + 4 <= len) {
          sc[u] = __ldcg(reinterpret_cast<const float4*>(a.score + s0 + j0));
          st[u] = __ldcg(reinterpret_cast<const uchar4*>(a.state + s0 + j0));
        }
      }
#pragma unroll
      for (uint32_t u = 0; u < kAhead; ++u) {
        if (u < nb) {
          const uint32_t cc = c - 1u - u;
          const uint32_t j0 = cc * kPChunk + 4u * t;
          uint32_t key[4];
          if (j0 + 4 <= len) {
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
  // every thread owns a contiguous run of bitmap words
  const uint32_t wpt = (a.words + kPThreads - 1) / kPThreads;
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
  if (t == 0) s_list_n = 0;

  // ---- phase A: keys and the first histogram ----
  // Without a hint the first histogram is digit 0 of a plain radix select (bits
  // 31..21 of every key).  With a hint it covers only the bracket [base0, base0 +
  // 2^22) around the hinted tau in 2,048 bins of 2^11 keys; keys below base0 set
  // their bit in s_bit_l (and are counted), keys inside go on the list: scores
  // move little from one epoch to the next, so the k-th key is almost always
  // inside, and then nothing but the list is looked at again.
  const bool hint = a.sel->hint_valid != 0 && a.sel->hint_n == a.n;
  const uint32_t hint_tau = a.sel->hint_tau;
  const uint32_t base0 = hint ? (hint_tau > kBracketHalf ? hint_tau - kBracketHalf : 0u) : 0u;
  const uint32_t shift0 = hint ? kBracketShift : 21u;
  WarpHist wh;
  auto phase_a = [&](uint32_t c, const uint32_t key[4]) {
    if (!hint) {
#pragma unroll
      for (int q = 0; q < 4; ++q) wh.add(s_hist, key[q] != kExcluded, key[q] >> 21);
      return;
    }
    const uint32_t j0 = c * kPChunk + 4u * t;
    uint32_t nib = 0, d[4], m[4], total = 0;
    bool in[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      d[q] = key[q] - base0;
      nib |= (uint32_t)(key[q] < base0) << q;   // (an excluded key is 0xFFFFFFFF: never below)
      in[q] = key[q] != kExcluded && key[q] >= base0 && (d[q] >> kBracketBits) == 0u;
      m[q] = __ballot_sync(0xFFFFFFFFu, in[q]);
      total += (uint32_t)__popc(m[q]);
    }
    store_word(s_bit_l, nib, j0);
    if (total == 0) return;   // (uniform over the warp)
    uint32_t at = 0;
    if (lane == 0) at = atomicAdd(&s_list_n, total);
    at = __shfl_sync(0xFFFFFFFFu, at, 0);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      wh.add_voted(s_hist, m[q], in[q], d[q] >> kBracketShift);
      const uint32_t pos = at + (uint32_t)__popc(m[q] & ((1u << lane) - 1u));
      if (in[q] && pos < a.list_cap) {
        s_list_jb[pos] = (j0 + q) | ((d[q] >> kBracketShift) << kPIdxBits);
        s_list_low[pos] = (uint16_t)(d[q] & ((1u << kBracketShift) - 1u));
      }
      at += (uint32_t)__popc(m[q]);
    }
  };
  clear_hist();
  if constexpr (FUSED) {
    // the slice's entries go through the EMA and score update on the way
    const int policy = a.pd.policy;
    const uint32_t jt = 4u * t;
    EntryVec cur;
    if (jt + 4 <= len) cur = entry_load4(a.st, (s0 + jt) / 4, policy);
    for (uint32_t c = 0; c < n_chunks; ++c) {
      const uint32_t j0 = c * kPChunk + jt;
      const unsigned long long i0 = s0 + j0;
      // the next chunk's loads fly while this one is finished
      EntryVec nxt;
      if (c + 1 < n_chunks && j0 + kPChunk + 4 <= len) nxt = entry_load4(a.st, (i0 + kPChunk) / 4, policy);
      uint32_t key[4] = {kExcluded, kExcluded, kExcluded, kExcluded};
      if (j0 + 4 <= len) {
        float4 sc;
        entry_finish4(a.st, i0 / 4, cur, sP, policy, a.epoch, a.hw, sc);
        key[0] = cur.st.x == KV_STATE_RESIDENT ? p_score_key(sc.x) : kExcluded;
        key[1] = cur.st.y == KV_STATE_RESIDENT ? p_score_key(sc.y) : kExcluded;
        key[2] = cur.st.z == KV_STATE_RESIDENT ? p_score_key(sc.z) : kExcluded;
        key[3] = cur.st.w == KV_STATE_RESIDENT ? p_score_key(sc.w) : kExcluded;
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (j0 + j < len) {
            float sc;
            uint32_t s1;
            entry_update1(a.st, i0 + j, sP, policy, a.epoch, a.hw, sc, s1);
            if (s1 == KV_STATE_RESIDENT) key[j] = p_score_key(sc);
          }
        }
      }
      cur = nxt;
      phase_a(c, key);
    }
  } else {
    for_chunks(phase_a);
  }
  wh.flush(s_hist);
  flush_hist(a.hist, kPHistBins);   // (begins with a block barrier: the bitmap words are all written)
  if (hint) {
    uint32_t below = 0, cta_below0;
    for (uint32_t w = w0; w < w1; ++w) below += (uint32_t)__popc(s_bit_l[w]);
    (void)block_scan_excl(below, s_warp, cta_below0);
    if (t == 0 && cta_below0) atomicAdd(&a.sel->below, (unsigned long long)cta_below0);
  }
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
    bool use_list = false;   // rank k is inside the bracket and this CTA's list holds all its bracket keys
    const uint32_t n_list = s_list_n;
    auto hist_pass = [&](uint32_t width_log2, uint32_t new_shift, uint32_t h_new) {
      // histogram of ((key - base) >> new_shift) over the keys in [base, base + 2^width_log2)
      clear_hist();
      const uint32_t top = width_log2 - new_shift;  // log2 of the number of bins
      WarpHist w2;
      if (new_shift != 0) {
        for_chunks([&](uint32_t, const uint32_t key[4]) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint32_t d = key[q] - base;
            w2.add(s_hist, key[q] != kExcluded && key[q] >= base && ((d >> new_shift) >> top) == 0u,
                   d >> new_shift);
          }
        });
      } else if (use_list) {
        // the last histogram (single keys of the bracket bin that holds rank k) from the
        // list; listed keys of earlier bins are below the range: their bit joins s_bit_l
        const uint32_t bin_k = (base - base0) >> kBracketShift;
        const uint32_t iters = (n_list + kPThreads - 1) / kPThreads;
        for (uint32_t i = 0; i < iters; ++i) {
          const uint32_t e = i * kPThreads + t;
          uint32_t b = 0xFFFFFFFFu, j = 0, low = 0;
          if (e < n_list) {
            const uint32_t v = s_list_jb[e];
            b = v >> kPIdxBits;
            j = v & (kPMaxSlice - 1u);
            low = s_list_low[e];
          }
          if (b < bin_k) atomicOr(&s_bit_l[j >> 5], 1u << (j & 31u));
          w2.add(s_hist, b == bin_k, low);
        }
      } else {
        // the last histogram (single keys) from the arrays; it also leaves the bitmaps "key
        // below the range" in s_bit_l and "key inside the range" in s_bit_e
        for_chunks([&](uint32_t c, const uint32_t key[4]) {
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
        use_list = n_list <= a.list_cap;
      } else {
        // rank k is outside the bracket: digit 0 of the plain radix select
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
    if (use_list) {
      const uint32_t bin_k = (base - base0) >> kBracketShift;
      for (uint32_t e = t; e < n_list; e += kPThreads) {
        const uint32_t v = s_list_jb[e];
        if ((v >> kPIdxBits) != bin_k) continue;
        const uint32_t j = v & (kPMaxSlice - 1u), low = s_list_low[e];
        if (low < tau_low) atomicOr(&s_bit_l[j >> 5], 1u << (j & 31u));
        else if (low == tau_low) atomicOr(&s_bit_e[j >> 5], 1u << (j & 31u));
      }
      __syncthreads();
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
            const uint32_t key = p_score_key(__ldcg(a.score + s0 + 32u * w + b));
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
    if (t == 0) a.cta_counts[blockIdx.x] = make_uint2(tot_l, tot_e);
    stamp(5);
    ok = grid_barrier(bar, ++nbar * G);
    stamp(6);
    if (!ok) goto fail;
    retire(h);

    unsigned long long less_before, eq_before;
    {
      unsigned long long la = 0, ea = 0;  // sums over the CTAs before this one
      for (uint32_t g = t; g < blockIdx.x; g += kPThreads) {
        const uint2 cc = __ldcg(&a.cta_counts[g]);
        la += cc.x; ea += cc.y;
      }
      // (G <= 1024: one value per thread at most, each below 2^18)
      uint32_t tl, te;
      (void)block_scan_excl((uint32_t)la, s_warp, tl);
      (void)block_scan_excl((uint32_t)ea, s_warp, te);
      less_before = tl; eq_before = te;
    }
    if (found) {
      // Position of a victim.  With L entries below tau and E entries equal to tau before it
      // in id order, an entry below tau goes to L + min(E, need_eq) and an entry equal to tau,
      // taken while E < need_eq, to L + E.
      unsigned long long n_l = less_before + ex_l, n_e = eq_before + ex_e;
      for (uint32_t w = w0; w < w1; ++w) {
        const uint32_t bl = s_bit_l[w], be = s_bit_e[w];
        uint32_t bits = bl | be;
        while (bits) {
          const uint32_t b = (uint32_t)__ffs(bits) - 1u;
          bits &= bits - 1u;
          const unsigned long long id = s0 + 32ull * w + b;
          if ((bl >> b) & 1u) {
            const unsigned long long pos = n_l + (n_e < need_eq ? n_e : need_eq);
            if (pos < a.k) a.victims[pos] = (uint32_t)id;
            ++n_l;
          } else {
            if (n_e < need_eq) {
              const unsigned long long pos = n_l + n_e;
              if (pos < a.k) a.victims[pos] = (uint32_t)id;
            }
            ++n_e;
          }
        }
      }
    }
    if (blockIdx.x == G - 1 && t == 0) {
      // every entry has been counted: the selection must hold exactly k ids
      unsigned long long tl = 0, te = 0;
      for (uint32_t g = 0; g < G; ++g) { const uint2 cc = __ldcg(&a.cta_counts[g]); tl += cc.x; te += cc.y; }
      const unsigned long long got = tl + (te < need_eq ? te : need_eq);
      if (!found || got != a.k) atomicOr(a.status, KV_DEV_SELECT_MISMATCH);
      a.sel->tau = tau;
      a.sel->need_eq = need_eq;
      // hint for the next selection over the same keys: this tau moved on by as much as it
      // moved since the selection before (while a pool warms up its scores grow epoch after
      // epoch, and the trend is a better centre for the bracket than the last value)
      const bool had = a.sel->hint_valid != 0 && a.sel->hint_n == a.n;
      const long long step = had ? (long long)tau - (long long)a.sel->hint_last : 0ll;
      long long guess = (long long)tau + step;
      if (guess < 0) guess = 0;
      if (guess > 0xFFFFFFFEll) guess = 0xFFFFFFFEll;
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

// Dynamic shared memory of a launch: two bitmaps and the bracket list.
inline size_t persist_smem(uint32_t words, uint32_t list_cap) {
  return (size_t)words * 8u + (size_t)list_cap * 6u;
}
}  // namespace

// Launches the persistent selection (fused with the entry pass when fs is given)
// if the device can hold one CTA per SM of it co-resident and the slices fit the
// bitmaps; *used = false (and nothing launched) otherwise.
cudaError_t launch_select_persistent(const EntryState& st, uint64_t k, uint32_t* d_victims,
                                     const Workspace& ws, cudaStream_t s, bool* used, const FusedScore* fs) {
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
      cudaFuncAttributes fa{}, fb{};
      cudaError_t e = cudaFuncGetAttributes(&fa, select_persistent_kernel<false>);
      if (e == cudaSuccess) e = cudaFuncGetAttributes(&fb, select_persistent_kernel<true>);
      const size_t fixed = fa.sharedSizeBytes > fb.sharedSizeBytes ? fa.sharedSizeBytes : fb.sharedSizeBytes;
      // the most a launch asks for: the largest bitmaps and the longest list
      const size_t want = persist_smem(kPMaxSlice / 32, kPListCapMax);
      if ((size_t)optin < fixed + want) e = cudaErrorInvalidValue;
      d.smem_max = want;
      if (e == cudaSuccess)
        e = cudaFuncSetAttribute(select_persistent_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)want);
      if (e == cudaSuccess)
        e = cudaFuncSetAttribute(select_persistent_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)want);
      if (e == cudaSuccess)
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks, select_persistent_kernel<false>,
                                                          (int)kPThreads, want);
      if (e == cudaSuccess)
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks_f, select_persistent_kernel<true>,
                                                          (int)kPThreads, want);
      d.state = (e == cudaSuccess && coop && blocks >= 1 && blocks_f >= 1 && d.n_sm > 0) ? 1 : -1;
      (void)cudaGetLastError();
    }
    pd = d;
  }
  if (pd.state != 1) return cudaSuccess;
  unsigned int G = (unsigned int)pd.n_sm;
  if (G > kPThreads) G = kPThreads;  // the prefix over the per-CTA counts takes one CTA per thread
  const uint64_t min_per = kPChunk;  // do not spread tiny pools over more CTAs than they have chunks
  if ((st.n + min_per - 1) / min_per < G) G = (unsigned int)((st.n + min_per - 1) / min_per);
  if (G == 0) G = 1;
  if (G + 2 > ws.n_tiles) return cudaSuccess;  // cta_counts live in the tile-count scratch
  PArgs a;
  a.score = st.score;
  a.state = st.state;
  a.n = st.n;
  a.k = k;
  a.victims = d_victims;
  a.hist = ws.hist;
  a.sel = ws.sel;
  a.cta_counts = ws.tile_counts;
  a.status = ws.status;
  a.per = ((st.n + G - 1) / G + 3) / 4 * 4;
  if (a.per > kPMaxSlice) return cudaSuccess;  // slices beyond the bitmaps: the multi-launch selection runs
  a.words = (uint32_t)((a.per + 31) / 32 + 3) / 4 * 4;
  // The list holds the keys inside the hint's bracket, typically 5-10 % of a slice; a CTA whose
  // list overflows re-reads its keys instead.  What this kernel does not take of the shared
  // memory stays with the L1, whose lines hold the loads in flight of the streaming entry pass.
  uint64_t list_cap = (a.per / 4 + 7) / 8 * 8;
  if (const char* e = std::getenv("KVTIER_SELECT_LIST")) list_cap = (uint64_t)std::atoi(e) / 8 * 8;
  if (list_cap < 8) list_cap = 8;
  if (list_cap > kPListCapMax) list_cap = kPListCapMax;
  a.list_cap = (uint32_t)list_cap;
  const size_t smem = persist_smem(a.words, a.list_cap);
  if (smem > pd.smem_max) return cudaSuccess;
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
  void* fn = fs ? (void*)select_persistent_kernel<true> : (void*)select_persistent_kernel<false>;
  cudaError_t e = cudaLaunchCooperativeKernel(fn, dim3(G), dim3(kPThreads), args, smem, s);
  if (e != cudaSuccess) return e;
  count_launches(1);
  *used = true;
  return cudaSuccess;
}

}  // namespace kvt
