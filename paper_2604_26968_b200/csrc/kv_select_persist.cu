// k-lowest selection as ONE cooperative, persistent launch.
//
// The multi-launch selection in kv_select.cu spends most of its time between
// kernels when the pool has a few million entries: ten dependent launches of
// 3-10 us each.  Here one CTA per SM stays resident for the whole selection.
// Each CTA owns a contiguous slice of the entries, converts its slice's scores
// to order-preserving keys ONCE and keeps them in shared memory (up to 40 K keys
// per SM, i.e. 6 M entries on 148 SMs; the rest of a larger slice is re-read
// from the score array, which then sits in L2), and the phases of the
// selection -- the histograms, the count, the ordered write -- are separated
// by grid-wide barriers instead of kernel boundaries.
//
// The grid barrier is a counter in global memory that every CTA increments and
// then polls.  A cooperative launch guarantees that all CTAs are resident, so
// the wait ends; it is nevertheless bounded, and a CTA that gives up sets
// KV_DEV_WAIT_EXPIRED and leaves (every other CTA then runs into the same limit).
//
// The same kernel also exists fused with the per-entry scoring pass (FUSED =
// true): every CTA first updates the entries of its own slice (posterior, EMA,
// score) and turns the fresh scores straight into keys -- the score array is
// written for the caller but never read back, and a kernel boundary disappears.
// The event reduction stays a launch of its own ahead of it: its scattered gathers
// and atomics ran 2.5x slower inside this kernel when that was tried, and a grid
// barrier costs about what the launch boundary does.
#include "kv_score_device.cuh"

namespace kvt {

constexpr uint32_t kPThreads = 1024;
constexpr uint32_t kPChunk = kPThreads * 4;             // 4096 entries: one 16-byte vector per thread
constexpr uint32_t kPKeyCap = 40960;                    // most keys kept in shared memory per CTA (160 KB)
constexpr uint32_t kPHistBins = 2048;
constexpr uint32_t kExcluded = 0xFFFFFFFFu;             // key of a non-candidate (FREE) entry
constexpr uint32_t kBarrierSpins = 1u << 22;
constexpr uint32_t kBracketShift = 11;                  // a bracket bin is 2^11 keys wide ...
constexpr uint32_t kBracketHalf = 1u << 21;             // ... and the 2,048 bins reach 2^21 keys to either side of the hint

static_assert(kPKeyCap % kPChunk == 0, "the cached part of a slice is a whole number of chunks");
static_assert(kPKeyCap < 65536, "per-CTA counts of the cached part are packed in 16 bits");

__device__ __forceinline__ uint32_t p_score_key(float s) {
  uint32_t b = __float_as_uint(s);
  if (b == 0x80000000u) b = 0u;  // -0.0 orders with +0.0
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Adds one to s_hist[bin] for every active lane; one atomic when the warp agrees
// on the bin (the common case while most scores are equal).
__device__ __forceinline__ void p_warp_hist_add(uint32_t* s_hist, bool active, uint32_t bin) {
  const unsigned m = __ballot_sync(0xFFFFFFFFu, active);
  if (m == 0) return;
  const int leader = __ffs(m) - 1;
  const uint32_t b0 = __shfl_sync(0xFFFFFFFFu, bin, leader);
  const bool same = !active || bin == b0;
  if (__all_sync(0xFFFFFFFFu, same)) {
    if ((int)(threadIdx.x & 31u) == leader) atomicAdd(&s_hist[b0], (uint32_t)__popc(m));
  } else if (active) {
    atomicAdd(&s_hist[bin], 1u);
  }
}

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
  unsigned long long per; // entries per CTA slice (multiple of 4)
  uint32_t cap;           // keys of a slice kept in shared memory (a multiple of kPChunk, at most kPKeyCap)
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
  extern __shared__ __align__(16) uint32_t s_keys[];  // a.cap keys
  __shared__ uint32_t s_hist[kPHistBins];
  __shared__ uint32_t s_hist_first[kPHistBins];  // the CTA's own first (bracket) histogram
  __shared__ uint32_t s_warp[32];
  __shared__ uint32_t s_pick[2];
  __shared__ float sP[16];
  const uint32_t t = threadIdx.x;
  unsigned int* bar = &a.sel->bar_arrive;
  const unsigned int G = gridDim.x;
  const unsigned long long s0 = (unsigned long long)blockIdx.x * a.per;
  const unsigned long long s1 = (s0 + a.per < a.n) ? s0 + a.per : a.n;
  const uint32_t len = s1 > s0 ? (uint32_t)(s1 - s0) : 0u;
  const uint32_t cached = len < a.cap ? len : a.cap;               // local [0, cached) lives in s_keys
  const uint32_t first_far = a.cap / kPChunk;                      // first chunk beyond the cache
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

  // Applies f(key) to every key of the slice, all threads in lock step (f may
  // vote across the warp): the cached part with a stride of one block, the far
  // part chunk by chunk from the arrays.
  auto for_each_key = [&](auto f) {
    const uint32_t iters = (cached + kPThreads - 1) / kPThreads;
    for (uint32_t i = 0; i < iters; ++i) {
      const uint32_t j = i * kPThreads + t;
      f(j < cached ? s_keys[j] : kExcluded);
    }
    for (uint32_t c = first_far; c < n_chunks; ++c) {
      uint32_t key[4];
      keys_from_arrays(c, key);
#pragma unroll
      for (int j = 0; j < 4; ++j) f(key[j]);
    }
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

  if constexpr (FUSED) {
    // reuse estimates from the totals plus this epoch's counts (final: the event
    // reduction is an earlier launch)
    if (t < 16) {
      unsigned long long h, m, wh, wm;
      const float P = posterior(a.pd, t, h, m);
      sP[t] = reuse_estimate(a.pd, t, P, h, m, wh, wm);
    }
  }

  // ---- phase A: keys into shared memory, and the first histogram ----
  // Without a hint the first histogram is digit 0 of a plain radix select (bits
  // 31..21 of every key).  With a hint -- tau of the previous selection over the
  // same number of keys -- it covers only the bracket [lo, lo + 2^22) around that
  // tau in 2,048 bins of 2^11 keys, and keys below lo are merely counted: scores
  // move little from one epoch to the next, so the k-th key is almost always
  // inside, few keys need an atomic, and one later pass (2^11 keys wide) finishes
  // the selection instead of two.  If rank k falls outside the bracket the plain
  // radix select runs after all, from the cached keys.
  const bool hint = a.sel->hint_valid != 0 && a.sel->hint_n == a.n;
  const uint32_t hint_tau = a.sel->hint_tau;
  const uint32_t base0 = hint ? (hint_tau > kBracketHalf ? hint_tau - kBracketHalf : 0u) : 0u;
  const uint32_t shift0 = hint ? kBracketShift : 21u;
  uint32_t n_below0 = 0;  // keys of this thread below the bracket
  auto first_pass = [&](uint32_t key) {
    n_below0 += (key < base0);  // (an excluded key is 0xFFFFFFFF: never below)
    const bool cand = key != kExcluded && key >= base0 && ((key - base0) >> shift0) < kPHistBins;
    p_warp_hist_add(s_hist, cand, (key - base0) >> shift0);
  };
  clear_hist();
  if constexpr (FUSED) {
    // the slice's entries go through the EMA and score update on the way; keys of
    // the far part are histogrammed here too, from registers
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
      if (c < first_far) {
        reinterpret_cast<uint4*>(s_keys)[c * kPThreads + t] = make_uint4(key[0], key[1], key[2], key[3]);
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) first_pass(key[j]);
      }
    }
    __syncthreads();
    const uint32_t iters = (cached + kPThreads - 1) / kPThreads;
    for (uint32_t i = 0; i < iters; ++i) {
      const uint32_t j = i * kPThreads + t;
      first_pass(j < cached ? s_keys[j] : kExcluded);
    }
  } else {
    const uint32_t cached_chunks = (cached + kPChunk - 1) / kPChunk;
#pragma unroll 4
    for (uint32_t c = 0; c < cached_chunks; ++c) {
      uint32_t key[4];
      keys_from_arrays(c, key);
      reinterpret_cast<uint4*>(s_keys)[c * kPThreads + t] = make_uint4(key[0], key[1], key[2], key[3]);
    }
    __syncthreads();
    for_each_key(first_pass);
  }
  flush_hist(a.hist, kPHistBins);
  uint32_t cta_below0 = 0;  // keys of this CTA's slice below the bracket
  if (hint) {
    (void)block_scan_excl(n_below0, s_warp, cta_below0);
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
    // ---- phases B, C: narrow [base, base + 2^shift) around rank k, one histogram per step ----
    // The current histogram is a.hist[h]; it was built over [base, base + 2048 << shift).
    // Every CTA reads the same global data, so all of them take the same path.
    uint32_t h = 0, nbar = 1, base = base0, shift = shift0;
    unsigned long long k_rem = a.k;
    uint32_t bin, before;
    bool found = true;
    bool clear_below = hint;
    bool bracket_hit = false;   // rank k was inside the bracket: two histograms in all
    uint32_t bin_first = 0;     // ... and this was its bin of the first one
    auto hist_pass = [&](uint32_t width_log2, uint32_t new_shift, uint32_t h_new) {
      // histogram of ((key - base) >> new_shift) over the keys in [base, base + 2^width_log2)
      clear_hist();
      const uint32_t top = width_log2 - new_shift;  // log2 of the number of bins
      for_each_key([&](uint32_t key) {
        const uint32_t d = key - base;
        p_warp_hist_add(s_hist, key != kExcluded && key >= base && ((d >> new_shift) >> top) == 0u, d >> new_shift);
      });
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
        // The CTA's own first histogram is still in s_hist: keep it.  Together with its own
        // second histogram it gives this slice's counts below and at tau without another
        // pass over the keys.
        bracket_hit = true;
        bin_first = bin;
        for (uint32_t b = t; b < kPHistBins; b += kPThreads) s_hist_first[b] = s_hist[b];
      } else {
        // rank k is outside the bracket: digit 0 of the plain radix select, from the cached keys
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
      if (shift == 0) break;
      const uint32_t new_shift = shift > 11u ? shift - 11u : 0u;
      const uint32_t h_new = (h + 1u) % 3u;
      hist_pass(shift, new_shift, h_new);
      ok = grid_barrier(bar, ++nbar * G);
      if (step < 2) stamp(3 + step);
      if (!ok) goto fail;
      retire(h);
      pick_bin(a.hist + h_new * kPHistBins, 1u << (shift - new_shift), k_rem, s_warp, s_pick, bin, before);
      h = h_new;
      shift = new_shift;
    }

    // ---- phase D: tau is known; count (key < tau, key == tau) in the slice ----
    const uint32_t tau = base;
    const unsigned long long need_eq = k_rem;
    if (bracket_hit) {
      // below tau = below the bracket + bins of the first histogram before rank k's bin +
      // bins of the second (single keys, still in s_hist) before tau; at tau = tau's bin
      const uint32_t bin_tau = tau - (base0 + (bin_first << kBracketShift));
      uint32_t v = 0;
      for (uint32_t b = t; b < kPHistBins; b += kPThreads)
        v += (b < bin_first ? s_hist_first[b] : 0u) + (b < bin_tau ? s_hist[b] : 0u);
      uint32_t tot_less;
      (void)block_scan_excl(v, s_warp, tot_less);
      if (t == 0) a.cta_counts[blockIdx.x] = make_uint2(cta_below0 + tot_less, s_hist[bin_tau]);
    } else {
      uint32_t n_less = 0, n_eq = 0;
      for_each_key([&](uint32_t key) {
        n_less += (key != kExcluded && key < tau);
        n_eq += (key != kExcluded && key == tau);
      });
      uint32_t tot_less, tot_eq;
      (void)block_scan_excl(n_less, s_warp, tot_less);
      (void)block_scan_excl(n_eq, s_warp, tot_eq);
      if (t == 0) a.cta_counts[blockIdx.x] = make_uint2(tot_less, tot_eq);
    }
    stamp(5);
    ok = grid_barrier(bar, ++nbar * G);
    stamp(6);
    if (!ok) goto fail;
    retire(h);

    // ---- phase E: ordered write ----
    unsigned long long less_before, eq_before;
    {
      uint32_t la = 0, ea = 0;  // partial sums over the CTAs before this one
      for (uint32_t g = t; g < blockIdx.x; g += kPThreads) {
        const uint2 cc = __ldcg(&a.cta_counts[g]);
        la += cc.x; ea += cc.y;
      }
      uint32_t tl, te;
      (void)block_scan_excl(la, s_warp, tl);
      (void)block_scan_excl(ea, s_warp, te);
      less_before = tl; eq_before = te;
    }
    // Position of a victim.  With L entries below tau and E entries equal to tau before it
    // in id order, an entry below tau goes to L + min(E, need_eq) and an entry equal to tau,
    // taken while E < need_eq, to L + E.  Everything before the current piece of the slice is
    // folded into pos0 and room once per piece, so the per-key arithmetic is 32-bit: ml and me
    // count inside the piece.
    unsigned long long pos0 = 0;
    uint32_t room = 0;
    auto set_piece = [&]() {
      pos0 = less_before + (eq_before < need_eq ? eq_before : need_eq);
      const unsigned long long left = need_eq > eq_before ? need_eq - eq_before : 0ull;
      room = left > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)left;
    };
    auto emit = [&](uint32_t key, unsigned long long id, uint32_t& ml, uint32_t& me) {
      if (key > tau) return;   // most keys (an excluded key is 0xFFFFFFFF)
      if (key < tau) {
        const unsigned long long pos = pos0 + ml + (me < room ? me : room);
        if (pos < a.k) a.victims[pos] = (uint32_t)id;
        ++ml;
      } else if (key != kExcluded) {
        if (me < room) {
          const unsigned long long pos = pos0 + ml + me;
          if (pos < a.k) a.victims[pos] = (uint32_t)id;
        }
        ++me;
      }
    };
    if (found) {
      // cached part: every thread owns a contiguous run of L keys (L odd: the
      // strided shared-memory reads of a warp then fall into distinct banks)
      {
        uint32_t L = (cached + kPThreads - 1) / kPThreads;
        L |= 1u;
        const uint32_t j0 = t * L;
        const uint32_t j1 = (j0 + L < cached) ? j0 + L : cached;
        uint32_t v = 0;
        for (uint32_t j = j0; j < j1; ++j) {
          const uint32_t key = s_keys[j];
          v += (key < tau) + ((uint32_t)(key == tau && key != kExcluded) << 16);
        }
        uint32_t total;
        const uint32_t excl = block_scan_excl(v, s_warp, total);
        set_piece();
        uint32_t ml = excl & 0xFFFFu, me = excl >> 16;
        for (uint32_t j = j0; j < j1; ++j) emit(s_keys[j], s0 + j, ml, me);
        less_before += total & 0xFFFFu;
        eq_before += total >> 16;
      }
      // far part: chunk by chunk, a vector per thread
      for (uint32_t c = first_far; c < n_chunks; ++c) {
        uint32_t key[4];
        keys_from_arrays(c, key);
        uint32_t v = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j)
          v += (key[j] < tau) + ((uint32_t)(key[j] == tau && key[j] != kExcluded) << 16);
        uint32_t total;
        const uint32_t excl = block_scan_excl(v, s_warp, total);
        set_piece();
        uint32_t ml = excl & 0xFFFFu, me = excl >> 16;
        const unsigned long long i0 = s0 + (unsigned long long)c * kPChunk + 4ull * t;
#pragma unroll
        for (int j = 0; j < 4; ++j) emit(key[j], i0 + j, ml, me);
        less_before += total & 0xFFFFu;
        eq_before += total >> 16;
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

// Launches the persistent selection (fused with the entry pass when fs is given)
// if the device can hold one CTA per SM of it co-resident; *used = false (and
// nothing launched) otherwise.
cudaError_t launch_select_persistent(const EntryState& st, uint64_t k, uint32_t* d_victims,
                                     const Workspace& ws, cudaStream_t s, bool* used, const FusedScore* fs) {
  *used = false;
  static int state = 0;  // 0 = not probed, 1 = usable, -1 = not usable
  static int n_sm = 0;
  const size_t smem_max = (size_t)kPKeyCap * 4;
  if (state == 0) {
    int dev = 0, coop = 0, blocks = 0, blocks_f = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cudaGetLastError();
    cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
    cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    cudaError_t e = cudaFuncSetAttribute(select_persistent_kernel<false>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(select_persistent_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               (int)smem_max);
    if (e == cudaSuccess)
      e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks, select_persistent_kernel<false>,
                                                        (int)kPThreads, smem_max);
    if (e == cudaSuccess)
      e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks_f, select_persistent_kernel<true>,
                                                        (int)kPThreads, smem_max);
    state = (e == cudaSuccess && coop && blocks >= 1 && blocks_f >= 1 && n_sm > 0) ? 1 : -1;
    (void)cudaGetLastError();
  }
  if (state != 1) return cudaSuccess;
  unsigned int G = (unsigned int)n_sm;
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
  // Shared memory only for the keys a slice has, and never all of it: what the key cache
  // does not take stays with the L1, whose lines hold the loads in flight.  Measured on
  // 11.8 M entries: with 192 KB of keys per SM the streaming entry pass of this kernel took
  // 68 us, with 160 KB 61 us (and the whole call 227 -> 213 us) although more keys are then
  // re-read from L2; a 3.1 M pool, whose slices need 96 KB, went from 66.7 to 63.5 us.
  const uint64_t want = (a.per + kPChunk - 1) / kPChunk * kPChunk;
  a.cap = (uint32_t)(want < kPKeyCap ? want : kPKeyCap);
  const size_t smem = (size_t)a.cap * 4;
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
