// Device-side pieces of the scoring pass, shared by the stand-alone scoring
// kernels (kv_score.cu) and the fused score + select kernel (kv_select_persist.cu).
//
// All binary32 arithmetic uses the explicitly rounded intrinsics (__fmul_rn,
// __fadd_rn, __fsub_rn, __fdiv_rn), which the compiler never contracts into a
// fused multiply-add, and denormals are kept (no flush-to-zero), so results
// are bit-identical to the same operations done one at a time on a CPU.
#pragma once
#include "kvtier_internal.cuh"

namespace kvt {

// ---- event reduction ---------------------------------------------------------
// Each event adds one to the (pair, hit) counter of its entry's pair -- the
// alpha += 1 / beta += 1 update of the Bayesian reuse section -- and one to the
// entry's touch count.  Counters are integers, so the order of the additions
// does not matter.
//
// Pair counters: every thread owns 16 packed counters in shared memory (one per
// pair: events in the low half, hits in the high half), laid out pair-major so
// that the threads of a warp always fall into 32 different banks.  Counting an
// event is a plain read-add-write of the thread's own word: no vote, no atomic.
// The block adds its columns up once at the end.
//
// Touch counts: every update is a 64-bit atomic on the aligned pair of 32-bit
// counts (touch[2i], touch[2i+1]) -- adding 1, 1 << 32 or both -- so that all
// atomics on a word have one size.  (A carry out of the low count would need
// 2^32 touches of one entry in one epoch, where the count wraps anyway.)  The
// one exception is the last entry of an array of odd length, whose partner
// would lie outside the array: it takes 32-bit atomics, and only those.
//
// Traces in which a touched block reports all its heads hand every thread four
// consecutive entries (an aligned group of four ids): one 4-byte load then
// fetches their pairs and FREE bits, and two atomics count the four touches.
constexpr uint32_t kEventVecs = 2;          // 4-event vectors a thread has in flight per iteration
constexpr uint32_t kEventFlushIters = 4096; // iterations between flushes: 8 events each, below 2^16

struct EventVec {
  uint32_t id[4];
  uint32_t hit4;   // bit 8j+7 set: event j carried a hit flag
  uint32_t pr4;    // byte j: pair byte of event j's entry (bit 7 = FREE or out of range)
  bool valid, run; // vector inside the trace; ids are an aligned run of four inside the pool
};

// bit 7 of every non-zero byte
__device__ __forceinline__ uint32_t nonzero_bytes(uint32_t x) {
  return (((x & 0x7F7F7F7Fu) + 0x7F7F7F7Fu) | x) & 0x80808080u;
}

__device__ __forceinline__ void touch_add(uint32_t* __restrict__ touch, uint32_t i, uint32_t n32,
                                          unsigned long long inc_pair) {
  // inc_pair: what to add to the aligned pair that contains entry i
  if ((i | 1u) < n32)
    atomicAdd(reinterpret_cast<unsigned long long*>(touch + (i & ~1u)), inc_pair);
  else
    atomicAdd(&touch[i], 1u);   // last entry of an odd-length array (i is even, inc_pair is 1)
}

// The calling block's share of the events.  s_cnt: kThreads * 16 words of shared
// memory, zero on entry; on return word [p * blockDim.x + t] holds thread t's
// counts for pair p (events | hits << 16) since the last flush.  delta: the 32
// global epoch counters (index 2 * pair + hit).  Returns the KV_DEV_* bits of
// refused events.  Every thread of the block must call it.
__device__ __forceinline__ uint32_t reduce_events(const uint32_t* __restrict__ ev_entry,
                                                  const uint8_t* __restrict__ ev_hit, uint64_t n_events,
                                                  const uint8_t* __restrict__ pair,
                                                  uint32_t* __restrict__ touch, uint64_t n, uint64_t gtid,
                                                  uint64_t stride, uint32_t* s_cnt,
                                                  unsigned long long* __restrict__ delta) {
  const uint64_t n4 = n_events / 4;
  const uint64_t iters = (n4 + stride * kEventVecs - 1) / (stride * kEventVecs);  // same for every thread
  // ids are 32-bit, so the bound is too (an id can never reach 2^32 - 1 = "no entry")
  const uint32_t n32 = n > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)n;
  uint32_t* my = s_cnt + threadIdx.x;
  const uint32_t col = blockDim.x;
  bool bad_id = false, not_resident = false;

  // adds the block's columns to the global counters and clears them; the 32 sums
  // go out as one warp's 32 neighbouring atomics (a single request per cache line)
  auto flush = [&]() {
    __shared__ uint32_t s_tot[32];
    __syncthreads();
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u, n_warps = blockDim.x >> 5;
    for (uint32_t p = warp; p < 16; p += n_warps) {
      uint32_t ev = 0, hi = 0;
      for (uint32_t t = lane; t < col; t += 32) {
        const uint32_t c = s_cnt[p * col + t];
        s_cnt[p * col + t] = 0;
        ev += c & 0xFFFFu;
        hi += c >> 16;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        ev += __shfl_xor_sync(0xFFFFFFFFu, ev, o);
        hi += __shfl_xor_sync(0xFFFFFFFFu, hi, o);
      }
      if (lane == 0) {
        s_tot[2 * p + 1] = hi;
        s_tot[2 * p] = ev - hi;
      }
    }
    __syncthreads();
    if (threadIdx.x < 32 && s_tot[threadIdx.x])
      atomicAdd(&delta[threadIdx.x], (unsigned long long)s_tot[threadIdx.x]);
    __syncthreads();
  };
  // counts event j of a vector (pair byte and hit bit already extracted)
  auto count = [&](uint32_t prj, uint32_t hitbit) { my[(prj & 15u) * col] += 1u + (hitbit << 16); };

  for (uint64_t it = 0; it < iters; ++it) {
    EventVec x[kEventVecs];
#pragma unroll
    for (uint32_t u = 0; u < kEventVecs; ++u) {  // all event loads first
      const uint64_t v = (it * kEventVecs + u) * stride + gtid;
      x[u].valid = v < n4;
      uint4 id4 = make_uint4(0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu);  // past the end: out of range
      uint32_t h4 = 0;
      if (x[u].valid) {
        id4 = reinterpret_cast<const uint4*>(ev_entry)[v];
        h4 = reinterpret_cast<const uint32_t*>(ev_hit)[v];
      }
      x[u].id[0] = id4.x; x[u].id[1] = id4.y; x[u].id[2] = id4.z; x[u].id[3] = id4.w;
      x[u].hit4 = nonzero_bytes(h4);
      x[u].run = !(id4.x & 3u) && id4.y == id4.x + 1u && id4.z == id4.x + 2u && id4.w == id4.x + 3u &&
                 id4.w < n32;
    }
#pragma unroll
    for (uint32_t u = 0; u < kEventVecs; ++u) {  // then all gathers, before any is used
      if (x[u].run) {
        x[u].pr4 = *reinterpret_cast<const uint32_t*>(pair + x[u].id[0]);
      } else {
        uint32_t pr4 = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j)
          pr4 |= (uint32_t)(x[u].id[j] < n32 ? pair[x[u].id[j]] : (uint8_t)kPairFree) << (8 * j);
        x[u].pr4 = pr4;
      }
    }
#pragma unroll
    for (uint32_t u = 0; u < kEventVecs; ++u) {
      const uint32_t pr4 = x[u].pr4, hit4 = x[u].hit4;
      if (x[u].run && !(pr4 & 0x80808080u)) {
        // four resident entries in a row: two atomics, four counts
        unsigned long long* t2 = reinterpret_cast<unsigned long long*>(touch + x[u].id[0]);
        atomicAdd(t2, 0x100000001ull);
        atomicAdd(t2 + 1, 0x100000001ull);
#pragma unroll
        for (int j = 0; j < 4; ++j) count(pr4 >> (8 * j), (hit4 >> (8 * j + 7)) & 1u);
        continue;
      }
      if (!x[u].valid) continue;
      bool ok[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const bool in = x[u].id[j] < n32;
        ok[j] = !((pr4 >> (8 * j)) & kPairFree);   // (out of range gathered nothing: FREE)
        bad_id |= !in;
        not_resident |= in && !ok[j];
      }
#pragma unroll
      for (int j = 0; j < 4; j += 2) {
        const uint32_t i0 = x[u].id[j], i1 = x[u].id[j + 1];
        if (ok[j] && ok[j + 1] && i1 == i0 + 1u && !(i0 & 1u)) {
          atomicAdd(reinterpret_cast<unsigned long long*>(touch + i0), 0x100000001ull);
        } else {
          if (ok[j]) touch_add(touch, i0, n32, (i0 & 1u) ? (1ull << 32) : 1ull);
          if (ok[j + 1]) touch_add(touch, i1, n32, (i1 & 1u) ? (1ull << 32) : 1ull);
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (ok[j]) count(pr4 >> (8 * j), (hit4 >> (8 * j + 7)) & 1u);
    }
    if ((it + 1) % kEventFlushIters == 0) flush();   // (uniform over the block)
  }
  uint32_t bad = 0;
  if (bad_id) bad |= KV_DEV_EVENT_BAD_ID;
  if (not_resident) bad |= KV_DEV_EVENT_NOT_RESIDENT;
  // ragged tail (n_events not a multiple of 4): first threads of the grid
  if (gtid < 3) {
    const uint64_t e = n4 * 4 + gtid;
    if (e < n_events) {
      const uint32_t i = ev_entry[e];
      const uint32_t pr = i < n32 ? pair[i] : kPairFree;
      if (i >= n32) {
        bad |= KV_DEV_EVENT_BAD_ID;
      } else if (pr & kPairFree) {
        bad |= KV_DEV_EVENT_NOT_RESIDENT;
      } else {
        count(pr, ev_hit[e] != 0);
        touch_add(touch, i, n32, (i & 1u) ? (1ull << 32) : 1ull);
      }
    }
  }
  flush();
  return bad;
}

// ---- head-granular weight -------------------------------------------------------
// Weight of entry i's (layer, KV head) from the partition's [layer][KV head]
// table (head-granular eviction section); 1 for partitions that are not weighted.
// id = base + (layer * blocks_per_layer + block) * heads + head.
__device__ __forceinline__ float head_weight(const HeadWeights& hw, uint64_t i) {
  int q = 0;
  while (q + 1 < hw.n_parts && i >= hw.base[q + 1]) ++q;
  if (!((hw.on >> q) & 1u)) return 1.0f;
  const uint32_t local = (uint32_t)(i - hw.base[q]);
  const uint32_t layer = local / hw.per_layer[q], head = local % hw.heads[q];
  return __ldg(&hw.w[hw.w_off[q] + layer * hw.heads[q] + head]);
}

// ---- per-entry step -----------------------------------------------------------
// One step of the per-entry EMA, then the eviction score of the chosen policy:
// 0 = reuse estimate x EMA importance, 1 = EMA only, 2 = LRU (epoch of the last
// touch, this epoch's touches included) -- the three policies the paper compares.
// w: weight of the entry's (layer, head), which the two importance-based policies
// multiply in (1 = unweighted; x * 1 is exact).
__device__ __forceinline__ void entry_step(float& ema, float decay, uint32_t touch, uint32_t pair,
                                           uint32_t state, const float* sP, int policy,
                                           uint32_t last_epoch, uint32_t epoch, float w, float& score) {
  if (state == KV_STATE_RESIDENT) {
    const float x = __uint2float_rn(touch);
    const float t1 = __fmul_rn(decay, ema);
    const float t2 = __fsub_rn(1.0f, decay);
    const float t3 = __fmul_rn(t2, x);
    ema = __fadd_rn(t1, t3);
    if (policy == 0) score = __fmul_rn(__fmul_rn(sP[pair & 15u], ema), w);
    else if (policy == 1) score = __fmul_rn(ema, w);
    else score = __uint2float_rn(touch ? epoch : last_epoch);
  } else {
    score = __int_as_float(0x7F800000);  // +inf: not a candidate
  }
}

// ---- the predictor ---------------------------------------------------------------
struct Predictor {
  uint64_t* hits;
  uint64_t* misses;
  float* P;
  float alpha0, beta0;
  unsigned long long* delta;   // [32] this epoch's counts, index 2*pair + hit
  unsigned int* ticket;        // blocks that have finished (the last one commits)
  int policy;
  float kappa;                 // confidence saturation constant of the blend
  uint32_t window;             // epochs in the sliding window; 0 = no blending
  BlendState* blend;
};

// Reuse estimate of pair p: the posterior P, or -- when a window is set -- its
// confidence-weighted blend with the hit frequency of the last `window` epochs
// (the current one included).  The paper describes the blend in words (Bayesian
// reuse section: confidence saturates toward 1 as observations accumulate; young
// pairs lean on the windowed frequency); the form used is c = n/(n+kappa),
// estimate = c*P + (1-c)*f, every operation rounded once.  wm/wh receive the
// window's new sums.
__device__ __forceinline__ float reuse_estimate(const Predictor& pd, unsigned p, float P,
                                                unsigned long long h, unsigned long long m,
                                                unsigned long long& wh, unsigned long long& wm) {
  wh = wm = 0;
  if (pd.window == 0) return P;
  const uint32_t head = pd.blend->head;
  wm = pd.blend->wsum[2 * p] - pd.blend->win[head * 32 + 2 * p] + __ldcg(&pd.delta[2 * p]);
  wh = pd.blend->wsum[2 * p + 1] - pd.blend->win[head * 32 + 2 * p + 1] + __ldcg(&pd.delta[2 * p + 1]);
  const float n = __ull2float_rn(h + m);
  const float c = __fdiv_rn(n, __fadd_rn(n, pd.kappa));
  const float fh = __ull2float_rn(wh);
  const float fn = __ull2float_rn(wh + wm);
  const float f = fn > 0.0f ? __fdiv_rn(fh, fn) : P;
  const float t1 = __fmul_rn(c, P);
  const float t2 = __fsub_rn(1.0f, c);
  const float t3 = __fmul_rn(t2, f);
  return __fadd_rn(t1, t3);
}

// Posterior mean of Eq. "reuse" for pair p from the running totals plus this
// epoch's counts: P = alpha / (alpha + beta), alpha = alpha0 + hits, beta =
// beta0 + misses.  The 64-bit counts convert to binary32 with round to nearest
// even; the division is IEEE.  The epoch's counts are read from L2 (other blocks
// of the same launch may have produced them).
__device__ __forceinline__ float posterior(const Predictor& pd, unsigned p, unsigned long long& h,
                                           unsigned long long& m) {
  h = pd.hits[p] + __ldcg(&pd.delta[2 * p + 1]);
  m = pd.misses[p] + __ldcg(&pd.delta[2 * p]);
  const float a = __fadd_rn(pd.alpha0, __ull2float_rn(h));
  const float b = __fadd_rn(pd.beta0, __ull2float_rn(m));
  return __fdiv_rn(a, __fadd_rn(a, b));
}

// End of an epoch, run by lanes 0..15 of one warp (p = lane) once every block
// has read the counters: folds the epoch's counts into the totals, publishes P
// and the estimate, advances the blend's window and clears the counts.
__device__ __forceinline__ void commit_predictor(const Predictor& pd, unsigned p) {
  unsigned long long h, m, wh, wm;
  const float P = posterior(pd, p, h, m);
  const float est = reuse_estimate(pd, p, P, h, m, wh, wm);
  pd.hits[p] = h;
  pd.misses[p] = m;
  pd.P[p] = P;
  pd.blend->estimate[p] = est;
  const uint32_t head = pd.blend->head;
  __syncwarp(0xFFFFu);  // all 16 lanes have read the head and the expiring window slot
  if (pd.window > 0) {   // this epoch's counts replace the oldest slot of the window
    pd.blend->win[head * 32 + 2 * p] = __ldcg(&pd.delta[2 * p]);
    pd.blend->win[head * 32 + 2 * p + 1] = __ldcg(&pd.delta[2 * p + 1]);
    pd.blend->wsum[2 * p] = wm;
    pd.blend->wsum[2 * p + 1] = wh;
    if (p == 0) pd.blend->head = (head + 1) % pd.window;
  }
  pd.delta[2 * p] = 0;
  pd.delta[2 * p + 1] = 0;
}

// Four consecutive entries (a 16-byte vector of each array) through entry_step,
// in two halves so that a caller can have the next vector's loads in flight
// while it finishes this one.  v indexes vectors.  The touch counts are read from
// L2: other blocks' atomics made them.
struct EntryVec {
  float4 e, d;
  uint4 t, le;
  uchar4 pr, st;
};

__device__ __forceinline__ EntryVec entry_load4(const EntryState& st, uint64_t v, int policy) {
  EntryVec x;
  x.e = reinterpret_cast<const float4*>(st.ema)[v];
  x.d = reinterpret_cast<const float4*>(st.decay)[v];
  x.t = __ldcg(reinterpret_cast<const uint4*>(st.touch) + v);
  x.pr = reinterpret_cast<const uchar4*>(st.pair)[v];
  x.st = reinterpret_cast<const uchar4*>(st.state)[v];
  x.le = make_uint4(0, 0, 0, 0);
  if (policy == 2) x.le = reinterpret_cast<const uint4*>(st.last_epoch)[v];  // only LRU reads it
  return x;
}

// touch and last_epoch are only written where an entry was touched.  kPlain: the caller
// knows that the policy is the Bayesian product and that no partition is weighted (the
// policy and weight tests then fold away at compile time).
template <bool kPlain = false>
__device__ __forceinline__ void entry_finish4(const EntryState& st, uint64_t v, EntryVec& x, const float* sP,
                                              int policy, uint32_t epoch, const HeadWeights& hw, float4& sc) {
  float4 w = make_float4(1.0f, 1.0f, 1.0f, 1.0f);
  if (!kPlain && hw.on) {
    w.x = head_weight(hw, 4 * v + 0);
    w.y = head_weight(hw, 4 * v + 1);
    w.z = head_weight(hw, 4 * v + 2);
    w.w = head_weight(hw, 4 * v + 3);
  }
  const int pol = kPlain ? 0 : policy;
  entry_step(x.e.x, x.d.x, x.t.x, x.pr.x, x.st.x, sP, pol, x.le.x, epoch, w.x, sc.x);
  entry_step(x.e.y, x.d.y, x.t.y, x.pr.y, x.st.y, sP, pol, x.le.y, epoch, w.y, sc.y);
  entry_step(x.e.z, x.d.z, x.t.z, x.pr.z, x.st.z, sP, pol, x.le.z, epoch, w.z, sc.z);
  entry_step(x.e.w, x.d.w, x.t.w, x.pr.w, x.st.w, sP, pol, x.le.w, epoch, w.w, sc.w);
  reinterpret_cast<float4*>(st.ema)[v] = x.e;
  reinterpret_cast<float4*>(st.score)[v] = sc;
  // touch counts of FREE entries are always zero (events on them are refused)
  if (x.t.x | x.t.y | x.t.z | x.t.w) {
    reinterpret_cast<uint4*>(st.touch)[v] = make_uint4(0, 0, 0, 0);
    if (x.t.x && x.t.y && x.t.z && x.t.w) {   // a block that reported all its heads: one store
      reinterpret_cast<uint4*>(st.last_epoch)[v] = make_uint4(epoch, epoch, epoch, epoch);
    } else {
      if (x.t.x) st.last_epoch[4 * v + 0] = epoch;
      if (x.t.y) st.last_epoch[4 * v + 1] = epoch;
      if (x.t.z) st.last_epoch[4 * v + 2] = epoch;
      if (x.t.w) st.last_epoch[4 * v + 3] = epoch;
    }
  }
}

// The same for one entry (ragged ends).
__device__ __forceinline__ void entry_update1(const EntryState& st, uint64_t i, const float* sP, int policy,
                                              uint32_t epoch, const HeadWeights& hw, float& sc,
                                              uint32_t& state1) {
  float e = st.ema[i];
  const uint32_t t = __ldcg(&st.touch[i]);
  state1 = st.state[i];
  const float w = hw.on ? head_weight(hw, i) : 1.0f;
  entry_step(e, st.decay[i], t, st.pair[i], state1, sP, policy, policy == 2 ? st.last_epoch[i] : 0u, epoch, w,
             sc);
  st.ema[i] = e;
  st.score[i] = sc;
  if (t) {
    st.touch[i] = 0;
    st.last_epoch[i] = epoch;
  }
}

}  // namespace kvt
