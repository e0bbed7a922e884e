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
// entry's touch count.  Counters are integers, so the order of the atomics does
// not matter.
//
// The 32 (pair, hit) counters are kept one per lane: for every event slot the
// warp takes six votes (valid, and the five bits of key = 2*pair + hit); lane L
// combines them into the mask of lanes whose key is L and adds its population
// count to a register.  No shared-memory atomics and no match instruction in the
// loop; a warp's 32 registers go to 32 shared counters once, at the end, and a
// block issues one 64-bit global atomic per non-zero counter.
constexpr uint32_t kEventVecs = 2;  // 4-event vectors a thread has in flight per iteration

struct EventCounter {
  uint32_t flip[5];  // bit b of the lane id clear -> all ones (selects lanes whose key bit b is clear)
  uint32_t cnt;      // events seen with key == lane id
  __device__ __forceinline__ void init(unsigned lane) {
#pragma unroll
    for (int b = 0; b < 5; ++b) flip[b] = ((lane >> b) & 1u) ? 0u : 0xFFFFFFFFu;
    cnt = 0;
  }
  // every lane of the warp must call it
  __device__ __forceinline__ void add(bool counted, uint32_t key) {
    uint32_t m = __ballot_sync(0xFFFFFFFFu, counted);
#pragma unroll
    for (int b = 0; b < 5; ++b) m &= __ballot_sync(0xFFFFFFFFu, (key >> b) & 1u) ^ flip[b];
    cnt += __popc(m);
  }
};

// The calling block's share of the events: thread `gtid` of `stride` takes
// kEventVecs vectors of four consecutive events at a time, so that all their
// scattered gathers are in flight together.  One byte per event is gathered: the entry's pair, whose bit 7 says
// that the entry is FREE.  Two consecutive events on the two entries of an
// aligned pair (2i, 2i+1) -- the normal case when a touched block reports all its
// heads -- share one 64-bit atomic on the two 32-bit touch counts (a carry out of
// the low count would need 2^32 touches, where the count wraps anyway).  Every
// thread of the block must call it (the votes need all lanes).  s_cnt: 32 zeroed
// shared-memory counters, index 2*pair + hit; returns the KV_DEV_* bits of
// refused events.
__device__ __forceinline__ uint32_t reduce_events(const uint32_t* __restrict__ ev_entry,
                                                  const uint8_t* __restrict__ ev_hit, uint64_t n_events,
                                                  const uint8_t* __restrict__ pair,
                                                  uint32_t* __restrict__ touch, uint64_t n, uint64_t gtid,
                                                  uint64_t stride, uint32_t* s_cnt) {
  const uint64_t n4 = n_events / 4;
  const uint64_t iters = (n4 + stride * kEventVecs - 1) / (stride * kEventVecs);  // same for every thread
  const unsigned lane = threadIdx.x & 31u;
  EventCounter ec;
  ec.init(lane);
  // ids are 32-bit, so the bound is too (an id can never reach 2^32 - 1 = "no entry")
  const uint32_t n32 = n > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)n;
  uint32_t bad = 0;
  bool bad_id = false, not_resident = false;
  for (uint64_t it = 0; it < iters; ++it) {
    uint32_t ids[kEventVecs][4], hit[kEventVecs][4], pr[kEventVecs][4];
    bool valid[kEventVecs];
#pragma unroll
    for (uint32_t u = 0; u < kEventVecs; ++u) {  // all event loads first
      const uint64_t v = (it * kEventVecs + u) * stride + gtid;
      valid[u] = v < n4;
      uint4 id4 = make_uint4(0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu);  // past the end: out of range
      uchar4 h4 = make_uchar4(0, 0, 0, 0);
      if (valid[u]) {
        id4 = reinterpret_cast<const uint4*>(ev_entry)[v];
        h4 = reinterpret_cast<const uchar4*>(ev_hit)[v];
      }
      ids[u][0] = id4.x; ids[u][1] = id4.y; ids[u][2] = id4.z; ids[u][3] = id4.w;
      hit[u][0] = h4.x != 0; hit[u][1] = h4.y != 0; hit[u][2] = h4.z != 0; hit[u][3] = h4.w != 0;
    }
#pragma unroll
    for (uint32_t u = 0; u < kEventVecs; ++u)
#pragma unroll
      for (int j = 0; j < 4; ++j)  // then all gathers, before any is used
        pr[u][j] = ids[u][j] < n32 ? pair[ids[u][j]] : kPairFree;
#pragma unroll
    for (uint32_t u = 0; u < kEventVecs; ++u) {
      bool ok[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const bool in = ids[u][j] < n32;
        ok[j] = !(pr[u][j] & kPairFree);   // (out of range gathered nothing: FREE)
        bad_id |= valid[u] && !in;
        not_resident |= in && !ok[j];
      }
#pragma unroll
      for (int j = 0; j < 4; j += 2) {
        if (ok[j] && ok[j + 1] && ids[u][j + 1] == ids[u][j] + 1u && !(ids[u][j] & 1u)) {
          atomicAdd(reinterpret_cast<unsigned long long*>(touch + ids[u][j]), 0x100000001ull);
        } else {
          if (ok[j]) atomicAdd(&touch[ids[u][j]], 1u);
          if (ok[j + 1]) atomicAdd(&touch[ids[u][j + 1]], 1u);
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) ec.add(ok[j], (pr[u][j] & 15u) * 2u + hit[u][j]);
    }
  }
  if (bad_id) bad |= KV_DEV_EVENT_BAD_ID;
  if (not_resident) bad |= KV_DEV_EVENT_NOT_RESIDENT;
  // ragged tail (n_events not a multiple of 4): first warp of the grid
  if (gtid < 32) {
    const uint64_t e = n4 * 4 + gtid;
    bool ok = false;
    uint32_t key = 0;
    if (e < n_events) {
      const uint32_t i = ev_entry[e];
      const uint32_t pr = i < n ? pair[i] : kPairFree;
      if (i >= n) {
        bad |= KV_DEV_EVENT_BAD_ID;
      } else if (pr & kPairFree) {
        bad |= KV_DEV_EVENT_NOT_RESIDENT;
      } else {
        ok = true;
        key = (pr & 15u) * 2u + (ev_hit[e] != 0);
        atomicAdd(&touch[i], 1u);
      }
    }
    ec.add(ok, key);
  }
  if (ec.cnt) atomicAdd(&s_cnt[lane], ec.cnt);
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

// touch and last_epoch are only written where an entry was touched.
__device__ __forceinline__ void entry_finish4(const EntryState& st, uint64_t v, EntryVec& x, const float* sP,
                                              int policy, uint32_t epoch, const HeadWeights& hw, float4& sc) {
  float4 w = make_float4(1.0f, 1.0f, 1.0f, 1.0f);
  if (hw.on) {
    w.x = head_weight(hw, 4 * v + 0);
    w.y = head_weight(hw, 4 * v + 1);
    w.z = head_weight(hw, 4 * v + 2);
    w.w = head_weight(hw, 4 * v + 3);
  }
  entry_step(x.e.x, x.d.x, x.t.x, x.pr.x, x.st.x, sP, policy, x.le.x, epoch, w.x, sc.x);
  entry_step(x.e.y, x.d.y, x.t.y, x.pr.y, x.st.y, sP, policy, x.le.y, epoch, w.y, sc.y);
  entry_step(x.e.z, x.d.z, x.t.z, x.pr.z, x.st.z, sP, policy, x.le.z, epoch, w.z, sc.z);
  entry_step(x.e.w, x.d.w, x.t.w, x.pr.w, x.st.w, sP, policy, x.le.w, epoch, w.w, sc.w);
  reinterpret_cast<float4*>(st.ema)[v] = x.e;
  reinterpret_cast<float4*>(st.score)[v] = sc;
  // touch counts of FREE entries are always zero (events on them are refused)
  if (x.t.x | x.t.y | x.t.z | x.t.w) {
    reinterpret_cast<uint4*>(st.touch)[v] = make_uint4(0, 0, 0, 0);
    if (x.t.x) st.last_epoch[4 * v + 0] = epoch;
    if (x.t.y) st.last_epoch[4 * v + 1] = epoch;
    if (x.t.z) st.last_epoch[4 * v + 2] = epoch;
    if (x.t.w) st.last_epoch[4 * v + 3] = epoch;
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
