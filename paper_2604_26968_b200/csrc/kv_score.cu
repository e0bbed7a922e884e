// Scoring kernels: event reduction, and the fused posterior + EMA + score pass.
//
// All binary32 arithmetic uses the explicitly rounded intrinsics (__fmul_rn,
// __fadd_rn, __fsub_rn, __fdiv_rn), which the compiler never contracts into a
// fused multiply-add, and denormals are kept (no flush-to-zero), so results
// are bit-identical to the same operations done one at a time on a CPU.
#include "kvtier_internal.cuh"

namespace kvt {

// ---- event reduction ---------------------------------------------------------
// Each event adds one to the (pair, hit) counter of its entry's pair -- the
// alpha += 1 / beta += 1 update of the Bayesian reuse section -- and one to the
// entry's touch count.  Counters are integers, so the order of the atomics does
// not matter.  A thread takes four consecutive events at a time so that its
// eight scattered gathers (state and pair of four entries) are in flight
// together; lanes of a warp that hit the same counter are merged first
// (match.any), then a 32-counter shared-memory table per block, then one 64-bit
// global atomic per non-zero counter per block.
__device__ __forceinline__ void count_event(uint32_t key, uint32_t* s_cnt, unsigned lane) {
  const unsigned peers = __match_any_sync(0xFFFFFFFFu, key);
  if (key < 32 && lane == (unsigned)(__ffs(peers) - 1)) atomicAdd(&s_cnt[key], __popc(peers));
}

__global__ void __launch_bounds__(kThreads)
event_reduce_kernel(const uint32_t* __restrict__ ev_entry, const uint8_t* __restrict__ ev_hit,
                    uint64_t n_events, const uint8_t* __restrict__ pair,
                    const uint8_t* __restrict__ state, uint32_t* __restrict__ touch, uint64_t n,
                    unsigned long long* __restrict__ delta, uint32_t* __restrict__ status) {
  __shared__ uint32_t s_cnt[32];
  if (threadIdx.x < 32) s_cnt[threadIdx.x] = 0;
  __syncthreads();
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  const uint64_t gtid = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const uint64_t n4 = n_events / 4;
  const uint64_t iters = (n4 + stride - 1) / stride;  // same for every thread: the votes need all lanes
  const unsigned lane = threadIdx.x & 31u;
  uint32_t bad = 0;
  for (uint64_t it = 0; it < iters; ++it) {
    const uint64_t v = it * stride + gtid;
    const bool valid = v < n4;
    uint4 id4 = make_uint4(0, 0, 0, 0);
    uchar4 h4 = make_uchar4(0, 0, 0, 0);
    if (valid) {
      id4 = reinterpret_cast<const uint4*>(ev_entry)[v];
      h4 = reinterpret_cast<const uchar4*>(ev_hit)[v];
    }
    const uint32_t ids[4] = {id4.x, id4.y, id4.z, id4.w};
    const uint32_t hit[4] = {h4.x != 0, h4.y != 0, h4.z != 0, h4.w != 0};
    uint32_t st[4], pr[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {  // all gathers issued before any is used
      const bool in = valid && ids[j] < n;
      st[j] = in ? state[ids[j]] : 0xFFu;
      pr[j] = in ? pair[ids[j]] : 0u;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t key = 32;  // 32 = nothing to count
      if (valid) {
        if (ids[j] >= n) {
          bad |= KV_DEV_EVENT_BAD_ID;
        } else if (st[j] != KV_STATE_RESIDENT) {
          bad |= KV_DEV_EVENT_NOT_RESIDENT;
        } else {
          key = pr[j] * 2u + hit[j];
          atomicAdd(&touch[ids[j]], 1u);
        }
      }
      count_event(key, s_cnt, lane);
    }
  }
  // ragged tail (n_events not a multiple of 4): first warp of the grid
  if (blockIdx.x == 0 && threadIdx.x < 32) {
    const uint64_t e = n4 * 4 + threadIdx.x;
    uint32_t key = 32;
    if (e < n_events) {
      const uint32_t i = ev_entry[e];
      if (i >= n) {
        bad |= KV_DEV_EVENT_BAD_ID;
      } else if (state[i] != KV_STATE_RESIDENT) {
        bad |= KV_DEV_EVENT_NOT_RESIDENT;
      } else {
        key = (uint32_t)pair[i] * 2u + (ev_hit[e] != 0);
        atomicAdd(&touch[i], 1u);
      }
    }
    count_event(key, s_cnt, lane);
  }
  if (bad) atomicOr(status, bad);
  __syncthreads();
  if (threadIdx.x < 32 && s_cnt[threadIdx.x])
    atomicAdd(&delta[threadIdx.x], (unsigned long long)s_cnt[threadIdx.x]);
}

cudaError_t launch_event_reduce(const uint32_t* ev_entry, const uint8_t* ev_hit, uint64_t n_events,
                                const EntryState& st, const Workspace& ws, cudaStream_t s) {
  if (n_events == 0) return cudaSuccess;
  uint64_t blocks = (n_events / 4 + kThreads - 1) / kThreads;
  if (blocks == 0) blocks = 1;
  const uint64_t cap = (uint64_t)kSMs * 8;
  if (blocks > cap) blocks = cap;
  event_reduce_kernel<<<(unsigned)blocks, kThreads, 0, s>>>(ev_entry, ev_hit, n_events, st.pair,
                                                            st.state, st.touch, st.n, ws.delta,
                                                            ws.status);
  count_launches(1);
  return cudaGetLastError();
}

// ---- fused entry pass ------------------------------------------------------------
// One step of the per-entry EMA, then the eviction score of the chosen policy:
// 0 = reuse estimate x EMA importance, 1 = EMA only, 2 = LRU (epoch of the last
// touch, this epoch's touches included) -- the three policies the paper compares.
__device__ __forceinline__ void entry_step(float& ema, float decay, uint32_t touch, uint32_t pair,
                                           uint32_t state, const float* sP, int policy,
                                           uint32_t last_epoch, uint32_t epoch, float& score) {
  if (state == KV_STATE_RESIDENT) {
    const float x = __uint2float_rn(touch);
    const float t1 = __fmul_rn(decay, ema);
    const float t2 = __fsub_rn(1.0f, decay);
    const float t3 = __fmul_rn(t2, x);
    ema = __fadd_rn(t1, t3);
    if (policy == 0) score = __fmul_rn(sP[pair & 15u], ema);
    else if (policy == 1) score = ema;
    else score = __uint2float_rn(touch ? epoch : last_epoch);
  } else {
    score = __int_as_float(0x7F800000);  // +inf: not a candidate
  }
}

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
  wm = pd.blend->wsum[2 * p] - pd.blend->win[head * 32 + 2 * p] + pd.delta[2 * p];
  wh = pd.blend->wsum[2 * p + 1] - pd.blend->win[head * 32 + 2 * p + 1] + pd.delta[2 * p + 1];
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
// even; the division is IEEE.
__device__ __forceinline__ float posterior(const Predictor& pd, unsigned p, unsigned long long& h,
                                           unsigned long long& m) {
  h = pd.hits[p] + pd.delta[2 * p + 1];
  m = pd.misses[p] + pd.delta[2 * p];
  const float a = __fadd_rn(pd.alpha0, __ull2float_rn(h));
  const float b = __fadd_rn(pd.beta0, __ull2float_rn(m));
  return __fdiv_rn(a, __fadd_rn(a, b));
}

// Every block forms the 16 posteriors itself (32 counters, read-only here), then
// streams its share of the entries: four per thread and iteration, every array
// read and written with 16-byte (for the byte arrays 4-byte) accesses.  touch and
// last_epoch are only written where an entry was touched.  The last block to
// finish folds the epoch's counts into the totals, clears them and publishes P;
// by then every block has read them.
__global__ void __launch_bounds__(kThreads)
entry_update_kernel(float* __restrict__ ema, const float* __restrict__ decay,
                    uint32_t* __restrict__ touch, uint32_t* __restrict__ last_epoch,
                    const uint8_t* __restrict__ pair, const uint8_t* __restrict__ state,
                    float* __restrict__ score, const Predictor pd, uint64_t n, uint32_t epoch) {
  __shared__ float sP[16];
  __shared__ bool s_last;
  const int policy = pd.policy;
  if (threadIdx.x < 16) {
    unsigned long long h, m, wh, wm;
    const float P = posterior(pd, threadIdx.x, h, m);
    sP[threadIdx.x] = reuse_estimate(pd, threadIdx.x, P, h, m, wh, wm);
  }
  __syncthreads();
  const uint64_t n4 = n / 4;
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t v = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; v < n4; v += stride) {
    float4 e = reinterpret_cast<const float4*>(ema)[v];
    const float4 d = reinterpret_cast<const float4*>(decay)[v];
    const uint4 t = reinterpret_cast<const uint4*>(touch)[v];
    const uchar4 pr = reinterpret_cast<const uchar4*>(pair)[v];
    const uchar4 st = reinterpret_cast<const uchar4*>(state)[v];
    uint4 le = make_uint4(0, 0, 0, 0);
    if (policy == 2) le = reinterpret_cast<const uint4*>(last_epoch)[v];  // only LRU reads it
    float4 sc;
    entry_step(e.x, d.x, t.x, pr.x, st.x, sP, policy, le.x, epoch, sc.x);
    entry_step(e.y, d.y, t.y, pr.y, st.y, sP, policy, le.y, epoch, sc.y);
    entry_step(e.z, d.z, t.z, pr.z, st.z, sP, policy, le.z, epoch, sc.z);
    entry_step(e.w, d.w, t.w, pr.w, st.w, sP, policy, le.w, epoch, sc.w);
    reinterpret_cast<float4*>(ema)[v] = e;
    reinterpret_cast<float4*>(score)[v] = sc;
    // touch counts of FREE entries are always zero (events on them are refused)
    if (t.x | t.y | t.z | t.w) {
      reinterpret_cast<uint4*>(touch)[v] = make_uint4(0, 0, 0, 0);
      if (t.x) last_epoch[4 * v + 0] = epoch;
      if (t.y) last_epoch[4 * v + 1] = epoch;
      if (t.z) last_epoch[4 * v + 2] = epoch;
      if (t.w) last_epoch[4 * v + 3] = epoch;
    }
  }
  // ragged tail (n not a multiple of 4)
  const uint64_t i = n4 * 4 + (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) {
    float e = ema[i];
    float sc;
    const uint32_t t = touch[i];
    entry_step(e, decay[i], t, pair[i], state[i], sP, policy, policy == 2 ? last_epoch[i] : 0u, epoch, sc);
    ema[i] = e;
    score[i] = sc;
    if (t) {
      touch[i] = 0;
      last_epoch[i] = epoch;
    }
  }
  // commit by the last block to finish
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    s_last = atomicAdd(pd.ticket, 1u) == gridDim.x - 1;
  }
  __syncthreads();
  if (s_last && threadIdx.x < 16) {
    const unsigned p = threadIdx.x;
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
      pd.blend->win[head * 32 + 2 * p] = pd.delta[2 * p];
      pd.blend->win[head * 32 + 2 * p + 1] = pd.delta[2 * p + 1];
      pd.blend->wsum[2 * p] = wm;
      pd.blend->wsum[2 * p + 1] = wh;
      if (p == 0) pd.blend->head = (head + 1) % pd.window;
    }
    pd.delta[2 * p] = 0;
    pd.delta[2 * p + 1] = 0;
    if (p == 0) *pd.ticket = 0;
  }
}

__global__ void blend_reset_kernel(BlendState* b) {
  for (uint32_t i = threadIdx.x; i < kMaxWindow * 32; i += blockDim.x) b->win[i] = 0;
  if (threadIdx.x < 32) b->wsum[threadIdx.x] = 0;
  if (threadIdx.x == 0) b->head = 0;
}

cudaError_t launch_blend_reset(const Workspace& ws, cudaStream_t s) {
  blend_reset_kernel<<<1, 256, 0, s>>>(ws.blend);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_entry_update(const EntryState& st, uint64_t* hits, uint64_t* misses, float* P,
                                float alpha0, float beta0, const Workspace& ws, uint32_t epoch,
                                const ScoreOptions& opt, cudaStream_t s) {
  uint64_t blocks = (st.n / 4 + kThreads - 1) / kThreads;
  if (blocks == 0) blocks = 1;
  const uint64_t cap = (uint64_t)kSMs * 8;
  if (blocks > cap) blocks = cap;
  const Predictor pd{hits,       misses,    P,          alpha0, beta0, ws.delta, &ws.sel->update_ticket,
                     opt.policy, opt.kappa, opt.window, ws.blend};
  entry_update_kernel<<<(unsigned)blocks, kThreads, 0, s>>>(st.ema, st.decay, st.touch, st.last_epoch,
                                                            st.pair, st.state, st.score, pd, st.n, epoch);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace kvt
