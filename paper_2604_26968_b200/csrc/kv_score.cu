// Scoring kernels: event reduction, and the fused posterior + EMA + score pass.
//
// The arithmetic itself lives in kv_score_device.cuh.
#include "kv_score_device.cuh"

namespace kvt {

// ---- event reduction ---------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
event_reduce_kernel(const uint32_t* __restrict__ ev_entry, const uint8_t* __restrict__ ev_hit,
                    uint64_t n_events, const uint8_t* __restrict__ pair,
                    uint32_t* __restrict__ touch, uint64_t n,
                    unsigned long long* __restrict__ delta, uint32_t* __restrict__ status) {
  __shared__ uint32_t s_cnt[16 * kThreads];   // [pair][thread]: events | hits << 16
  for (uint32_t i = threadIdx.x; i < 16 * kThreads; i += kThreads) s_cnt[i] = 0;
  __syncthreads();
  const uint32_t bad = reduce_events(ev_entry, ev_hit, n_events, pair, touch, n,
                                     (uint64_t)blockIdx.x * blockDim.x + threadIdx.x,
                                     (uint64_t)gridDim.x * blockDim.x, s_cnt, delta);
  if (bad) atomicOr(status, bad);
}

cudaError_t launch_event_reduce(const uint32_t* ev_entry, const uint8_t* ev_hit, uint64_t n_events,
                                const EntryState& st, const Workspace& ws, cudaStream_t s) {
  if (n_events == 0) return cudaSuccess;
  uint64_t blocks = (n_events / 4 + kThreads - 1) / kThreads;
  if (blocks == 0) blocks = 1;
  const uint64_t cap = (uint64_t)sm_count() * 4;  // measured: 4 blocks per SM beat 8 and 2
  if (blocks > cap) blocks = cap;
  const uint8_t* pair = st.pair;
  uint32_t* touch = st.touch;
  uint64_t n = st.n;
  unsigned long long* delta = ws.delta;
  uint32_t* status = ws.status;
  void* args[] = {&ev_entry, &ev_hit, &n_events, &pair, &touch, &n, &delta, &status};
  const cudaError_t e = launch_scoring_kernel((const void*)event_reduce_kernel, dim3((unsigned)blocks),
                                              dim3(kThreads), args, 0, s, false, ws);
  count_launches(1);
  return e != cudaSuccess ? e : cudaGetLastError();
}

// ---- entry pass ----------------------------------------------------------------------
// Every block forms the 16 posteriors itself (32 counters, read-only here), then
// streams its share of the entries: four per thread and iteration, every array
// read and written with 16-byte (for the byte arrays 4-byte) accesses.  The last
// block to finish folds the epoch's counts into the totals, clears them and
// publishes P; by then every block has read them.
__global__ void __launch_bounds__(kThreads, 4)
entry_update_kernel(const EntryState st, const Predictor pd, const HeadWeights hw, uint32_t epoch) {
  __shared__ float sP[16];
  __shared__ bool s_last;
  const int policy = pd.policy;
  if (threadIdx.x < 16) {
    unsigned long long h, m, wh, wm;
    const float P = posterior(pd, threadIdx.x, h, m);
    sP[threadIdx.x] = reuse_estimate(pd, threadIdx.x, P, h, m, wh, wm);
  }
  __syncthreads();
  const uint64_t n4 = st.n / 4;
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  uint64_t v = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  EntryVec cur;
  if (v < n4) cur = entry_load4(st, v, policy);
  for (; v < n4; v += stride) {   // the next vector's loads fly while this one is finished
    EntryVec nxt;
    if (v + stride < n4) nxt = entry_load4(st, v + stride, policy);
    float4 sc;
    entry_finish4(st, v, cur, sP, policy, epoch, hw, sc);
    cur = nxt;
  }
  // ragged tail (n not a multiple of 4)
  const uint64_t i = n4 * 4 + (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < st.n) {
    float sc;
    uint32_t s1;
    entry_update1(st, i, sP, policy, epoch, hw, sc, s1);
  }
  // commit by the last block to finish
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    s_last = atomicAdd(pd.ticket, 1u) == gridDim.x - 1;
  }
  __syncthreads();
  if (s_last && threadIdx.x < 16) {
    commit_predictor(pd, threadIdx.x);
    if (threadIdx.x == 0) *pd.ticket = 0;
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
                                const ScoreOptions& opt, const HeadWeights& hw, cudaStream_t s) {
  uint64_t blocks = (st.n / 4 + kThreads - 1) / kThreads;
  if (blocks == 0) blocks = 1;
  const uint64_t cap = (uint64_t)sm_count() * 8;
  if (blocks > cap) blocks = cap;
  const Predictor pd{hits,       misses,    P,          alpha0, beta0, ws.delta, &ws.sel->update_ticket,
                     opt.policy, opt.kappa, opt.window, ws.blend};
  EntryState st_arg = st;
  Predictor pd_arg = pd;
  HeadWeights hw_arg = hw;
  void* args[] = {&st_arg, &pd_arg, &hw_arg, &epoch};
  const cudaError_t e = launch_scoring_kernel((const void*)entry_update_kernel, dim3((unsigned)blocks),
                                              dim3(kThreads), args, 0, s, false, ws);
  count_launches(1);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace kvt
