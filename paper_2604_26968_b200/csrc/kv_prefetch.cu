// Per-layer prefetch window and the prefetch list of one sequence (RoPE-aware
// prefetching section).
//
// The section states that, with a sequence at position n, promotion requests go out for
// the blocks covering positions [n, n+w] (it also names [n-w, n] as the range likeliest
// to be read next), and that the window w adapts per layer to the observed attention
// pattern: narrow for local-attention layers, wide for global-attention layers.  It
// prints no formula; the form used here, per partition:
//   S[l] <- d*S[l] + (1-d)*x[l]     x[l]: attention span observed in layer l, tokens
//                                   (binary32, each operation rounded once)
//   w[l] = min(w_max, max(1, ceil(S[l] / block_tokens)))    blocks
// and the list of a sequence at position-block pos0 holds, ordered by (distance, layer,
// head), the ring slot of every block of the sequence's block table at distance < w[l]
// that sits in the host tier.
//
// The list is an ordered compaction of at most distance x layers x heads candidates.
// Two launches over the same chunks: the first counts the qualifying candidates of each
// chunk, the second sums the counts before its chunk and writes.  No block waits on
// another; the block table is read coalesced, d_loc by gather (both passes; the second
// finds it in L2).
#include "kvtier_internal.cuh"

namespace kvt {

namespace {

constexpr int kPfThreads = 256;

__device__ __forceinline__ bool span_ok(float v) {
  return v >= 0.0f && v <= 3.402823466e+38f;  // false for NaN, negatives and infinities
}

__device__ __forceinline__ uint32_t window_of(float span, float block_tokens, uint32_t w_max) {
  const float c = ceilf(__fdiv_rn(span, block_tokens));   // exact: the ceiling of a binary32 is one
  double w = (double)c;
  if (w < 1.0) w = 1.0;
  if (w > (double)w_max) w = (double)w_max;
  return (uint32_t)w;
}

// One block.  mode 0: EMA step with observations x; mode 1: every span = tokens.
// A bad observation anywhere leaves the whole partition as it was.
__global__ void prefetch_window_kernel(float* __restrict__ span, uint32_t* __restrict__ win,
                                       const float* __restrict__ x, float d, float tokens, int mode,
                                       uint32_t layers, float block_tokens, uint32_t w_max,
                                       uint32_t* __restrict__ status) {
  int bad = 0;
  if (mode == 0)
    for (uint32_t l = threadIdx.x; l < layers; l += blockDim.x) bad |= !span_ok(x[l]);
  if (__syncthreads_or(bad)) {
    if (threadIdx.x == 0) atomicOr(status, KV_DEV_BAD_SPAN_VALUE);
    return;
  }
  for (uint32_t l = threadIdx.x; l < layers; l += blockDim.x) {
    float s = tokens;
    if (mode == 0) {
      const float t1 = __fmul_rn(d, span[l]);
      const float t2 = __fsub_rn(1.0f, d);
      const float t3 = __fmul_rn(t2, x[l]);
      s = __fadd_rn(t1, t3);
    }
    span[l] = s;
    win[l] = window_of(s, block_tokens, w_max);
  }
}

struct ListArgs {
  const uint32_t* table;   // [n_pos][L][H] block handles
  const uint32_t* win;     // [L]
  const uint32_t* loc;     // [n_tags]
  unsigned long long* out;
  unsigned long long* count;
  uint32_t* chunk_counts;  // [gridDim.x]
  unsigned long long n_items;   // candidates the host can bound: distances x L x H
  unsigned long long chunk;     // candidates per block, a multiple of kPfThreads
  unsigned long long pos0, max_out, n_tags;
  uint32_t layers, heads;
  int dir;
};

// Ring slot of candidate i if it qualifies; candidates are numbered (distance, layer, head).
__device__ __forceinline__ bool candidate(const ListArgs& a, unsigned long long i, uint32_t row,
                                          uint32_t* slot) {
  const unsigned long long dist = i / row;
  const uint32_t r = (uint32_t)(i - dist * row);
  if (dist >= __ldg(a.win + r / a.heads)) return false;
  const unsigned long long pb = a.dir > 0 ? a.pos0 + dist : a.pos0 - dist;
  const uint32_t t = __ldg(a.table + pb * row + r);
  if (t >= a.n_tags) return false;
  const uint32_t where = __ldg(a.loc + t);
  if (where == KV_NONE || !(where & KV_LOC_HOST)) return false;
  *slot = where & ~KV_LOC_HOST;
  return true;
}

template <bool kWrite>
__global__ void __launch_bounds__(kPfThreads) prefetch_list_kernel(const ListArgs a) {
  __shared__ unsigned long long s_red[kPfThreads / 32];
  __shared__ uint32_t s_warp[kPfThreads / 32];
  __shared__ uint32_t s_wmax;
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t row = a.layers * a.heads;

  // the widest window bounds the distances any layer wants
  if (tid == 0) s_wmax = 0;
  __syncthreads();
  uint32_t wm = 0;
  for (uint32_t l = tid; l < a.layers; l += kPfThreads) wm = max(wm, __ldg(a.win + l));
  for (int o = 16; o > 0; o >>= 1) wm = max(wm, __shfl_xor_sync(0xFFFFFFFFu, wm, o));
  if (lane == 0 && wm) atomicMax(&s_wmax, wm);
  __syncthreads();
  const unsigned long long limit = min(a.n_items, (unsigned long long)s_wmax * row);
  const unsigned long long c0 = (unsigned long long)blockIdx.x * a.chunk;
  const unsigned long long c1 = min(c0 + a.chunk, limit);

  if (!kWrite) {
    uint32_t n = 0, slot;
    for (unsigned long long i = c0 + tid; i < c1; i += kPfThreads) n += candidate(a, i, row, &slot);
    for (int o = 16; o > 0; o >>= 1) n += __shfl_xor_sync(0xFFFFFFFFu, n, o);
    if (lane == 0) s_warp[warp] = n;
    __syncthreads();
    if (tid == 0) {
      uint32_t s = 0;
      for (int w = 0; w < kPfThreads / 32; ++w) s += s_warp[w];
      a.chunk_counts[blockIdx.x] = s;
    }
    return;
  }

  // candidates that qualify before this chunk (and, in block 0, in all chunks)
  unsigned long long before = 0, all = 0;
  for (uint32_t b = tid; b < gridDim.x; b += kPfThreads) {
    const uint32_t c = a.chunk_counts[b];
    all += c;
    if (b < blockIdx.x) before += c;
  }
  for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xFFFFFFFFu, before, o);
  if (lane == 0) s_red[warp] = before;
  __syncthreads();
  unsigned long long offset = 0;
  for (int w = 0; w < kPfThreads / 32; ++w) offset += s_red[w];
  if (blockIdx.x == 0) {
    __syncthreads();
    for (int o = 16; o > 0; o >>= 1) all += __shfl_xor_sync(0xFFFFFFFFu, all, o);
    if (lane == 0) s_red[warp] = all;
    __syncthreads();
    if (tid == 0) {
      unsigned long long s = 0;
      for (int w = 0; w < kPfThreads / 32; ++w) s += s_red[w];
      *a.count = s;
    }
  }

  for (unsigned long long base = c0; base < c1; base += kPfThreads) {   // block-uniform trip count
    const unsigned long long i = base + tid;
    uint32_t slot = 0;
    const bool q = i < c1 && candidate(a, i, row, &slot);
    const uint32_t m = __ballot_sync(0xFFFFFFFFu, q);
    __syncthreads();                       // s_warp of the tile before has been read
    if (lane == 0) s_warp[warp] = __popc(m);
    __syncthreads();
    uint32_t ahead = 0, total = 0;
    for (int w = 0; w < kPfThreads / 32; ++w) {
      const uint32_t c = s_warp[w];
      if (w < (int)warp) ahead += c;
      total += c;
    }
    if (q) {
      const unsigned long long at = offset + ahead + __popc(m & ((1u << lane) - 1u));
      if (at < a.max_out) a.out[at] = slot;
    }
    offset += total;
  }
}

}  // namespace

cudaError_t launch_prefetch_window(const PrefetchState& pf, int q, int mode, const float* x, float decay,
                                   float tokens, const Workspace& ws, cudaStream_t s) {
  prefetch_window_kernel<<<1, 128, 0, s>>>(pf.span + pf.off[q], pf.win + pf.off[q], x, decay, tokens, mode,
                                           pf.layers[q], (float)pf.block_tokens[q], pf.w_max[q], ws.status);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_prefetch_list(const PrefetchState& pf, int q, const uint32_t* table, uint64_t n_pos,
                                 uint64_t pos0, int dir, const uint32_t* loc, uint64_t n_tags,
                                 unsigned long long* out, uint64_t max_out, unsigned long long* count,
                                 cudaStream_t s) {
  ListArgs a;
  a.table = table;
  a.win = pf.win + pf.off[q];
  a.loc = loc;
  a.out = out;
  a.count = count;
  a.chunk_counts = pf.chunk_counts;
  a.layers = pf.layers[q];
  a.heads = pf.heads[q];
  a.dir = dir;
  a.pos0 = pos0;
  a.max_out = out ? max_out : 0;
  a.n_tags = n_tags;
  // distances inside the table on the chosen side, never more than the cap on the window
  uint64_t dists = n_pos == 0 ? 0 : (dir > 0 ? n_pos - pos0 : pos0 + 1);
  if (dists > pf.w_max[q]) dists = pf.w_max[q];
  a.n_items = dists * a.layers * a.heads;
  uint64_t chunk = (a.n_items + kPrefetchChunks - 1) / kPrefetchChunks;
  chunk = (chunk + kPfThreads - 1) / kPfThreads * kPfThreads;
  if (chunk < 4 * kPfThreads) chunk = 4 * kPfThreads;
  a.chunk = chunk;
  uint64_t blocks = (a.n_items + chunk - 1) / chunk;
  if (blocks == 0) blocks = 1;
  prefetch_list_kernel<false><<<(unsigned)blocks, kPfThreads, 0, s>>>(a);
  prefetch_list_kernel<true><<<(unsigned)blocks, kPfThreads, 0, s>>>(a);
  count_launches(2);
  return cudaGetLastError();
}

}  // namespace kvt
