// Selection of the k lowest (score, id) entries without sorting, and the
// ordered compaction it shares with free-slot listing.
//
// The eviction rule of the head-granular eviction section takes the lowest
// score; ties go to the lowest (partition, layer, block, head), i.e. the lowest
// global id.  Scores are mapped to 32-bit keys whose unsigned order equals the
// float order; a three-digit radix select (11 + 11 + 10 bits) finds the key tau
// of the k-th smallest entry; an ordered compaction then emits, in ascending id
// order, every entry with key < tau plus the first k - #{key < tau} entries with
// key == tau.  Nothing waits on another block: each phase is its own launch.
#include <mutex>

#include "kvtier_internal.cuh"

namespace kvt {

__device__ __forceinline__ uint32_t score_key(float s) {
  uint32_t b = __float_as_uint(s);
  if (b == 0x80000000u) b = 0u;  // -0.0 orders with +0.0
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

template <int PASS> struct Digit;
template <> struct Digit<0> { static constexpr uint32_t shift = 21, bits = 11, fixed_mask = 0u; };
template <> struct Digit<1> { static constexpr uint32_t shift = 10, bits = 11, fixed_mask = 0xFFE00000u; };
template <> struct Digit<2> { static constexpr uint32_t shift = 0, bits = 10, fixed_mask = 0xFFFFFC00u; };

// Adds one to s_hist[bin] for every active lane.  When all active lanes of the
// warp agree on the bin (the common case when most scores are equal, e.g. a
// freshly admitted pool where every score is +0) a single atomic is issued.
__device__ __forceinline__ void warp_hist_add(uint32_t* s_hist, bool active, uint32_t bin) {
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

template <int PASS>
__global__ void __launch_bounds__(kThreads)
select_hist_kernel(const float* __restrict__ score, const uint8_t* __restrict__ state, uint64_t n,
                   const SelectScalars* __restrict__ sel, uint32_t* __restrict__ hist) {
  using D = Digit<PASS>;
  constexpr uint32_t nbins = 1u << D::bits;
  __shared__ uint32_t s_hist[nbins];
  for (uint32_t b = threadIdx.x; b < nbins; b += blockDim.x) s_hist[b] = 0;
  __syncthreads();
  const uint32_t prefix = (PASS == 0) ? 0u : sel->prefix;
  const uint64_t n4 = n / 4;
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  const uint64_t gtid = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const uint64_t iters = (n4 + stride - 1) / stride;  // uniform: the warp votes need all lanes
  for (uint64_t it = 0; it < iters; ++it) {
    const uint64_t v = it * stride + gtid;
    const bool in = v < n4;
    float4 sc = make_float4(0.f, 0.f, 0.f, 0.f);
    uchar4 st = make_uchar4(0, 0, 0, 0);
    if (in) {
      sc = reinterpret_cast<const float4*>(score)[v];
      st = reinterpret_cast<const uchar4*>(state)[v];
    }
    const float s4[4] = {sc.x, sc.y, sc.z, sc.w};
    const uint8_t t4[4] = {st.x, st.y, st.z, st.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t key = score_key(s4[j]);
      const bool act = in && t4[j] == KV_STATE_RESIDENT && (key & D::fixed_mask) == prefix;
      warp_hist_add(s_hist, act, (key >> D::shift) & (nbins - 1u));
    }
  }
  // ragged tail
  {
    const uint64_t i = n4 * 4 + gtid;
    bool act = false;
    uint32_t key = 0;
    if (i < n) {
      key = score_key(score[i]);
      act = state[i] == KV_STATE_RESIDENT && (key & D::fixed_mask) == prefix;
    }
    if (gtid < 32) warp_hist_add(s_hist, act, (key >> D::shift) & (nbins - 1u));
  }
  __syncthreads();
  for (uint32_t b = threadIdx.x; b < nbins; b += blockDim.x) {
    const uint32_t c = s_hist[b];
    if (c) atomicAdd(&hist[b], c);
  }
}

// Finds the bin in which the cumulative count reaches k_rem, fixes that digit,
// and clears the histogram for the next call.  One block of 1024 threads, two
// bins per thread.
template <int PASS>
__global__ void __launch_bounds__(1024) select_pick_kernel(SelectScalars* __restrict__ sel,
                                                           uint32_t* __restrict__ hist) {
  using D = Digit<PASS>;
  constexpr uint32_t nbins = 1u << D::bits;
  __shared__ uint32_t s_warp[32];
  const uint32_t t = threadIdx.x;
  const uint32_t b0 = 2 * t, b1 = 2 * t + 1;
  const uint32_t c0 = b0 < nbins ? hist[b0] : 0u;
  const uint32_t c1 = b1 < nbins ? hist[b1] : 0u;
  if (b0 < nbins) hist[b0] = 0;
  if (b1 < nbins) hist[b1] = 0;
  uint32_t incl = c0 + c1;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if ((t & 31u) >= (uint32_t)o) incl += y;
  }
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
  const uint32_t before = incl - (c0 + c1) + ((t >> 5) ? s_warp[(t >> 5) - 1] : 0u);
  const unsigned long long k_rem = sel->k_rem;
  __syncthreads();  // everyone has read k_rem before one thread rewrites it
  // bin b holds ranks (before_b, before_b + c_b]; exactly one bin contains k_rem (k_rem >= 1)
  if (c0 && (unsigned long long)before < k_rem && k_rem <= (unsigned long long)before + c0) {
    const uint32_t prefix = (PASS == 0 ? 0u : sel->prefix) | (b0 << D::shift);
    sel->prefix = prefix;
    sel->k_rem = k_rem - before;
    if (PASS == 2) { sel->tau = prefix; sel->need_eq = k_rem - before; }
  }
  const uint32_t before1 = before + c0;
  if (c1 && (unsigned long long)before1 < k_rem && k_rem <= (unsigned long long)before1 + c1) {
    const uint32_t prefix = (PASS == 0 ? 0u : sel->prefix) | (b1 << D::shift);
    sel->prefix = prefix;
    sel->k_rem = k_rem - before1;
    if (PASS == 2) { sel->tau = prefix; sel->need_eq = k_rem - before1; }
  }
}

// ---- ordered compaction ---------------------------------------------------------
// Category of an entry: 0 = not taken, 1 = taken, 2 = taken while the running
// count of category-2 entries (in id order) is below need_eq.
struct SelectPred {
  const float* score;
  const uint8_t* state;
  uint32_t tau;
  __device__ __forceinline__ uint32_t cat(float s, uint8_t st) const {
    if (st != KV_STATE_RESIDENT) return 0u;
    const uint32_t key = score_key(s);
    return key < tau ? 1u : (key == tau ? 2u : 0u);
  }
};

// Loads the categories of the 8 consecutive entries starting at i0 (i0 is a
// multiple of 8).  MODE 0: selection by score; MODE 1: FREE entries in [lo, hi).
template <int MODE>
__device__ __forceinline__ void load_cats(const float* __restrict__ score,
                                          const uint8_t* __restrict__ state, uint64_t n, uint64_t lo,
                                          uint64_t hi, uint32_t tau, uint64_t i0, uint32_t cat[8]) {
  uint8_t st[8];
  float sc[8];
  if (i0 + 8 <= n) {
    const uchar4 a = reinterpret_cast<const uchar4*>(state + i0)[0];
    const uchar4 b = reinterpret_cast<const uchar4*>(state + i0)[1];
    st[0] = a.x; st[1] = a.y; st[2] = a.z; st[3] = a.w;
    st[4] = b.x; st[5] = b.y; st[6] = b.z; st[7] = b.w;
    if (MODE == 0) {
      const float4 u = reinterpret_cast<const float4*>(score + i0)[0];
      const float4 w = reinterpret_cast<const float4*>(score + i0)[1];
      sc[0] = u.x; sc[1] = u.y; sc[2] = u.z; sc[3] = u.w;
      sc[4] = w.x; sc[5] = w.y; sc[6] = w.z; sc[7] = w.w;
    }
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const bool in = i0 + j < n;
      st[j] = in ? state[i0 + j] : (uint8_t)0xFF;
      if (MODE == 0) sc[j] = in ? score[i0 + j] : 0.f;
    }
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    if (MODE == 0) {
      SelectPred p{score, state, tau};
      cat[j] = p.cat(sc[j], st[j]);
    } else {
      const uint64_t i = i0 + j;
      cat[j] = (i >= lo && i < hi && st[j] == KV_STATE_FREE) ? 1u : 0u;
    }
  }
}

// Block-wide exclusive scan of a packed (cat1 count | cat2 count << 16) value;
// also returns the block total.  Counts per block are at most 2048 each.
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* s_warp, uint32_t& total) {
  const uint32_t t = threadIdx.x;
  uint32_t incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if ((t & 31u) >= (uint32_t)o) incl += y;
  }
  if ((t & 31u) == 31u) s_warp[t >> 5] = incl;
  __syncthreads();
  if (t < 32) {
    uint32_t w = t < (kThreads / 32) ? s_warp[t] : 0u;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, w, o);
      if (t >= (uint32_t)o) w += y;
    }
    s_warp[t] = w;
  }
  __syncthreads();
  total = s_warp[kThreads / 32 - 1];
  return incl - v + ((t >> 5) ? s_warp[(t >> 5) - 1] : 0u);
}

template <int MODE>
__global__ void __launch_bounds__(kThreads)
tile_count_kernel(const float* __restrict__ score, const uint8_t* __restrict__ state, uint64_t n,
                  uint64_t lo, uint64_t hi, uint64_t tile0, const SelectScalars* __restrict__ sel,
                  uint2* __restrict__ tile_counts) {
  __shared__ uint32_t s_warp[32];
  const uint32_t tau = (MODE == 0) ? sel->tau : 0u;
  const uint64_t i0 = (tile0 + blockIdx.x) * (uint64_t)kTileEntries + (uint64_t)threadIdx.x * 8;
  uint32_t cat[8];
  load_cats<MODE>(score, state, n, lo, hi, tau, i0, cat);
  uint32_t v = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) v += (cat[j] == 1u) + ((cat[j] == 2u) << 16);
  uint32_t total;
  (void)block_excl_scan(v, s_warp, total);
  if (threadIdx.x == 0) tile_counts[blockIdx.x] = make_uint2(total & 0xFFFFu, total >> 16);
}

// Exclusive prefix over the tile counts (one block, running carry).
__global__ void __launch_bounds__(1024)
tile_scan_kernel(const uint2* __restrict__ tile_counts, uint2* __restrict__ tile_offsets,
                 uint32_t n_tiles) {
  __shared__ uint32_t s_a[32], s_b[32];
  uint32_t carry_a = 0, carry_b = 0;
  const uint32_t t = threadIdx.x;
  for (uint32_t base = 0; base < n_tiles; base += 1024) {
    const uint32_t i = base + t;
    uint2 c = i < n_tiles ? tile_counts[i] : make_uint2(0, 0);
    uint32_t a = c.x, b = c.y;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t ya = __shfl_up_sync(0xFFFFFFFFu, a, o);
      const uint32_t yb = __shfl_up_sync(0xFFFFFFFFu, b, o);
      if ((t & 31u) >= (uint32_t)o) { a += ya; b += yb; }
    }
    if ((t & 31u) == 31u) { s_a[t >> 5] = a; s_b[t >> 5] = b; }
    __syncthreads();
    if (t < 32) {
      uint32_t wa = s_a[t], wb = s_b[t];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t ya = __shfl_up_sync(0xFFFFFFFFu, wa, o);
        const uint32_t yb = __shfl_up_sync(0xFFFFFFFFu, wb, o);
        if (t >= (uint32_t)o) { wa += ya; wb += yb; }
      }
      s_a[t] = wa; s_b[t] = wb;
    }
    __syncthreads();
    const uint32_t wa = (t >> 5) ? s_a[(t >> 5) - 1] : 0u;
    const uint32_t wb = (t >> 5) ? s_b[(t >> 5) - 1] : 0u;
    if (i < n_tiles) tile_offsets[i] = make_uint2(carry_a + wa + a - c.x, carry_b + wb + b - c.y);
    carry_a += s_a[31];
    carry_b += s_b[31];
    __syncthreads();
  }
}

template <int MODE>
__global__ void __launch_bounds__(kThreads)
tile_write_kernel(const float* __restrict__ score, const uint8_t* __restrict__ state, uint64_t n,
                  uint64_t lo, uint64_t hi, uint64_t tile0, const SelectScalars* __restrict__ sel,
                  const uint2* __restrict__ tile_offsets, uint64_t limit, uint32_t* __restrict__ out) {
  __shared__ uint32_t s_warp[32];
  const uint32_t tau = (MODE == 0) ? sel->tau : 0u;
  const unsigned long long need_eq = (MODE == 0) ? sel->need_eq : 0ull;
  const uint64_t i0 = (tile0 + blockIdx.x) * (uint64_t)kTileEntries + (uint64_t)threadIdx.x * 8;
  uint32_t cat[8];
  load_cats<MODE>(score, state, n, lo, hi, tau, i0, cat);
  uint32_t v = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) v += (cat[j] == 1u) + ((cat[j] == 2u) << 16);
  uint32_t total;
  const uint32_t excl = block_excl_scan(v, s_warp, total);
  if (v == 0) return;
  const uint2 off = tile_offsets[blockIdx.x];
  unsigned long long n1 = (unsigned long long)off.x + (excl & 0xFFFFu);  // category-1 entries before
  unsigned long long n2 = (unsigned long long)off.y + (excl >> 16);      // category-2 entries before
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    if (cat[j] == 1u) {
      const unsigned long long pos = n1 + (n2 < need_eq ? n2 : need_eq);
      if (pos < limit) out[pos] = (uint32_t)(i0 + j);
      ++n1;
    } else if (cat[j] == 2u) {
      if (n2 < need_eq) {
        const unsigned long long pos = n1 + n2;
        if (pos < limit) out[pos] = (uint32_t)(i0 + j);
      }
      ++n2;
    }
  }
}

// Checks that selection produced exactly k ids (a cheap guard against a broken
// histogram): total = #less + min(#equal, need_eq) over all tiles.
__global__ void select_check_kernel(const uint2* __restrict__ tile_counts,
                                    const uint2* __restrict__ tile_offsets, uint32_t n_tiles,
                                    const SelectScalars* __restrict__ sel, unsigned long long k,
                                    uint32_t* __restrict__ status) {
  const uint2 c = tile_counts[n_tiles - 1], o = tile_offsets[n_tiles - 1];
  const unsigned long long less = (unsigned long long)c.x + o.x, eq = (unsigned long long)c.y + o.y;
  const unsigned long long got = less + (eq < sel->need_eq ? eq : sel->need_eq);
  if (got != k) atomicOr(status, KV_DEV_SELECT_MISMATCH);
}

__global__ void select_begin_kernel(SelectScalars* sel, unsigned long long k) {
  sel->prefix = 0;
  sel->tau = 0;
  sel->k_rem = k;
  sel->need_eq = 0;
}

static unsigned hist_grid(uint64_t n) {
  uint64_t blocks = (n / 4 + kThreads - 1) / kThreads;
  if (blocks == 0) blocks = 1;
  const uint64_t cap = (uint64_t)sm_count() * 8;
  return (unsigned)(blocks > cap ? cap : blocks);
}

cudaError_t launch_select(const EntryState& st, uint64_t k, uint32_t* d_victims, const Workspace& ws,
                          cudaStream_t s, int variant, const PartCounts* pc) {
  if (k == 0 || st.n == 0) return cudaSuccess;
  if (variant == 1) {
    bool used = false;
    const cudaError_t e = launch_select_persistent(st, k, d_victims, ws, s, &used, nullptr, pc);
    if (e != cudaSuccess || used) return e;
  }
  const unsigned g = hist_grid(st.n);
  select_begin_kernel<<<1, 1, 0, s>>>(ws.sel, k);
  select_hist_kernel<0><<<g, kThreads, 0, s>>>(st.score, st.state, st.n, ws.sel, ws.hist);
  select_pick_kernel<0><<<1, 1024, 0, s>>>(ws.sel, ws.hist);
  select_hist_kernel<1><<<g, kThreads, 0, s>>>(st.score, st.state, st.n, ws.sel, ws.hist + kHistBins);
  select_pick_kernel<1><<<1, 1024, 0, s>>>(ws.sel, ws.hist + kHistBins);
  select_hist_kernel<2><<<g, kThreads, 0, s>>>(st.score, st.state, st.n, ws.sel, ws.hist + 2 * kHistBins);
  select_pick_kernel<2><<<1, 1024, 0, s>>>(ws.sel, ws.hist + 2 * kHistBins);
  const uint32_t n_tiles = (uint32_t)((st.n + kTileEntries - 1) / kTileEntries);
  tile_count_kernel<0><<<n_tiles, kThreads, 0, s>>>(st.score, st.state, st.n, 0, st.n, 0, ws.sel,
                                                    ws.tile_counts);
  tile_scan_kernel<<<1, 1024, 0, s>>>(ws.tile_counts, ws.tile_offsets, n_tiles);
  tile_write_kernel<0><<<n_tiles, kThreads, 0, s>>>(st.score, st.state, st.n, 0, st.n, 0, ws.sel,
                                                    ws.tile_offsets, k, d_victims);
  select_check_kernel<<<1, 1, 0, s>>>(ws.tile_counts, ws.tile_offsets, n_tiles, ws.sel, k, ws.status);
  count_launches(11);
  if (pc && pc->n_parts > 1) return launch_partition_counts(d_victims, k, *pc, s);
  return cudaGetLastError();
}

cudaError_t launch_free_list(const EntryState& st, uint64_t lo, uint64_t hi, uint64_t limit,
                             const Workspace& ws, cudaStream_t s, uint64_t out_offset) {
  if (hi <= lo || limit == 0) return cudaSuccess;
  const uint64_t tile0 = lo / kTileEntries;
  const uint32_t n_tiles = (uint32_t)((hi + kTileEntries - 1) / kTileEntries - tile0);
  tile_count_kernel<1><<<n_tiles, kThreads, 0, s>>>(st.score, st.state, st.n, lo, hi, tile0, ws.sel,
                                                    ws.tile_counts);
  tile_scan_kernel<<<1, 1024, 0, s>>>(ws.tile_counts, ws.tile_offsets, n_tiles);
  tile_write_kernel<1><<<n_tiles, kThreads, 0, s>>>(st.score, st.state, st.n, lo, hi, tile0, ws.sel,
                                                    ws.tile_offsets, limit, ws.free_list + out_offset);
  count_launches(3);
  return cudaGetLastError();
}

// counts[q] = number of victims with base[q] <= id < base[q+1]; victims ascending.
__global__ void partition_counts_kernel(const uint32_t* __restrict__ victims, unsigned long long m,
                                        const PartCounts pc) {
  __shared__ unsigned long long s_lb[5];
  const int q = threadIdx.x;
  if (q <= pc.n_parts) {
    unsigned long long lo = 0, hi = m;  // first index with victims[idx] >= base[q]
    while (lo < hi) {
      const unsigned long long mid = (lo + hi) >> 1;
      if ((unsigned long long)victims[mid] < pc.base[q]) lo = mid + 1; else hi = mid;
    }
    s_lb[q] = lo;
  }
  __syncthreads();
  if (q < 4) {
    const unsigned long long c = (q < pc.n_parts) ? s_lb[q + 1] - s_lb[q] : 0ull;
    pc.d_counts[q] = c;
    if (pc.h_counts) pc.h_counts[q] = c;
  }
}

cudaError_t launch_partition_counts(const uint32_t* d_victims, uint64_t m, const PartCounts& pc,
                                    cudaStream_t s) {
  partition_counts_kernel<<<1, 32, 0, s>>>(d_victims, m, pc);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace kvt

// ---- selection without any caller-provided or allocated scratch -------------------
// Some callers of this library must not allocate: a serving engine that has
// already handed every byte of device memory to its own pools, or code running
// where cudaMalloc is forbidden (inside a latency-critical loop, or under an
// allocator that owns the whole device).  For them the scratch that selection
// needs -- three digit histograms, a handful of scalars and the per-tile counts
// of the compaction -- lives in this fixed array, which every GPU that loads the
// library holds until the process exits.  Its size bounds the problem:
// kStaticMaxEntries entries.
namespace {

constexpr uint64_t kStaticMaxEntries = 1ull << 22;  // 4,194,304 entries
constexpr uint64_t kStaticMaxTiles = kStaticMaxEntries / kvt::kTileEntries + 2;
// layout (bytes): [0, 24576) histograms | [24576, 24832) scalars | [24832, 25088) status |
//                 [25088, +tiles*8) tile counts | then tile offsets
constexpr uint64_t kOffHist = 0;
constexpr uint64_t kOffSel = 3 * kvt::kHistBins * 4;
constexpr uint64_t kOffStatus = kOffSel + 256;
static_assert(sizeof(kvt::SelectScalars) <= 256, "the scalars have 256 bytes of the built-in scratch");
constexpr uint64_t kOffTileCounts = kOffStatus + 256;
constexpr uint64_t kOffTileOffsets = kOffTileCounts + ((kStaticMaxTiles * 8 + 255) / 256) * 256;
constexpr uint64_t kStaticScratchBytes = kOffTileOffsets + ((kStaticMaxTiles * 8 + 255) / 256) * 256;

static __device__ __align__(256) unsigned char g_select_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
unsigned char* g_scratch_addr[kMaxDevices] = {nullptr};

// The array's name is only a stand-in on the host; the address a kernel can use
// comes from the runtime, once per device, with that device current.
cudaError_t static_scratch(unsigned char** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_select_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_addr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" int32_t kv_select_victims_static(const float* d_score, const uint8_t* d_state, uint64_t n,
                                            uint64_t k, uint32_t* d_victims, uint32_t* d_status,
                                            kv_stream_t stream) {
  if (n == 0 || n > kStaticMaxEntries) return KV_ERR_INVALID_ARG;  // beyond the built-in scratch
  if (k > n) return KV_ERR_K_TOO_LARGE;
  if (!d_score || !d_state || (reinterpret_cast<uintptr_t>(d_score) & 15u) ||
      (reinterpret_cast<uintptr_t>(d_state) & 15u))
    return KV_ERR_INVALID_ARG;
  if (k == 0) return KV_OK;
  if (!d_victims || (reinterpret_cast<uintptr_t>(d_victims) & 15u)) return KV_ERR_INVALID_ARG;
  unsigned char* base = nullptr;
  if (static_scratch(&base) != cudaSuccess) return KV_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // The array keeps whatever the previous call left: start the histograms and the
  // status word from zero (the scalars are reset by the first kernel of the pass).
  if (cudaMemsetAsync(base + kOffHist, 0, kOffTileCounts, s) != cudaSuccess) return KV_ERR_CUDA;
  kvt::Workspace ws{};
  ws.hist = reinterpret_cast<uint32_t*>(base + kOffHist);
  ws.sel = reinterpret_cast<kvt::SelectScalars*>(base + kOffSel);
  ws.status = d_status ? d_status : reinterpret_cast<uint32_t*>(base + kOffStatus);
  ws.tile_counts = reinterpret_cast<uint2*>(base + kOffTileCounts);
  ws.tile_offsets = reinterpret_cast<uint2*>(base + kOffTileOffsets);
  ws.n_tiles = (uint32_t)kStaticMaxTiles;
  kvt::EntryState st{};
  st.score = const_cast<float*>(d_score);   // selection only reads score and state
  st.state = const_cast<uint8_t*>(d_state);
  st.n = n;
  if (kvt::launch_select(st, k, d_victims, ws, s) != cudaSuccess) return KV_ERR_CUDA;
  return KV_OK;
}
