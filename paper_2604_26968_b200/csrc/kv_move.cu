// Admission of fresh blocks (a harness step: pattern fill of every FREE slot) and
// initialisation of a pool's state.  The gather and scatter kernels of demotion
// and promotion are in kv_move_tma.cu.
#include "kvtier_internal.cuh"

namespace kvt {

constexpr uint32_t kPieceBytes = 2048;  // 32 lanes x 4 x 16 bytes

// Byte offset of chunk c of local entry `local` inside the partition slab.
__device__ __forceinline__ uint64_t chunk_offset(const PartGeom& g, uint64_t local, uint32_t c) {
  const uint64_t lb = local / g.heads;  // layer * blocks_per_layer + block
  const uint64_t head = local - lb * g.heads;
  return ((lb * g.n_chunks + c) * g.heads + head) * (uint64_t)g.chunk_bytes;
}

static unsigned move_grid(uint64_t total_pieces) {
  uint64_t blocks = (total_pieces * 32 + kThreads - 1) / kThreads;
  if (blocks == 0) blocks = 1;
  const uint64_t cap = (uint64_t)sm_count() * 8;
  return (unsigned)(blocks > cap ? cap : blocks);
}

static uint64_t pieces_per_entry(const PartGeom& g) {
  return (uint64_t)((g.chunk_bytes + kPieceBytes - 1) / kPieceBytes) * g.n_chunks;
}

// SplitMix64 output function (Steele, Lea, Flood: "Fast splittable pseudorandom
// number generators", 2014).
__device__ __forceinline__ unsigned long long splitmix64(unsigned long long x) {
  unsigned long long z = x + 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

__global__ void __launch_bounds__(kThreads)
admit_kernel(const PartGeom g, const EntryState st, uint32_t* __restrict__ loc,
             const uint32_t* __restrict__ free_ids, uint64_t first, uint64_t count, uint64_t first_tag,
             const uint8_t* __restrict__ new_pairs, uint32_t epoch, float decay, int fill_pattern,
             uint32_t* __restrict__ status) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t ppc = (g.chunk_bytes + kPieceBytes - 1) / kPieceBytes;
  const uint32_t ppe = fill_pattern ? ppc * g.n_chunks : 1u;
  const uint64_t total = count * ppe;
  const uint64_t warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
  for (uint64_t piece = (((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5); piece < total;
       piece += warps) {
    const uint64_t j = piece / ppe;
    const uint32_t r = (uint32_t)(piece - j * ppe);
    const uint32_t f = free_ids[first + j];
    if ((uint64_t)f < g.base || (uint64_t)f >= g.base + g.n) {
      if (lane == 0) atomicOr(status, KV_DEV_BAD_INDEX);
      continue;
    }
    const unsigned long long t = first_tag + first + j;
    if (fill_pattern) {
      const uint32_t c = r / ppc;
      const uint32_t pp = r - c * ppc;
      const uint32_t in_chunk = pp * kPieceBytes;
      const uint32_t len = min(kPieceBytes, g.chunk_bytes - in_chunk);
      uint8_t* dst = g.slab + chunk_offset(g, (uint64_t)f - g.base, c) + in_chunk;
      const uint32_t image_off = c * g.chunk_bytes + in_chunk;  // offset inside the entry image
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const uint32_t off = (u * 32 + lane) * 16;
        if (off < len) {
          const unsigned long long w = (image_off + off) >> 3;
          uint4 val;
          const unsigned long long a = splitmix64((t << 20) + w), b = splitmix64((t << 20) + w + 1);
          val.x = (uint32_t)a; val.y = (uint32_t)(a >> 32);
          val.z = (uint32_t)b; val.w = (uint32_t)(b >> 32);
          __stcs(reinterpret_cast<uint4*>(dst + off), val);
        }
      }
    }
    if (r == 0 && lane == 0) {
      if (st.state[f] != KV_STATE_FREE) {
        atomicOr(status, KV_DEV_BAD_INDEX);
        continue;
      }
      st.tag[f] = (uint32_t)t;
      st.pair[f] = new_pairs[first + j] & 15u;
      st.ema[f] = 0.0f;
      st.decay[f] = decay;
      st.last_epoch[f] = epoch;
      st.touch[f] = 0;
      st.state[f] = KV_STATE_RESIDENT;
      loc[t] = f;
    }
  }
}

cudaError_t launch_admit(const PartGeom& g, const EntryState& st, uint32_t* loc, const uint32_t* free_ids,
                         uint64_t first, uint64_t count, uint64_t first_tag, const uint8_t* new_pairs,
                         uint32_t epoch, float decay, int fill_pattern, const Workspace& ws,
                         cudaStream_t s) {
  if (count == 0) return cudaSuccess;
  const uint64_t pieces = count * (fill_pattern ? pieces_per_entry(g) : 1);
  admit_kernel<<<move_grid(pieces), kThreads, 0, s>>>(g, st, loc, free_ids, first, count, first_tag,
                                                      new_pairs, epoch, decay, fill_pattern, ws.status);
  count_launches(1);
  return cudaGetLastError();
}

// ---- initialisation ---------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
init_entries_kernel(const EntryState st, uint32_t* __restrict__ loc, uint64_t n_tags) {
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  const uint64_t g0 = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  for (uint64_t i = g0; i < st.n; i += stride) {
    st.ema[i] = 0.0f;
    st.decay[i] = 0.0f;
    st.touch[i] = 0;
    st.last_epoch[i] = 0;
    st.pair[i] = (uint8_t)kPairFree;
    st.state[i] = KV_STATE_FREE;
    st.tag[i] = KV_NONE;
    st.score[i] = __int_as_float(0x7F800000);
  }
  for (uint64_t t = g0; t < n_tags; t += stride) loc[t] = KV_NONE;
}

__global__ void __launch_bounds__(kThreads) init_ring_kernel(const PartGeom g) {
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t s = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; s < g.ring_slots; s += stride) {
    g.r_tag[s] = KV_NONE;
    g.r_last_epoch[s] = 0;
    g.r_depoch[s] = 0;
    g.r_ema[s] = 0.0f;
    g.r_decay[s] = 0.0f;
    g.r_pair[s] = 0;
  }
}

__global__ void init_scalars_kernel(uint64_t* hits, uint64_t* misses, float* P, float p0,
                                    const Workspace ws) {
  const uint32_t t = threadIdx.x;
  if (t < 16) { hits[t] = 0; misses[t] = 0; P[t] = p0; ws.blend->estimate[t] = p0; }
  if (t < 32) { ws.delta[t] = 0; ws.blend->wsum[t] = 0; }
  for (uint32_t i = t; i < kMaxWindow * 32; i += blockDim.x) ws.blend->win[i] = 0;
  if (t == 0) { ws.blend->head = 0; ws.blend->pad = 0; }
  for (uint32_t b = t; b < 3 * kHistBins; b += blockDim.x) ws.hist[b] = 0;
  if (t < 4) ws.part_counts[t] = 0;
  if (t == 0) {
    *ws.status = 0;
    ws.sel->prefix = 0; ws.sel->tau = 0; ws.sel->k_rem = 0; ws.sel->need_eq = 0;
    ws.sel->bar_arrive = 0; ws.sel->bar_done = 0; ws.sel->update_ticket = 0; ws.sel->hint_last = 0;
    ws.sel->hint_valid = 0; ws.sel->hint_tau = 0; ws.sel->hint_n = 0; ws.sel->below = 0;
    ws.sel->hint_shift = 11; ws.sel->hint_resid = 0;
    ws.sel->n_select = 0; ws.sel->n_hint_hit = 0; ws.sel->n_hint_miss = 0; ws.sel->n_reread = 0;
  }
}

cudaError_t launch_init(const EntryState& st, uint64_t* hits, uint64_t* misses, float* P, float p0,
                        uint32_t* loc, uint64_t n_tags, const PartGeom* parts, int n_parts,
                        const Workspace& ws, cudaStream_t s) {
  const uint64_t most = st.n > n_tags ? st.n : n_tags;
  uint64_t blocks = (most + kThreads - 1) / kThreads;
  const uint64_t cap = (uint64_t)sm_count() * 8;
  if (blocks > cap) blocks = cap;
  if (blocks == 0) blocks = 1;
  init_entries_kernel<<<(unsigned)blocks, kThreads, 0, s>>>(st, loc, n_tags);
  for (int q = 0; q < n_parts; ++q) {
    if (parts[q].ring_slots == 0) continue;
    uint64_t rb = ((uint64_t)parts[q].ring_slots + kThreads - 1) / kThreads;
    if (rb > cap) rb = cap;
    init_ring_kernel<<<(unsigned)rb, kThreads, 0, s>>>(parts[q]);
    count_launches(1);
  }
  init_scalars_kernel<<<1, 256, 0, s>>>(hits, misses, P, p0, ws);
  count_launches(2);
  return cudaGetLastError();
}

}  // namespace kvt
