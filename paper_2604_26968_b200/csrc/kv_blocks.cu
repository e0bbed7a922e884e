// Block-granular selection: the aggregate importance of a paged block over its
// KV heads, and the expansion of selected blocks into their entries.
//
// The head-granular eviction section evicts "the block with the lowest weighted
// aggregate importance score across heads" with architecture-dependent head
// weights (uniform for MHA, proportional to group size for GQA).  The aggregate
// used here is w * (s_0 + ... + s_{H-1}) over the block's KV-head entries, summed
// in head order with every binary32 operation rounded once, w = query heads per
// KV-head entry; a block is a candidate only while all its heads are RESIDENT.
// Selection itself is the same radix select as for entries, run on the
// per-block arrays.
#include "kvtier_internal.cuh"

namespace kvt {

__device__ __forceinline__ int block_partition(const BlockGeom& bg, uint64_t gb) {
  int q = 0;
  while (q + 1 < bg.n_parts && gb >= bg.block_base[q + 1]) ++q;
  return q;
}

__global__ void __launch_bounds__(kThreads)
block_aggregate_kernel(const float* __restrict__ score, const uint8_t* __restrict__ state,
                       const BlockGeom bg, float* __restrict__ bscore, uint8_t* __restrict__ bstate) {
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  const uint64_t n_blocks = bg.block_base[bg.n_parts];
  for (uint64_t gb = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; gb < n_blocks; gb += stride) {
    const int q = block_partition(bg, gb);
    const uint32_t H = bg.heads[q];
    const uint64_t first = bg.entry_base[q] + (gb - bg.block_base[q]) * H;
    bool all = true;
    float sum = 0.0f;
    for (uint32_t h = 0; h < H; ++h) {
      all = all && state[first + h] == KV_STATE_RESIDENT;
      sum = __fadd_rn(sum, score[first + h]);
    }
    bscore[gb] = all ? __fmul_rn(bg.weight[q], sum) : __int_as_float(0x7F800000);
    bstate[gb] = all ? (uint8_t)KV_STATE_RESIDENT : (uint8_t)KV_STATE_FREE;
  }
}

// victims[off ..] = the H entries of the j-th selected block, where off counts the
// entries of all selected blocks before it (blocks are ascending, partitions are
// contiguous, so off follows from the per-partition block counts).
__global__ void __launch_bounds__(kThreads)
block_expand_kernel(const uint32_t* __restrict__ block_victims, uint64_t k_blocks, const BlockGeom bg,
                    const unsigned long long* __restrict__ part_counts, uint32_t* __restrict__ victims,
                    unsigned long long* __restrict__ h_entry_counts) {
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  if (h_entry_counts && blockIdx.x == 0 && threadIdx.x < 4)   // what kv_demote will want to know
    h_entry_counts[threadIdx.x] = (int)threadIdx.x < bg.n_parts
                                      ? (bg.n_parts == 1 ? k_blocks : part_counts[threadIdx.x]) * bg.heads[threadIdx.x]
                                      : 0ull;
  for (uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; j < k_blocks; j += stride) {
    const uint64_t gb = block_victims[j];
    const int q = block_partition(bg, gb);
    uint64_t start = 0, off = 0;  // selected blocks / entries in the partitions before q
    for (int r = 0; r < q; ++r) {
      start += part_counts[r];
      off += part_counts[r] * bg.heads[r];
    }
    const uint32_t H = bg.heads[q];
    off += (j - start) * H;
    const uint64_t first = bg.entry_base[q] + (gb - bg.block_base[q]) * H;
    for (uint32_t h = 0; h < H; ++h) victims[off + h] = (uint32_t)(first + h);
  }
}

static unsigned grid_for(uint64_t n) {
  uint64_t blocks = (n + kThreads - 1) / kThreads;
  const uint64_t cap = (uint64_t)sm_count() * 8;
  if (blocks > cap) blocks = cap;
  return (unsigned)(blocks ? blocks : 1);
}

cudaError_t launch_select_blocks(const EntryState& st, const BlockGeom& bg, uint64_t k_blocks,
                                 uint32_t* d_victims, const Workspace& ws, cudaStream_t s,
                                 unsigned long long* h_entry_counts) {
  const uint64_t n_blocks = bg.block_base[bg.n_parts];
  block_aggregate_kernel<<<grid_for(n_blocks), kThreads, 0, s>>>(st.score, st.state, bg, ws.block_score,
                                                                 ws.block_state);
  count_launches(1);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  EntryState bs{};
  bs.score = ws.block_score;
  bs.state = ws.block_state;
  bs.n = n_blocks;
  PartCounts pc;   // the selected blocks per partition, a by-product of the selection
  for (int q = 0; q <= 4; ++q) pc.base[q] = bg.block_base[q < bg.n_parts ? q : bg.n_parts];
  pc.n_parts = bg.n_parts;
  pc.d_counts = ws.part_counts;
  e = launch_select(bs, k_blocks, ws.block_victims, ws, s, 1, &pc);
  if (e != cudaSuccess) return e;
  block_expand_kernel<<<grid_for(k_blocks), kThreads, 0, s>>>(ws.block_victims, k_blocks, bg, ws.part_counts,
                                                              d_victims, h_entry_counts);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace kvt
