// Gather (demotion) and scatter (promotion) of head-granular KV entries with the
// bulk asynchronous copy engine of the SM (cp.async.bulk, the 1-D form of TMA).
//
// A victim's K and V chunks (or its single MLA chunk) are contiguous runs of
// 2-72 KB at block-table-dependent addresses.  One elected lane per CTA streams
// them global -> shared -> global through a ring of shared-memory stages: a
// bulk load completes on the stage's mbarrier, the same lane then issues the
// bulk store out of the stage, and the stage is refilled once the store has
// finished reading it.  The bytes never pass through registers, a single lane
// keeps (stages - 1) x 4 KB in flight, and four such CTAs per SM keep ~176 KB
// per SM in flight, which is what a gather of scattered 4 KB pieces needs to
// approach streaming HBM bandwidth.  A second warp of each CTA moves the
// per-entry metadata (block table, ring-slot mirror, slot state).
//
// Every wait is bounded: a lane that gives up sets KV_DEV_WAIT_EXPIRED in the
// device status word, drains its own stores and leaves.
#include "kvtier_internal.cuh"

namespace kvt {

constexpr uint32_t kStageBytes = 4096;
constexpr uint32_t kStages = 12;               // 48 KB of shared memory per CTA
constexpr uint32_t kMoveThreads = 64;          // warp 0: copy lane; warp 1: metadata
constexpr uint32_t kMoveCtasPerSm = 4;
constexpr uint32_t kMetaBytes = 24;            // sizeof(kv_slot_meta)
constexpr uint32_t kWaitLimit = 1u << 24;      // mbarrier polls before giving up (seconds)

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}

// Polls the barrier's phase with the given parity; false if the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  const uint32_t addr = smem_u32(bar);
  for (uint32_t it = 0; it < kWaitLimit; ++it) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(addr), "r"(parity)
        : "memory");
    if (done) return true;
  }
  return false;
}

__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, uint32_t bytes,
                                          uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(smem_dst)),
      "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}

__device__ __forceinline__ void bulk_store(void* gmem_dst, const void* smem_src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gmem_dst),
               "r"(smem_u32(smem_src)), "r"(bytes)
               : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

__device__ __forceinline__ void bulk_wait_read_1() {
  asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
}
__device__ __forceinline__ void bulk_wait_all() {
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void fence_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// Byte offset of chunk c of local entry `local` inside the partition slab.
__device__ __forceinline__ uint64_t slab_chunk_offset(const PartGeom& g, uint64_t local, uint32_t c) {
  const uint64_t lb = local / g.heads;  // layer * blocks_per_layer + block
  const uint64_t head = local - lb * g.heads;
  return ((lb * g.n_chunks + c) * g.heads + head) * (uint64_t)g.chunk_bytes;
}

// A demotion can run its metadata for all victims first and move the payload
// chunk by chunk later (so that a promotion can already take the freed slots
// that have been packed).
constexpr uint32_t kMoveAll = 0, kMoveMetaOnly = 1, kMoveCopyOnly = 2;

struct MoveArgs {
  PartGeom g;
  EntryState st;
  uint32_t* loc;
  const uint32_t* ids;     // pack: victim ids; unpack: destination (free) ids
  const uint32_t* slots;   // unpack: ring slot of each entry (pack: unused)
  uint64_t count;
  uint64_t ring_start;     // pack: ring slot of entry 0
  uint8_t* staging;
  uint64_t meta_offset;    // pack: where the kv_slot_meta records go (~0 = none)
  uint32_t* status;
  uint32_t mode;           // pack only: kMoveAll, kMoveMetaOnly or kMoveCopyOnly
};

// Metadata of one demoted entry (ring slot mirror, block table, slot state).
__device__ __forceinline__ void demote_meta(const MoveArgs& a, uint64_t j, uint32_t v) {
  const PartGeom& g = a.g;
  const EntryState& st = a.st;
  const uint32_t t = st.tag[v];
  if (st.state[v] != KV_STATE_RESIDENT || t == KV_NONE) {
    atomicOr(a.status, KV_DEV_VICTIM_NOT_RESIDENT);
    return;
  }
  const uint32_t slot = (uint32_t)((a.ring_start + j) % g.ring_slots);
  const uint32_t old = g.r_tag[slot];
  if (old != KV_NONE) a.loc[old] = KV_NONE;  // an overwritten host entry is dropped
  const uint32_t pr = st.pair[v], le = st.last_epoch[v];
  const float em = st.ema[v], de = st.decay[v];
  g.r_tag[slot] = t;
  g.r_pair[slot] = (uint8_t)pr;
  g.r_ema[slot] = em;
  g.r_decay[slot] = de;
  g.r_last_epoch[slot] = le;
  g.r_depoch[slot] = g.epoch_now;
  a.loc[t] = KV_LOC_HOST | slot;
  st.state[v] = KV_STATE_FREE;
  st.pair[v] = (uint8_t)(pr | kPairFree);
  st.tag[v] = KV_NONE;
  st.touch[v] = 0;
  if (a.meta_offset != ~0ull) {
    uint32_t* rec = reinterpret_cast<uint32_t*>(a.staging + a.meta_offset + j * kMetaBytes);
    rec[0] = t;
    rec[1] = le;
    rec[2] = __float_as_uint(em);
    rec[3] = __float_as_uint(de);
    rec[4] = pr;
    rec[5] = g.epoch_now;
  }
}

// Metadata of one promoted entry: restored as it was when demoted (with lazy decay on,
// the EMA first takes the steps it missed).
__device__ __forceinline__ void promote_meta(const MoveArgs& a, uint32_t f, uint32_t slot) {
  const PartGeom& g = a.g;
  const EntryState& st = a.st;
  const uint32_t t = g.r_tag[slot];
  if (t == KV_NONE || st.state[f] != KV_STATE_FREE) {
    atomicOr(a.status, KV_DEV_BAD_INDEX);
    return;
  }
  st.pair[f] = g.r_pair[slot];
  const float de = g.r_decay[slot];
  float em = g.r_ema[slot];
  if (g.lazy_decay && g.epoch_now > g.r_depoch[slot]) em = ema_catch_up(em, de, g.epoch_now - g.r_depoch[slot]);
  st.ema[f] = em;
  st.decay[f] = de;
  st.last_epoch[f] = g.r_last_epoch[slot];
  st.tag[f] = t;
  st.touch[f] = 0;
  st.state[f] = KV_STATE_RESIDENT;
  a.loc[t] = f;
  g.r_tag[slot] = KV_NONE;  // the host slot is dead
}

// PACK = true: slab -> staging (entry images back to back).  PACK = false: staging -> slab.
// Each CTA owns a contiguous range of entries [e0, e1).
template <bool PACK>
__global__ void __launch_bounds__(kMoveThreads)
move_tma_kernel(const MoveArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ __align__(8) uint64_t bars[kStages];
  const PartGeom& g = a.g;
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t warp = threadIdx.x >> 5;
  const uint64_t per = (a.count + gridDim.x - 1) / gridDim.x;
  const uint64_t e0 = (uint64_t)blockIdx.x * per;
  const uint64_t e1 = (e0 + per < a.count) ? e0 + per : a.count;
  if (e0 >= e1) return;

  if (warp == 1) {
    // ---- metadata warp: one lane per entry ----
    for (uint64_t j = e0 + lane; j < e1; j += 32) {
      const uint32_t id = a.ids[j];
      if ((uint64_t)id < g.base || (uint64_t)id >= g.base + g.n) {
        atomicOr(a.status, KV_DEV_BAD_INDEX);
        continue;
      }
      if (PACK) {
        if (a.mode == kMoveCopyOnly) {
          // the entry's metadata moved earlier: the record for the host mirror comes from the ring mirror
          if (a.meta_offset != ~0ull) {
            const uint32_t slot = (uint32_t)((a.ring_start + j) % g.ring_slots);
            uint32_t* rec = reinterpret_cast<uint32_t*>(a.staging + a.meta_offset + j * kMetaBytes);
            rec[0] = g.r_tag[slot];
            rec[1] = g.r_last_epoch[slot];
            rec[2] = __float_as_uint(g.r_ema[slot]);
            rec[3] = __float_as_uint(g.r_decay[slot]);
            rec[4] = g.r_pair[slot];
            rec[5] = g.r_depoch[slot];
          }
          continue;
        }
        demote_meta(a, j, id);
      } else {
        const uint32_t slot = a.slots[j];
        if (slot >= g.ring_slots) {
          atomicOr(a.status, KV_DEV_BAD_INDEX);
          continue;
        }
        promote_meta(a, id, slot);
      }
    }
    return;
  }

  // ---- copy warp: lane 0 drives the bulk copies, all lanes fetch entry ids ----
  if (PACK && a.mode == kMoveMetaOnly) return;
  if (lane == 0) {
    for (uint32_t s = 0; s < kStages; ++s) mbar_init(&bars[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();

  const uint32_t ppc = (g.chunk_bytes + kStageBytes - 1) / kStageBytes;  // pieces per chunk
  const uint32_t ppe = ppc * g.n_chunks;                                  // pieces per entry
  // Software pipeline over the pieces of this CTA, in order: piece number `issued`
  // is the next to load, `stored` the next to store.  Loads run kStages-1 ahead.
  uint64_t issued = 0, stored = 0;
  bool ok = true;
  // destinations of the pieces in flight, indexed by stage (lane 0 only)
  __shared__ uint8_t* dst_of[kStages];
  __shared__ uint32_t len_of[kStages];

  uint32_t next_id = (e0 + lane < e1) ? a.ids[e0 + lane] : 0u;
  for (uint64_t jb = e0; jb < e1 && ok; jb += 32) {
    const uint32_t my_id = next_id;
    if (jb + 32 + lane < e1) next_id = a.ids[jb + 32 + lane];  // prefetch the next batch of ids
    const uint32_t in_batch = (uint32_t)((e1 - jb < 32) ? e1 - jb : 32);
    for (uint32_t t = 0; t < in_batch; ++t) {
      const uint32_t id = __shfl_sync(0xFFFFFFFFu, my_id, t);
      if (lane != 0) continue;
      const uint64_t j = jb + t;
      if ((uint64_t)id < g.base || (uint64_t)id >= g.base + g.n) continue;  // flagged by the metadata warp
      const uint64_t local = (uint64_t)id - g.base;
      uint8_t* image = a.staging + j * (uint64_t)g.entry_bytes;
      for (uint32_t r = 0; r < ppe && ok; ++r) {
        const uint32_t c = r / ppc;
        const uint32_t in_chunk = (r - c * ppc) * kStageBytes;
        const uint32_t len = min(kStageBytes, g.chunk_bytes - in_chunk);
        uint8_t* in_slab = g.slab + slab_chunk_offset(g, local, c) + in_chunk;
        uint8_t* in_image = image + (uint64_t)c * g.chunk_bytes + in_chunk;
        // keep at most kStages-1 loads ahead of the stores: retire the oldest first
        if (issued - stored == kStages - 1) {
          const uint32_t s = (uint32_t)(stored % kStages);
          ok = mbar_wait(&bars[s], (uint32_t)((stored / kStages) & 1u));
          if (!ok) break;
          fence_async_smem();
          bulk_store(dst_of[s], smem + s * kStageBytes, len_of[s]);
          ++stored;
          bulk_wait_read_1();  // every store but the newest has finished reading its stage
        }
        const uint32_t s = (uint32_t)(issued % kStages);
        dst_of[s] = PACK ? in_image : in_slab;
        len_of[s] = len;
        mbar_expect_tx(&bars[s], len);
        bulk_load(smem + s * kStageBytes, PACK ? in_slab : in_image, len, &bars[s]);
        ++issued;
      }
    }
    ok = __shfl_sync(0xFFFFFFFFu, (int)ok, 0) != 0;
  }
  if (lane == 0) {
    while (ok && stored < issued) {  // drain
      const uint32_t s = (uint32_t)(stored % kStages);
      ok = mbar_wait(&bars[s], (uint32_t)((stored / kStages) & 1u));
      if (!ok) break;
      fence_async_smem();
      bulk_store(dst_of[s], smem + s * kStageBytes, len_of[s]);
      ++stored;
    }
    if (!ok) {
      atomicOr(a.status, KV_DEV_WAIT_EXPIRED);
      // give the loads still in flight a (bounded) chance to land before the CTA's
      // shared memory goes away
      for (uint64_t p = stored; p < issued; ++p)
        (void)mbar_wait(&bars[p % kStages], (uint32_t)((p / kStages) & 1u));
    }
    bulk_wait_all();
  }
}

// ---- promotion of scattered host entries --------------------------------------------
// A prefetch list ordered by token position names, for every block, its layers one after
// the other; in the host ring only a block's heads are neighbours, its layers lie a whole
// demotion's share apart.  Such a list breaks into runs of a few slots, and one DMA
// transfer per run spends its time on set-up.  This kernel fetches the listed entries
// itself, through the address at which the device sees the pinned ring, and writes them
// straight into their paged slots: no staging buffer, no per-run transfer.  A warp moves
// one piece of up to 2 KB at a time with four 16-byte loads in flight per lane.
constexpr uint32_t kGatherPiece = 2048;   // 32 lanes x 4 x 16 bytes
constexpr uint32_t kGatherThreads = 256;

__global__ void __launch_bounds__(kGatherThreads)
gather_promote_kernel(const MoveArgs a, const uint8_t* __restrict__ ring) {
  const PartGeom& g = a.g;
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t ppc = (g.chunk_bytes + kGatherPiece - 1) / kGatherPiece;  // pieces per chunk
  const uint32_t ppe = ppc * g.n_chunks;                                    // pieces per entry
  const uint64_t total = a.count * ppe;
  const uint64_t warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
  for (uint64_t piece = (((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5); piece < total; piece += warps) {
    const uint64_t j = piece / ppe;
    const uint32_t r = (uint32_t)(piece - j * ppe);
    const uint32_t c = r / ppc;
    const uint32_t in_chunk = (r - c * ppc) * kGatherPiece;
    const uint32_t f = a.ids[j];
    const uint32_t slot = a.slots[j];
    if ((uint64_t)f < g.base || (uint64_t)f >= g.base + g.n || slot >= g.ring_slots) {
      if (lane == 0 && r == 0) atomicOr(a.status, KV_DEV_BAD_INDEX);
      continue;
    }
    const uint32_t len = min(kGatherPiece, g.chunk_bytes - in_chunk);
    const uint8_t* src = ring + (uint64_t)slot * g.entry_bytes + (uint64_t)c * g.chunk_bytes + in_chunk;
    uint8_t* dst = g.slab + slab_chunk_offset(g, (uint64_t)f - g.base, c) + in_chunk;
    uint4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint32_t off = (u * 32 + lane) * 16;
      if (off < len) v[u] = __ldcs(reinterpret_cast<const uint4*>(src + off));
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint32_t off = (u * 32 + lane) * 16;
      if (off < len) __stcs(reinterpret_cast<uint4*>(dst + off), v[u]);
    }
    if (r == 0 && lane == 0) promote_meta(a, f, slot);
  }
}

cudaError_t launch_gather_promote(const PartGeom& g, const EntryState& st, uint32_t* loc, const uint32_t* slots,
                                  const uint32_t* free_ids, uint64_t count, const uint8_t* ring_dev,
                                  const Workspace& ws, cudaStream_t s) {
  if (count == 0) return cudaSuccess;
  MoveArgs a{g, st, loc, free_ids, slots, count, 0, nullptr, ~0ull, ws.status, kMoveAll};
  const uint64_t pieces = count * ((g.chunk_bytes + kGatherPiece - 1) / kGatherPiece) * g.n_chunks;
  uint64_t blocks = (pieces * 32 + kGatherThreads - 1) / kGatherThreads;
  // 32 blocks keep 512 KB of reads in flight, several round trips' worth of the host link; more
  // blocks crowd out the D2H transfers of a demotion running at the same time without moving more
  // (measured: both directions together carry ~63 GB/s whatever the split)
  const uint64_t cap = 32;
  if (blocks > cap) blocks = cap;
  gather_promote_kernel<<<(unsigned)(blocks ? blocks : 1), kGatherThreads, 0, s>>>(a, ring_dev);
  count_launches(1);
  return cudaGetLastError();
}

static unsigned tma_grid(uint64_t count) {
  const uint64_t cap = (uint64_t)sm_count() * kMoveCtasPerSm;
  uint64_t blocks = count < cap ? count : cap;
  return (unsigned)(blocks ? blocks : 1);
}

template <bool PACK>
static cudaError_t launch_move(const MoveArgs& a, cudaStream_t s) {
  // the opt-in for the shared memory belongs to a device: once per device ordinal
  static std::atomic<bool> configured[64];
  const size_t smem = (size_t)kStages * kStageBytes;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return cudaGetLastError();
  if (dev < 0 || dev >= 64 || !configured[dev].load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(move_tma_kernel<PACK>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev].store(true, std::memory_order_release);
  }
  move_tma_kernel<PACK><<<tma_grid(a.count), kMoveThreads, smem, s>>>(a);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_pack_tma(const PartGeom& g, const EntryState& st, uint32_t* loc, const uint32_t* victims,
                            uint64_t count, uint64_t ring_start, uint8_t* staging, uint64_t meta_offset,
                            const Workspace& ws, cudaStream_t s, uint32_t mode) {
  if (count == 0) return cudaSuccess;
  MoveArgs a{g, st, loc, victims, nullptr, count, ring_start, staging, meta_offset, ws.status, mode};
  return launch_move<true>(a, s);
}

cudaError_t launch_unpack_tma(const PartGeom& g, const EntryState& st, uint32_t* loc, const uint32_t* slots,
                              const uint32_t* free_ids, uint64_t count, const uint8_t* staging,
                              const Workspace& ws, cudaStream_t s) {
  if (count == 0) return cudaSuccess;
  MoveArgs a{g, st, loc, free_ids, slots, count, 0, const_cast<uint8_t*>(staging), ~0ull, ws.status, kMoveAll};
  return launch_move<false>(a, s);
}

}  // namespace kvt
