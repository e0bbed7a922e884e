// Content hashing and deduplication of head-granular entries.
//
// The paper keeps a content-addressable store in which blocks are indexed by the
// SHA-256 hash of their content; a new block whose hash is already in the store
// gets a reference instead of a second copy (content-addressable deduplication
// section).  Here both halves run on the GPU, next to the data:
//
//   hash_entries_kernel   one thread per entry walks the entry's image (K chunk
//                         then V chunk, or the MLA chunk) in 64-byte blocks through
//                         the SHA-256 compression function of FIPS 180-4.  The
//                         work is integer arithmetic (about 25 instructions per
//                         byte), not memory traffic: a thread reads its 64 bytes as
//                         four 16-byte loads and then spends ~1,600 instructions on
//                         them.  Shifts and logic operations fill the integer pipe, so
//                         the additions are issued as multiply-adds, which run on the
//                         FMA pipe beside it (861 -> 1,025 GB/s on 8 KB entries).
//   dedup_insert_kernel / dedup_resolve_kernel
//                         an open-addressing table of list positions, probed from
//                         the first 8 bytes of the digest (a SHA-256 digest is as
//                         good a hash key as any), with the full 32 bytes compared
//                         on every probe.  Insertion keeps the SMALLEST position per
//                         digest (atomicMin), so the result does not depend on the
//                         order in which threads run: the first block of the list
//                         with a given content is the stored copy, as in a store
//                         that blocks enter one after the other.
//
// The round constants and the initial hash value are the ones FIPS 180-4 defines
// (the first 32 bits of the fractional parts of the cube roots of the first 64
// primes, and of the square roots of the first 8).
#include "kvtier_internal.cuh"

namespace kvt {

__constant__ uint32_t kShaK[64] = {
    0x428a2f98u, 0x71374491u, 0xb5c0fbcfu, 0xe9b5dba5u, 0x3956c25bu, 0x59f111f1u, 0x923f82a4u, 0xab1c5ed5u,
    0xd807aa98u, 0x12835b01u, 0x243185beu, 0x550c7dc3u, 0x72be5d74u, 0x80deb1feu, 0x9bdc06a7u, 0xc19bf174u,
    0xe49b69c1u, 0xefbe4786u, 0x0fc19dc6u, 0x240ca1ccu, 0x2de92c6fu, 0x4a7484aau, 0x5cb0a9dcu, 0x76f988dau,
    0x983e5152u, 0xa831c66du, 0xb00327c8u, 0xbf597fc7u, 0xc6e00bf3u, 0xd5a79147u, 0x06ca6351u, 0x14292967u,
    0x27b70a85u, 0x2e1b2138u, 0x4d2c6dfcu, 0x53380d13u, 0x650a7354u, 0x766a0abbu, 0x81c2c92eu, 0x92722c85u,
    0xa2bfe8a1u, 0xa81a664bu, 0xc24b8b70u, 0xc76c51a3u, 0xd192e819u, 0xd6990624u, 0xf40e3585u, 0x106aa070u,
    0x19a4c116u, 0x1e376c08u, 0x2748774cu, 0x34b0bcb5u, 0x391c0cb3u, 0x4ed8aa4au, 0x5b9cca4fu, 0x682e6ff3u,
    0x748f82eeu, 0x78a5636fu, 0x84c87814u, 0x8cc70208u, 0x90befffau, 0xa4506cebu, 0xbef9a3f7u, 0xc67178f2u};

struct HashGeom {
  PartGeom part[4];
  int n_parts;
};

__device__ __forceinline__ uint32_t rotr(uint32_t x, uint32_t n) { return __funnelshift_r(x, x, n); }
// the standard reads the message as big-endian 32-bit words
__device__ __forceinline__ uint32_t be32(uint32_t x) { return __byte_perm(x, 0, 0x0123); }

// One application of the compression function: st <- st + compress(st, w), w = the
// 16 message words of the block (overwritten by the message schedule).
// x + y as an integer multiply-add x * one + y (one = 1, a kernel argument so that it stays a
// multiply-add): it issues to the FMA pipe, while the shifts, logic operations and plain adds of
// the compression function all queue for the integer pipe, which is the kernel's bottleneck.
__device__ __forceinline__ uint32_t add_on_fma_pipe(uint32_t x, uint32_t y, uint32_t one) {
  uint32_t r;
  asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(x), "r"(one), "r"(y));
  return r;
}

__device__ __forceinline__ void sha256_block(uint32_t st[8], uint32_t w[16], uint32_t one) {
  uint32_t a = st[0], b = st[1], c = st[2], d = st[3], e = st[4], f = st[5], g = st[6], h = st[7];
#pragma unroll
  for (int i = 0; i < 64; ++i) {
    if (i >= 16) {
      const uint32_t w15 = w[(i + 1) & 15], w2 = w[(i + 14) & 15];
      const uint32_t s0 = rotr(w15, 7) ^ rotr(w15, 18) ^ (w15 >> 3);
      const uint32_t s1 = rotr(w2, 17) ^ rotr(w2, 19) ^ (w2 >> 10);
      w[i & 15] = add_on_fma_pipe(add_on_fma_pipe(w[i & 15], s0, one), add_on_fma_pipe(w[(i + 9) & 15], s1, one), one);
    }
    const uint32_t S1 = rotr(e, 6) ^ rotr(e, 11) ^ rotr(e, 25);
    const uint32_t ch = (e & f) ^ (~e & g);
    const uint32_t t1 = add_on_fma_pipe(add_on_fma_pipe(h, S1, one), add_on_fma_pipe(ch, add_on_fma_pipe(w[i & 15], kShaK[i], one), one), one);
    const uint32_t S0 = rotr(a, 2) ^ rotr(a, 13) ^ rotr(a, 22);
    const uint32_t maj = (a & b) ^ (a & c) ^ (b & c);
    const uint32_t t2 = add_on_fma_pipe(S0, maj, one);
    h = g; g = f; f = e; e = add_on_fma_pipe(d, t1, one); d = c; c = b; b = a; a = add_on_fma_pipe(t1, t2, one);
  }
  st[0] += a; st[1] += b; st[2] += c; st[3] += d; st[4] += e; st[5] += f; st[6] += g; st[7] += h;
}

__device__ __forceinline__ uint64_t hash_chunk_offset(const PartGeom& g, uint64_t local, uint32_t c) {
  const uint64_t lb = local / g.heads;
  const uint64_t head = local - lb * g.heads;
  return ((lb * g.n_chunks + c) * g.heads + head) * (uint64_t)g.chunk_bytes;
}

// digests[j] = SHA-256 of the image of entry ids[j] (ids == nullptr: entry j).
// Chunk sizes are multiples of 16 bytes (a pool with others is refused), so a 16-byte piece
// of the image never straddles the K and V chunks.
__global__ void __launch_bounds__(128)
hash_entries_kernel(const HashGeom hg, const uint32_t* __restrict__ ids, uint64_t m,
                    uint8_t* __restrict__ digests, uint32_t* __restrict__ status, uint32_t one) {
  const uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= m) return;
  const uint64_t id = ids ? ids[j] : j;
  int q = -1;
  for (int i = 0; i < hg.n_parts; ++i)
    if (id >= hg.part[i].base && id < hg.part[i].base + hg.part[i].n) q = i;
  if (q < 0) {
    atomicOr(status, KV_DEV_BAD_INDEX);
    return;
  }
  const PartGeom& g = hg.part[q];
  const uint64_t local = id - g.base;
  const uint8_t* ck = g.slab + hash_chunk_offset(g, local, 0);
  const uint8_t* cv = g.n_chunks > 1 ? g.slab + hash_chunk_offset(g, local, 1) : ck;
  const uint32_t cb = g.chunk_bytes, eb = g.entry_bytes;
  auto piece = [&](uint32_t off) -> uint4 {   // 16 bytes of the image at byte offset off
    const uint8_t* p = off < cb ? ck + off : cv + (off - cb);
    return __ldg(reinterpret_cast<const uint4*>(p));
  };
  uint32_t st[8] = {0x6a09e667u, 0xbb67ae85u, 0x3c6ef372u, 0xa54ff53au,
                    0x510e527fu, 0x9b05688cu, 0x1f83d9abu, 0x5be0cd19u};
  uint32_t w[16];
  const uint32_t full = eb / 64;
  for (uint32_t b = 0; b < full; ++b) {
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint4 v = piece(b * 64 + u * 16);
      w[4 * u + 0] = be32(v.x); w[4 * u + 1] = be32(v.y); w[4 * u + 2] = be32(v.z); w[4 * u + 3] = be32(v.w);
    }
    sha256_block(st, w, one);
  }
  // last block: what is left of the image (0, 16, 32 or 48 bytes), the 1 bit, zeros, the length in bits
  const uint32_t rem = eb - full * 64;
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    uint4 v = make_uint4(0, 0, 0, 0);
    if ((uint32_t)u * 16 < rem) v = piece(full * 64 + u * 16);
    w[4 * u + 0] = be32(v.x); w[4 * u + 1] = be32(v.y); w[4 * u + 2] = be32(v.z); w[4 * u + 3] = be32(v.w);
  }
#pragma unroll
  for (int i = 0; i < 16; ++i)
    if ((uint32_t)i * 4 == rem) w[i] = 0x80000000u;
  w[14] = (uint32_t)(((uint64_t)eb * 8) >> 32);   // rem <= 48: the length always fits this block
  w[15] = (uint32_t)((uint64_t)eb * 8);
  sha256_block(st, w, one);
  uint4* out = reinterpret_cast<uint4*>(digests + j * 32);
  out[0] = make_uint4(be32(st[0]), be32(st[1]), be32(st[2]), be32(st[3]));
  out[1] = make_uint4(be32(st[4]), be32(st[5]), be32(st[6]), be32(st[7]));
}

cudaError_t launch_hash_entries(const PartGeom* parts, int n_parts, const uint32_t* ids, uint64_t m,
                                uint8_t* digests, const Workspace& ws, cudaStream_t s) {
  if (m == 0) return cudaSuccess;
  HashGeom hg;
  for (int q = 0; q < 4; ++q) hg.part[q] = parts[q < n_parts ? q : 0];
  hg.n_parts = n_parts;
  const uint64_t blocks = (m + 127) / 128;
  hash_entries_kernel<<<(unsigned)blocks, 128, 0, s>>>(hg, ids, m, digests, ws.status, 1u);
  count_launches(1);
  return cudaGetLastError();
}

// ---- reference counting ----------------------------------------------------------
constexpr uint32_t kEmpty = 0xFFFFFFFFu;

__device__ __forceinline__ bool same_digest(const uint8_t* d, uint64_t a, uint64_t b) {
  const uint4* pa = reinterpret_cast<const uint4*>(d + a * 32);
  const uint4* pb = reinterpret_cast<const uint4*>(d + b * 32);
  const uint4 a0 = __ldg(pa), a1 = __ldg(pa + 1), b0 = __ldg(pb), b1 = __ldg(pb + 1);
  return a0.x == b0.x && a0.y == b0.y && a0.z == b0.z && a0.w == b0.w &&
         a1.x == b1.x && a1.y == b1.y && a1.z == b1.z && a1.w == b1.w;
}

__device__ __forceinline__ uint64_t probe_start(const uint8_t* d, uint64_t j, uint64_t mask) {
  return __ldg(reinterpret_cast<const unsigned long long*>(d + j * 32)) & mask;
}

__global__ void dedup_clear_kernel(uint32_t* table, uint64_t slots, uint32_t* refcount, uint64_t m,
                                   uint32_t* n_unique) {
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  const uint64_t i0 = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  for (uint64_t i = i0; i < slots; i += stride) table[i] = kEmpty;
  for (uint64_t i = i0; i < m; i += stride) refcount[i] = 0;
  if (i0 == 0 && n_unique) *n_unique = 0;
}

// Every position j enters the table: an empty slot is claimed, a slot that holds a
// position with the same digest keeps the smaller of the two, any other slot is
// passed by.  The table has at least 2*m slots, so a probe sequence always ends;
// it is bounded by the table size all the same.
__global__ void dedup_insert_kernel(const uint8_t* __restrict__ digests, uint64_t m, uint32_t* table,
                                    uint64_t mask, uint32_t* status) {
  const uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= m) return;
  uint64_t s = probe_start(digests, j, mask);
  for (uint64_t step = 0; step <= mask; ++step, s = (s + 1) & mask) {
    uint32_t cur = atomicCAS(&table[s], kEmpty, (uint32_t)j);
    if (cur == kEmpty) return;
    if (same_digest(digests, cur, j)) {   // whoever holds the slot has this digest: it can only be replaced by one that does
      atomicMin(&table[s], (uint32_t)j);
      return;
    }
  }
  atomicOr(status, KV_DEV_WAIT_EXPIRED);
}

// After all insertions: canon[j] = the smallest position with j's digest; its
// reference count goes up by one.
__global__ void dedup_resolve_kernel(const uint8_t* __restrict__ digests, uint64_t m,
                                     const uint32_t* __restrict__ table, uint64_t mask,
                                     uint32_t* __restrict__ canon, uint32_t* refcount, uint32_t* n_unique,
                                     uint32_t* status) {
  const uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= m) return;
  uint64_t s = probe_start(digests, j, mask);
  for (uint64_t step = 0; step <= mask; ++step, s = (s + 1) & mask) {
    const uint32_t cur = table[s];
    if (cur == kEmpty) break;
    if (same_digest(digests, cur, j)) {
      canon[j] = cur;
      atomicAdd(&refcount[cur], 1u);
      if (cur == (uint32_t)j && n_unique) atomicAdd(n_unique, 1u);
      return;
    }
  }
  atomicOr(status, KV_DEV_BAD_INDEX);   // j was inserted, so it must be found
}

cudaError_t launch_dedup(const uint8_t* digests, uint64_t m, uint32_t* canon, uint32_t* refcount,
                         uint32_t* table, uint64_t table_slots, uint32_t* n_unique, uint32_t* status,
                         cudaStream_t s) {
  const uint64_t cap = (uint64_t)sm_count() * 8;
  uint64_t cb = ((table_slots > m ? table_slots : m) + kThreads - 1) / kThreads;
  if (cb == 0) cb = 1;
  dedup_clear_kernel<<<(unsigned)(cb > cap ? cap : cb), kThreads, 0, s>>>(table, table_slots, refcount, m, n_unique);
  count_launches(1);
  if (m == 0) return cudaGetLastError();
  const uint64_t blocks = (m + kThreads - 1) / kThreads;
  dedup_insert_kernel<<<(unsigned)blocks, kThreads, 0, s>>>(digests, m, table, table_slots - 1, status);
  dedup_resolve_kernel<<<(unsigned)blocks, kThreads, 0, s>>>(digests, m, table, table_slots - 1, canon, refcount,
                                                           n_unique, status);
  count_launches(2);
  return cudaGetLastError();
}

}  // namespace kvt
