// Head-granular importance: the [layer][head] importance matrix of the
// head-granular eviction section, kept per partition.
//
// The paper states that the matrix is an exponential moving average updated on
// every attention step, that for GQA the query heads sharing a KV head are
// grouped and the group's maximum is the KV head's score, that for MLA the
// matrix is [layer][1], and that per-head multipliers bias eviction at task
// transitions; it prints no formula.  The form used here:
//   M[l][j] <- d*M[l][j] + (1-d)*x[l][j]        (binary32, each operation rounded once)
//   W[l][h] = max over the group of h of M[l][.]  *  mult[l][h]
// and the entry pass multiplies the score of entry (l, block, h) by W[l][h].
#include "kvtier_internal.cuh"

namespace kvt {

__device__ __forceinline__ bool head_value_ok(float v) {
  return v >= 0.0f && v <= 3.402823466e+38f;  // false for NaN, negatives and infinities
}

// One thread per (layer, KV head) of the partition.
__global__ void head_update_kernel(float* __restrict__ imp, float* __restrict__ mult, float* __restrict__ w,
                                   const float* __restrict__ src, float d, uint32_t layers, uint32_t q_heads,
                                   uint32_t heads, int mode, uint32_t* __restrict__ status) {
  const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= layers * heads) return;
  const uint32_t l = i / heads, h = i % heads;
  const uint32_t G = q_heads / heads;
  uint32_t bad = 0;
  if (mode == 1) {
    float v = 1.0f;
    if (src) v = src[i];
    if (head_value_ok(v)) mult[i] = v; else bad = 1;
  }
  float m = 0.0f;
  for (uint32_t g = 0; g < G; ++g) {
    const uint32_t j = l * q_heads + h * G + g;
    float v = imp[j];
    if (mode == 0) {
      const float x = src[j];
      if (head_value_ok(x)) {
        const float t1 = __fmul_rn(d, v);
        const float t2 = __fsub_rn(1.0f, d);
        const float t3 = __fmul_rn(t2, x);
        v = __fadd_rn(t1, t3);
        imp[j] = v;
      } else {
        bad = 1;
      }
    }
    m = (g == 0 || v > m) ? v : m;
  }
  w[i] = __fmul_rn(m, mult[i]);
  if (bad) atomicOr(status, KV_DEV_BAD_HEAD_VALUE);
}

__global__ void head_init_kernel(float* imp, float* mult, float* w, uint32_t n_imp, uint32_t n_w) {
  const uint32_t stride = gridDim.x * blockDim.x;
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n_imp; i += stride) imp[i] = 1.0f;
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n_w; i += stride) {
    mult[i] = 1.0f;
    w[i] = 1.0f;
  }
}

cudaError_t launch_head_update(const HeadWeights& hw, int q, int mode, const float* src, float decay,
                               const Workspace& ws, cudaStream_t s) {
  const uint32_t n = hw.layers[q] * hw.heads[q];
  head_update_kernel<<<(n + 127) / 128, 128, 0, s>>>(hw.imp + hw.imp_off[q], hw.mult + hw.w_off[q],
                                                     hw.w + hw.w_off[q], src, decay, hw.layers[q],
                                                     hw.q_heads[q], hw.heads[q], mode, ws.status);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_head_init(const HeadWeights& hw, uint32_t n_imp, uint32_t n_w, cudaStream_t s) {
  head_init_kernel<<<8, 256, 0, s>>>(hw.imp, hw.mult, hw.w, n_imp, n_w);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace kvt
