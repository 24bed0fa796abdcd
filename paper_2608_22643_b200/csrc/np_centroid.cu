// Selection through centroid heads: the predictor's last stage as the paper
// describes it (Section 3.3: two groups of per-layer heads emit logits over a
// vocabulary of K centroids and each head takes its most likely centroid;
// Section 3.4: a layer's active set is the gate centroid's mask AND the up
// centroid's mask).
//
// One block per (layer, sequence).  Both heads' arg-max are found with a packed
// (order key, inverted index) maximum, so equal logits resolve to the lower
// centroid ID; then the two bank rows are ANDed word by word into the layer's
// bitmap (ORed over sequences when B > 1).
#include "np_device.cuh"
#include "np_internal.h"

namespace npi {
using namespace npd;

constexpr int kCentroidThreads = 256;

__device__ __forceinline__ uint32_t centroid_order_key(uint32_t b) {  // the fp32 value's bit pattern (a float move may flush a denormal)
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__global__ void __launch_bounds__(kCentroidThreads)
    k_centroid_select(const float* __restrict__ logits,   // [B][L][2][K]
                      const uint32_t* __restrict__ bank,  // [L][2][K][W]
                      int32_t* __restrict__ ids_out,      // [B][L][2] or NULL
                      uint32_t* __restrict__ bitmap,      // [L][W]
                      int L, int K, int W, int use_atomic) {
  __shared__ unsigned long long s_best[2][kCentroidThreads / 32];
  __shared__ int s_pick[2];
  const int layer = blockIdx.x, b = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const float* z = logits + ((size_t)b * L + layer) * 2 * K;

  for (int h = 0; h < 2; ++h) {
    unsigned long long best = 0ull;  // below every real entry: keys are never 0 with index bits set
    for (int c = tid; c < K; c += kCentroidThreads) {
      const unsigned long long v =
          ((unsigned long long)centroid_order_key(__ldg(reinterpret_cast<const uint32_t*>(z) + (size_t)h * K + c)) << 32) | (uint32_t)(~(uint32_t)c);
      best = v > best ? v : best;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
      best = other > best ? other : best;
    }
    if (lane == 0) s_best[h][wid] = best;
  }
  __syncthreads();
  if (tid < 2) {
    unsigned long long best = 0ull;
    for (int w = 0; w < kCentroidThreads / 32; ++w) best = s_best[tid][w] > best ? s_best[tid][w] : best;
    const int pick = (int)(~(uint32_t)(best & 0xffffffffull));
    s_pick[tid] = pick;
    if (ids_out) ids_out[((size_t)b * L + layer) * 2 + tid] = pick;
  }
  __syncthreads();
  const uint32_t* g = bank + (((size_t)layer * 2 + 0) * K + s_pick[0]) * W;
  const uint32_t* u = bank + (((size_t)layer * 2 + 1) * K + s_pick[1]) * W;
  uint32_t* out = bitmap + (size_t)layer * W;
  for (int w = tid; w < W; w += kCentroidThreads) {
    const uint32_t m = __ldg(g + w) & __ldg(u + w);
    if (use_atomic) {
      if (m) atomicOr(out + w, m);
    } else {
      out[w] = m;
    }
  }
}

cudaError_t launch_centroid_select(const Dims& d, const float* logits, int B, int K, const uint32_t* bank,
                                   int32_t* ids_out, uint32_t* bitmap, cudaStream_t s) {
  const int use_atomic = B > 1 ? 1 : 0;
  if (use_atomic) {
    cudaError_t e = cudaMemsetAsync(bitmap, 0, (size_t)d.L * d.W * 4, s);
    if (e != cudaSuccess) return e;
  }
  dim3 grid(d.L, B);
  k_centroid_select<<<grid, kCentroidThreads, 0, s>>>(logits, bank, ids_out, bitmap, d.L, K, d.W, use_atomic);
  return cudaGetLastError();
}

}  // namespace npi
