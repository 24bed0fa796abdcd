// Stage 2: per-layer top-k of the predictor's logits -> active-neuron bitmap.
// (The paper turns predictor outputs into one active set per layer, Section 3.4;
// here the set is the k highest-scoring neurons, the K_max budget of Section 4.1.)
//
// One block per (layer, sequence).  The layer's logits are mapped to
// order-preserving uint32 keys in shared memory, a 4-pass 8-bit radix select
// finds the k-th largest key, and a ballot pass over 32-neuron words admits
// every key above the threshold plus the lowest-indexed keys equal to it.
#include "np_device.cuh"
#include "np_internal.h"

namespace npi {
using namespace npd;

constexpr int kTopkThreads = 1024;

__device__ __forceinline__ uint32_t order_key(float z) {
  const uint32_t b = __float_as_uint(z);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__global__ void __launch_bounds__(kTopkThreads) k_topk(const float* __restrict__ logits,  // [B][L][M]
                                                       uint32_t* __restrict__ bitmap,     // [L][W]
                                                       int L, int M, int k, int use_atomic) {
  extern __shared__ __align__(16) uint32_t smem[];
  const int W = M >> 5;
  uint32_t* keys = smem;                            // [M]
  int* eq_cnt = reinterpret_cast<int*>(keys + M);   // [W]
  int* whist = eq_cnt + W;                          // [32][256] per-warp histograms
  int* hist = whist + 32 * 256;                     // [256]
  int* red = hist + 256;                            // [40]
  __shared__ uint32_t s_prefix;
  __shared__ int s_remaining;

  const int layer = blockIdx.x, b = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const float* z = logits + ((size_t)b * L + layer) * M;
  uint32_t* out = bitmap + (size_t)layer * W;

  if (k <= 0) {  // nothing selected
    if (!use_atomic)
      for (int w = tid; w < W; w += blockDim.x) out[w] = 0u;
    return;
  }
  if (k >= M) {
    for (int w = tid; w < W; w += blockDim.x) {
      if (use_atomic) atomicOr(out + w, 0xffffffffu);
      else out[w] = 0xffffffffu;
    }
    return;
  }

  for (int i = tid; i < M; i += blockDim.x) keys[i] = order_key(z[i]);
  if (tid == 0) {
    s_prefix = 0u;
    s_remaining = k;
  }
  __syncthreads();

  uint32_t mask = 0u;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int i = tid; i < 32 * 256; i += blockDim.x) whist[i] = 0;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    for (int i = tid; i < M; i += blockDim.x) {
      const uint32_t key = keys[i];
      if ((key & mask) == prefix) atomicAdd(&whist[wid * 256 + ((key >> shift) & 255u)], 1);
    }
    __syncthreads();
    if (tid < 256) {
      int s = 0;
#pragma unroll 8
      for (int w = 0; w < 32; ++w) s += whist[w * 256 + tid];
      hist[tid] = s;
    }
    __syncthreads();
    if (wid == 0) {
      // lane handles bins [8*lane, 8*lane+8); find the highest bin whose suffix count reaches `remaining`
      const int remaining = s_remaining;
      int local[8], lsum = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        local[j] = hist[lane * 8 + j];
        lsum += local[j];
      }
      // suffix sum over lanes above this one
      int above = lsum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_down_sync(0xffffffffu, above, o);
        if (lane + o < 32) above += t;
      }
      above -= lsum;  // count in bins of higher lanes
      int found_bin = -1, found_above = 0;
      int run = above;
#pragma unroll
      for (int j = 7; j >= 0; --j) {
        if (found_bin < 0 && run < remaining && run + local[j] >= remaining) {
          found_bin = lane * 8 + j;
          found_above = run;
        }
        run += local[j];
      }
      const uint32_t vote = __ballot_sync(0xffffffffu, found_bin >= 0);
      const int src = 31 - __clz(vote);  // exactly one lane finds it; be safe with the highest
      const int bin = __shfl_sync(0xffffffffu, found_bin, src);
      const int abv = __shfl_sync(0xffffffffu, found_above, src);
      if (lane == 0) {
        s_prefix = prefix | ((uint32_t)bin << shift);
        s_remaining = remaining - abv;
      }
    }
    mask |= 0xffu << shift;
    __syncthreads();
  }

  const uint32_t thr = s_prefix;   // key of the k-th largest element
  const int admit = s_remaining;   // how many keys equal to thr are taken, lowest index first

  // per-word population of keys equal to the threshold
  for (int w = wid; w < W; w += (blockDim.x >> 5)) {
    const uint32_t key = keys[w * 32 + lane];
    const uint32_t eq = __ballot_sync(0xffffffffu, key == thr);
    if (lane == 0) eq_cnt[w] = __popc(eq);
  }
  block_exclusive_scan(eq_cnt, W, red);
  for (int w = wid; w < W; w += (blockDim.x >> 5)) {
    const uint32_t key = keys[w * 32 + lane];
    const uint32_t gt = __ballot_sync(0xffffffffu, key > thr);
    const uint32_t eq = __ballot_sync(0xffffffffu, key == thr);
    if (lane == 0) {
      const uint32_t word = gt | lowest_bits(eq, admit - eq_cnt[w]);
      if (use_atomic) {
        if (word) atomicOr(out + w, word);
      } else {
        out[w] = word;
      }
    }
  }
}

cudaError_t launch_topk(const Dims& d, const float* logits, int B, uint32_t* bitmap, cudaStream_t s) {
  const int W = d.W;
  const size_t sm = (size_t)d.M * 4 + (size_t)W * 4 + 32 * 256 * 4 + 256 * 4 + 40 * 4;
  // set on every launch: the attribute belongs to the current device's context
  if (sm > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(k_topk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (e != cudaSuccess) return e;
  }
  const int use_atomic = B > 1 ? 1 : 0;
  if (use_atomic) {
    cudaError_t e = cudaMemsetAsync(bitmap, 0, (size_t)d.L * W * 4, s);
    if (e != cudaSuccess) return e;
  }
  dim3 grid(d.L, B);
  k_topk<<<grid, kTopkThreads, sm, s>>>(logits, bitmap, d.L, d.M, d.k, use_atomic);
  return cudaGetLastError();
}

}  // namespace npi
