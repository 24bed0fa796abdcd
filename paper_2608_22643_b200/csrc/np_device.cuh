// Device-side helpers: bf16 unpacking, cache-hinted 128-bit loads, block scans.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace npd {

// device status bits (Tables::status[0])
constexpr int kStatBadSlot = 1;     // slot index outside [0, C)
constexpr int kStatBadNeuron = 2;   // neuron index outside [0, M)
constexpr int kStatBadCount = 4;    // a list count larger than its capacity
constexpr int kStatRange = 16;      // a partial MLP sum outside the range of the counted fixed-point words (or not a number)

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// 16-byte streaming load: read-only path, no L1 allocation (each weight byte is used once).
__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ void stg_stream(void* p, uint4 v) {
  asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y),
               "r"(v.z), "r"(v.w)
               : "memory");
}

// 8 bf16 (one uint4) times 8 fp32, accumulated.
__device__ __forceinline__ float dot8(uint4 w, const float4 a, const float4 b, float acc) {
  acc = fmaf(bf16_lo(w.x), a.x, acc);
  acc = fmaf(bf16_hi(w.x), a.y, acc);
  acc = fmaf(bf16_lo(w.y), a.z, acc);
  acc = fmaf(bf16_hi(w.y), a.w, acc);
  acc = fmaf(bf16_lo(w.z), b.x, acc);
  acc = fmaf(bf16_hi(w.z), b.y, acc);
  acc = fmaf(bf16_lo(w.w), b.z, acc);
  acc = fmaf(bf16_hi(w.w), b.w, acc);
  return acc;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__device__ __forceinline__ int warp_sum_int(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Block-wide sum of one int per thread; result returned to every thread.
// `red` is shared scratch of at least 33 ints.  Contains __syncthreads().
__device__ __forceinline__ int block_sum_int(int v, int* red) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum_int(v);
  __syncthreads();
  if (lane == 0) red[wid] = v;
  __syncthreads();
  if (wid == 0) {
    int t = lane < nw ? red[lane] : 0;
    t = warp_sum_int(t);
    if (lane == 0) red[32] = t;
  }
  __syncthreads();
  return red[32];
}

// In-place exclusive scan of a[0..n) in shared memory by the whole block;
// returns the total to every thread.  `red` is shared scratch of >= 34 ints.
__device__ __forceinline__ int block_exclusive_scan(int* a, int n, int* red) {
  const int T = blockDim.x, tid = threadIdx.x;
  const int lane = tid & 31, wid = tid >> 5, nw = (T + 31) >> 5;
  const int seg = (n + T - 1) / T;
  const int lo = min(n, tid * seg), hi = min(n, lo + seg);
  __syncthreads();
  int s = 0;
  for (int i = lo; i < hi; ++i) s += a[i];
  // inclusive scan of s across the block
  int inc = s;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) red[wid] = inc;
  __syncthreads();
  if (wid == 0) {
    int w = lane < nw ? red[lane] : 0;
    int winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int t = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += t;
    }
    red[lane] = winc - w;          // exclusive offset of each warp
    if (lane == 31) red[33] = winc;  // total
  }
  __syncthreads();
  int run = red[wid] + inc - s;
  const int total = red[33];
  for (int i = lo; i < hi; ++i) {
    int v = a[i];
    a[i] = run;
    run += v;
  }
  __syncthreads();
  return total;
}

// Inclusive scan of one int per thread over a block of 1024 threads, in thread order; returns
// this thread's inclusive value and leaves the block's total in wsum[32].  wsum: 33 ints of
// shared scratch.  Two block-wide barriers; a caller that scans again puts one between the calls.
__device__ __forceinline__ int block_inclusive_scan_1024(int v, int* wsum, int lane, int wid) {
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) wsum[wid] = inc;
  __syncthreads();
  if (wid == 0) {
    const int ws = wsum[lane];
    int winc = ws;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += t;
    }
    wsum[lane] = winc - ws;
    if (lane == 31) wsum[32] = winc;
  }
  __syncthreads();
  return wsum[wid] + inc;
}

// The n lowest set bits of m (all of m if it has fewer).
__device__ __forceinline__ uint32_t lowest_bits(uint32_t m, int n) {
  if (n <= 0) return 0u;
  if (n >= __popc(m)) return m;
  uint32_t out = 0;
  for (int i = 0; i < n; ++i) {
    uint32_t b = m & (0u - m);
    out |= b;
    m ^= b;
  }
  return out;
}

}  // namespace npd
