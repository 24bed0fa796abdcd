// Stage 3c: fused deinterleave + scatter (Section 3.5).  Each staged record
// holds a neuron's gate, up and transposed-down rows back to back; the kernel
// writes the three rows to the slot the delta step assigned, in the three
// projection-specific resident buffers.  Pure 16-byte coalesced copies.
//
// The same kernel serves the zero-copy transfer mode, where `src` is the whole
// layer of the pinned record store and records are addressed by neuron ID.
#include "np_device.cuh"
#include "np_internal.h"

namespace npi {
using namespace npd;

constexpr int kScatterThreads = 256;

template <bool kFromStore>
__global__ void __launch_bounds__(kScatterThreads) k_deinterleave_scatter(
    const uint4* __restrict__ src, const int32_t* __restrict__ ids, const int32_t* __restrict__ slots,
    const int32_t* __restrict__ count_ptr, int first, int max_rows, uint4* __restrict__ gate,
    uint4* __restrict__ up, uint4* __restrict__ downT, int row_chunks /* D*2/16 */, int M, int C,
    int32_t* status, int check) {
  int n = *count_ptr - first;  // rows of this chunk
  if (n > max_rows) n = max_rows;
  for (int r = blockIdx.x; r < n; r += gridDim.x) {
    const int slot = slots[first + r];
    size_t rec;
    if (kFromStore) {
      const int id = ids[first + r];
      if (check && (id < 0 || id >= M)) {
        if (threadIdx.x == 0) atomicOr(status, kStatBadNeuron);
        continue;
      }
      rec = (size_t)id;
    } else {
      rec = (size_t)r;
    }
    if (check && (slot < 0 || slot >= C)) {
      if (threadIdx.x == 0) atomicOr(status, kStatBadSlot);
      continue;
    }
    const uint4* s = src + rec * 3 * row_chunks;
    const size_t dst = (size_t)slot * row_chunks;
    // up to 4 loads in flight per thread per projection
    for (int c0 = threadIdx.x; c0 < row_chunks; c0 += kScatterThreads * 4) {
      uint4 g[4], u[4], d[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int c = c0 + j * kScatterThreads;
        if (c < row_chunks) {
          g[j] = ldg_stream(s + c);
          u[j] = ldg_stream(s + row_chunks + c);
          d[j] = ldg_stream(s + 2 * row_chunks + c);
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int c = c0 + j * kScatterThreads;
        if (c < row_chunks) {
          gate[dst + c] = g[j];
          up[dst + c] = u[j];
          downT[dst + c] = d[j];
        }
      }
    }
  }
}

cudaError_t launch_scatter(const Dims& d, const void* src, bool src_is_store, const int32_t* ids,
                           const int32_t* slots, const int32_t* count_ptr, int first, int max_rows,
                           void* gate_l, void* up_l, void* downT_l, int32_t* status, int check,
                           cudaStream_t s, int sm_count) {
  if (max_rows <= 0) return cudaSuccess;
  const int row_chunks = d.D * 2 / 16;
  int blocks = max_rows;
  const int cap = sm_count * 8;
  if (blocks > cap) blocks = cap;
  if (src_is_store) {
    k_deinterleave_scatter<true><<<blocks, kScatterThreads, 0, s>>>(
        static_cast<const uint4*>(src), ids, slots, count_ptr, first, max_rows, static_cast<uint4*>(gate_l),
        static_cast<uint4*>(up_l), static_cast<uint4*>(downT_l), row_chunks, d.M, d.C, status, check);
  } else {
    k_deinterleave_scatter<false><<<blocks, kScatterThreads, 0, s>>>(
        static_cast<const uint4*>(src), ids, slots, count_ptr, first, max_rows, static_cast<uint4*>(gate_l),
        static_cast<uint4*>(up_l), static_cast<uint4*>(downT_l), row_chunks, d.M, d.C, status, check);
  }
  return cudaGetLastError();
}

}  // namespace npi
