// Stage 3c: fused deinterleave + scatter (Section 3.5).  Each staged record
// holds a neuron's gate, up and transposed-down rows back to back; the kernel
// writes the three rows to the slot the delta step assigned, in the three
// projection-specific resident buffers.  Pure 16-byte coalesced copies.
//
// The same kernel serves the zero-copy transfer mode, where `src` is the whole
// layer of the pinned record store and records are addressed by neuron ID.
#include <cuda_bf16.h>

#include <algorithm>

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

// 8-bit records (int8 gate | up | downT rows, three fp32 scales, padding): the rows are
// dequantised on their way into the resident buffers, w = bf16_rn(float(q) * scale), so only
// half the bytes of a bf16 record cross PCIe or sit in staging.  A thread turns 16 bytes of one
// row into 32 bytes of bf16.
__device__ __forceinline__ uint32_t dequant2(uint32_t q4, int shift, float scale) {
  const float a = (float)(int)(signed char)((q4 >> shift) & 0xffu) * scale;
  const float b = (float)(int)(signed char)((q4 >> (shift + 8)) & 0xffu) * scale;
  const uint32_t lo = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(a));
  const uint32_t hi = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(b));
  return lo | (hi << 16);
}

template <bool kFromStore>
__global__ void __launch_bounds__(kScatterThreads) k_dequant_scatter(
    const unsigned char* __restrict__ src, const int32_t* __restrict__ ids, const int32_t* __restrict__ slots,
    const int32_t* __restrict__ count_ptr, int first, int max_rows, uint4* __restrict__ gate,
    uint4* __restrict__ up, uint4* __restrict__ downT, int D, size_t rec_bytes, int M, int C, int dst_pitch,
    int32_t* status, int check) {
  // count_ptr == NULL: exactly max_rows rows (the dense prefix is dequantised once, at start-up)
  int n = count_ptr ? *count_ptr - first : max_rows;
  if (n > max_rows) n = max_rows;
  const int q_chunks = D >> 4;  // 16-byte pieces of one int8 row
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
    const unsigned char* s = src + rec * rec_bytes;
    const float* scales = reinterpret_cast<const float*>(s + (size_t)3 * D);
    const size_t dst = (size_t)slot * dst_pitch;  // uint4 units from one slot's row to the next
    // up to four loads of a thread are issued before the first is converted
    for (int c0 = threadIdx.x; c0 < 3 * q_chunks; c0 += kScatterThreads * 4) {
      uint4 q[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int c = c0 + j * kScatterThreads;
        if (c < 3 * q_chunks) {
          const int p = c / q_chunks, cc = c - p * q_chunks;
          q[j] = ldg_stream(s + (size_t)p * D + (size_t)cc * 16);
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int c = c0 + j * kScatterThreads;
        if (c < 3 * q_chunks) {
          const int p = c / q_chunks, cc = c - p * q_chunks;
          const float scale = __ldg(scales + p);
          uint4 lo, hi;
          lo.x = dequant2(q[j].x, 0, scale);
          lo.y = dequant2(q[j].x, 16, scale);
          lo.z = dequant2(q[j].y, 0, scale);
          lo.w = dequant2(q[j].y, 16, scale);
          hi.x = dequant2(q[j].z, 0, scale);
          hi.y = dequant2(q[j].z, 16, scale);
          hi.z = dequant2(q[j].w, 0, scale);
          hi.w = dequant2(q[j].w, 16, scale);
          uint4* row = p == 0 ? gate : (p == 1 ? up : downT);
          row[dst + 2 * cc] = lo;
          row[dst + 2 * cc + 1] = hi;
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
  if (d.rec_int8) {
    if (src_is_store)
      k_dequant_scatter<true><<<blocks, kScatterThreads, 0, s>>>(
          static_cast<const unsigned char*>(src), ids, slots, count_ptr, first, max_rows, static_cast<uint4*>(gate_l),
          static_cast<uint4*>(up_l), static_cast<uint4*>(downT_l), d.D, d.rec_bytes, d.M, d.C, (d.D >> 4) * 2, status,
          check);
    else
      k_dequant_scatter<false><<<blocks, kScatterThreads, 0, s>>>(
          static_cast<const unsigned char*>(src), ids, slots, count_ptr, first, max_rows, static_cast<uint4*>(gate_l),
          static_cast<uint4*>(up_l), static_cast<uint4*>(downT_l), d.D, d.rec_bytes, d.M, d.C, (d.D >> 4) * 2, status,
          check);
    return cudaGetLastError();
  }
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

// Start-up only: the 8-bit records of one dense layer, read from the pinned store, become whole
// bf16 records [M][gate | up | downT][D] in the dense buffer (slot = neuron, rows three times
// as far apart as in a slot buffer).
cudaError_t launch_dequant_dense_layer(const Dims& d, const void* store_l, const int32_t* identity, void* dense_l,
                                       int32_t* status, cudaStream_t s, int sm_count) {
  const size_t row_bytes = (size_t)d.D * 2;
  char* base = static_cast<char*>(dense_l);
  const int blocks = std::min(d.M, sm_count * 8);
  k_dequant_scatter<true><<<blocks, kScatterThreads, 0, s>>>(
      static_cast<const unsigned char*>(store_l), identity, identity, nullptr, 0, d.M,
      reinterpret_cast<uint4*>(base), reinterpret_cast<uint4*>(base + row_bytes),
      reinterpret_cast<uint4*>(base + 2 * row_bytes), d.D, d.rec_bytes, d.M, d.M, 3 * (d.D >> 4) * 2, status, 1);
  return cudaGetLastError();
}

}  // namespace npi
