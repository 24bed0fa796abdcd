// Stage 4: sparse SwiGLU MLP over the active resident rows, through the slot map
// (Section 3.4: for each active neuron i the runtime uses row i of the gate, up
// and transposed-down projections, located by S).
//
//   y[b] = sum_{i in act} silu(gate[s_i] . x[b]) * (up[s_i] . x[b]) * downT[s_i]
//
// Every active row is read exactly once (3 * D bf16), so the kernel is a
// bandwidth problem: a persistent grid of one block per SM, each block owning a
// contiguous share of the active list.  Phase 1 streams the gate and up rows
// (a warp per row segment, 16-byte loads, x in shared memory) and leaves the
// activations a_i in shared memory; phase 2 streams the down rows with each
// thread owning 8 output columns in registers; the per-block partial y is added
// to the output with vector floating-point atomics.
#include <algorithm>

#include "np_device.cuh"
#include "np_internal.h"

namespace npi {
using namespace npd;

constexpr int kMlpThreads = 512;
constexpr int kMlpWarps = kMlpThreads / 32;
constexpr int kTileRows = 16;  // active rows handled per phase-1/phase-2 round
constexpr int kMaxSeg = 16;    // a row can be split over up to this many warps

struct MlpKernelArgs {
  const uint4* gate;
  const uint4* up;
  const uint4* downT;
  const int32_t* slots;
  const int32_t* n_ptr;
  const float* xa;
  const float* xb;
  float* yacc;
  float* x_store;
  float* zero_out;
  int32_t* status;
  int B, D, C, seg, check;
};

template <int NB, int kMaxCols>  // kMaxCols: column rounds per thread, D <= 8 * kMlpThreads * kMaxCols
__global__ void __launch_bounds__(kMlpThreads, 1) k_sparse_mlp(MlpKernelArgs a) {
  extern __shared__ __align__(16) float msm[];
  const int D = a.D, chunks = D >> 3;
  float* xs = msm;                                   // [NB][D]
  float* part = xs + (size_t)NB * D;                 // [NB][kTileRows][kMaxSeg][2]
  float* act = part + NB * kTileRows * kMaxSeg * 2;  // [NB][kTileRows]
  __shared__ int s_slot[kTileRows];

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int b0 = blockIdx.y * NB;  // first sequence of this batch group
  const int nb = min(NB, a.B - b0);

  // x = xa (+ xb) into shared memory; block 0 of the group keeps the chain's side effects
  for (int i = tid; i < nb * D; i += kMlpThreads) {
    const size_t gi = (size_t)b0 * D + i;
    float v = a.xa[gi];
    if (a.xb) v += a.xb[gi];
    xs[i] = v;
    if (blockIdx.x == 0) {
      if (a.x_store) a.x_store[gi] = v;
      if (a.zero_out) a.zero_out[gi] = 0.f;
    }
  }

  int n = *a.n_ptr;
  if (a.check && (n < 0 || n > a.C)) {
    if (tid == 0) atomicOr(a.status, kStatBadCount);
    n = 0;
  }
  const int G = gridDim.x;
  const int r_begin = (int)(((long long)n * blockIdx.x) / G);
  const int r_end = (int)(((long long)n * (blockIdx.x + 1)) / G);
  const int seg = a.seg;                       // warps per row in phase 1
  const int seg_chunks = (chunks + seg - 1) / seg;

  float acc[NB][kMaxCols][8];
#pragma unroll
  for (int b = 0; b < NB; ++b)
#pragma unroll
    for (int j = 0; j < kMaxCols; ++j)
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[b][j][e] = 0.f;
  __syncthreads();

  for (int t0 = r_begin; t0 < r_end; t0 += kTileRows) {
    const int rows = min(kTileRows, r_end - t0);
    if (tid < rows) {
      int s = a.slots[t0 + tid];
      if (a.check && (s < 0 || s >= a.C)) {
        atomicOr(a.status, kStatBadSlot);
        s = 0;
      }
      s_slot[tid] = s;
    }
    __syncthreads();

    // ---- phase 1: g_i = gate[s_i].x, u_i = up[s_i].x ; work item = (row, segment) ----
    for (int item = wid; item < rows * seg; item += kMlpWarps) {
      const int i = item / seg, sg = item - i * seg;
      const size_t rbase = (size_t)s_slot[i] * chunks;
      const int c_lo = sg * seg_chunks, c_hi = min(chunks, c_lo + seg_chunks);
      float g[NB], u[NB];
#pragma unroll
      for (int b = 0; b < NB; ++b) g[b] = u[b] = 0.f;
      for (int c0 = c_lo + lane; c0 < c_hi; c0 += 32 * 8) {
        uint4 gw[8], uw[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int c = c0 + 32 * j;
          if (c < c_hi) {
            gw[j] = ldg_stream(a.gate + rbase + c);
            uw[j] = ldg_stream(a.up + rbase + c);
          }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int c = c0 + 32 * j;
          if (c < c_hi) {
#pragma unroll
            for (int b = 0; b < NB; ++b) {
              const float4* xp = reinterpret_cast<const float4*>(xs + (size_t)b * D + c * 8);
              const float4 x0 = xp[0], x1 = xp[1];
              g[b] = dot8(gw[j], x0, x1, g[b]);
              u[b] = dot8(uw[j], x0, x1, u[b]);
            }
          }
        }
      }
#pragma unroll
      for (int b = 0; b < NB; ++b) {
        const float gs = warp_sum(g[b]), us = warp_sum(u[b]);
        if (lane == 0) {
          float* pp = part + (((size_t)b * kTileRows + i) * kMaxSeg + sg) * 2;
          pp[0] = gs;
          pp[1] = us;
        }
      }
    }
    __syncthreads();
    if (tid < rows * NB) {
      const int b = tid / rows, i = tid - b * rows;
      float gs = 0.f, us = 0.f;
      for (int sg = 0; sg < seg; ++sg) {
        const float* pp = part + (((size_t)b * kTileRows + i) * kMaxSeg + sg) * 2;
        gs += pp[0];
        us += pp[1];
      }
      act[b * kTileRows + i] = gs / (1.f + __expf(-gs)) * us;
    }
    __syncthreads();

    // ---- phase 2: y[:, cols] += a_i * downT[s_i][cols]; thread owns 8 columns per round ----
#pragma unroll
    for (int j = 0; j < kMaxCols; ++j) {
      const int c = tid + j * kMlpThreads;
      if (c < chunks) {
        for (int i0 = 0; i0 < rows; i0 += 8) {
          uint4 w[8];
#pragma unroll
          for (int q = 0; q < 8; ++q)
            if (i0 + q < rows) w[q] = ldg_stream(a.downT + (size_t)s_slot[i0 + q] * chunks + c);
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            if (i0 + q < rows) {
#pragma unroll
              for (int b = 0; b < NB; ++b) {
                const float av = act[b * kTileRows + i0 + q];
                acc[b][j][0] = fmaf(av, bf16_lo(w[q].x), acc[b][j][0]);
                acc[b][j][1] = fmaf(av, bf16_hi(w[q].x), acc[b][j][1]);
                acc[b][j][2] = fmaf(av, bf16_lo(w[q].y), acc[b][j][2]);
                acc[b][j][3] = fmaf(av, bf16_hi(w[q].y), acc[b][j][3]);
                acc[b][j][4] = fmaf(av, bf16_lo(w[q].z), acc[b][j][4]);
                acc[b][j][5] = fmaf(av, bf16_hi(w[q].z), acc[b][j][5]);
                acc[b][j][6] = fmaf(av, bf16_lo(w[q].w), acc[b][j][6]);
                acc[b][j][7] = fmaf(av, bf16_hi(w[q].w), acc[b][j][7]);
              }
            }
          }
        }
      }
    }
    __syncthreads();  // s_slot / act are rewritten by the next round
  }

  if (r_end > r_begin) {
#pragma unroll
    for (int j = 0; j < kMaxCols; ++j) {
      const int c = tid + j * kMlpThreads;
      if (c < chunks) {
#pragma unroll
        for (int b = 0; b < NB; ++b) {
          if (b < nb) {
            float4* yp = reinterpret_cast<float4*>(a.yacc + (size_t)(b0 + b) * D + (size_t)c * 8);
            atomicAdd(yp, make_float4(acc[b][j][0], acc[b][j][1], acc[b][j][2], acc[b][j][3]));
            atomicAdd(yp + 1, make_float4(acc[b][j][4], acc[b][j][5], acc[b][j][6], acc[b][j][7]));
          }
        }
      }
    }
  }
}

template <int NB, int COLS>
static cudaError_t mlp_launch_cols(const MlpKernelArgs& ka, int groups, int grid_x, cudaStream_t s) {
  const size_t sm = ((size_t)NB * ka.D + (size_t)NB * kTileRows * kMaxSeg * 2 + NB * kTileRows) * 4;
  auto kfn = k_sparse_mlp<NB, COLS>;
  static size_t configured = 0;
  if (sm > 48 * 1024 && sm > configured) {
    cudaError_t e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (e != cudaSuccess) return e;
    configured = sm;
  }
  dim3 grid(grid_x, groups);
  kfn<<<grid, kMlpThreads, sm, s>>>(ka);
  return cudaGetLastError();
}

template <int NB>
static cudaError_t mlp_launch_nb(const MlpKernelArgs& ka, int groups, int grid_x, cudaStream_t s) {
  const int rounds = ((ka.D >> 3) + kMlpThreads - 1) / kMlpThreads;
  if (rounds <= 1) return mlp_launch_cols<NB, 1>(ka, groups, grid_x, s);
  if (rounds <= 2) return mlp_launch_cols<NB, 2>(ka, groups, grid_x, s);
  if (rounds <= 4) return mlp_launch_cols<NB, 4>(ka, groups, grid_x, s);
  return cudaErrorInvalidValue;  // D > 16384 is rejected by np_init
}

cudaError_t launch_sparse_mlp(const Dims& d, const MlpArgs& a, cudaStream_t s, int sm_count) {
  MlpKernelArgs ka;
  ka.gate = static_cast<const uint4*>(a.gate_l);
  ka.up = static_cast<const uint4*>(a.up_l);
  ka.downT = static_cast<const uint4*>(a.downT_l);
  ka.slots = a.active_slots;
  ka.n_ptr = a.n_active_ptr;
  ka.xa = a.xa;
  ka.xb = a.xb;
  ka.yacc = a.yacc;
  ka.x_store = a.x_store;
  ka.zero_out = a.zero_out;
  ka.status = a.status;
  ka.B = a.B;
  ka.D = d.D;
  ka.C = a.C;
  ka.check = a.check;
  // warps per row in phase 1: spread the block's expected share of rows over its warps,
  // but keep at least one 16-byte chunk per lane in a segment
  const int chunks = d.D >> 3;
  const long long expect = std::min<long long>(d.C, (long long)d.k * a.B);
  const int per_block = (int)std::max<long long>(1, (expect + sm_count - 1) / sm_count);
  int seg = 1;
  while (seg * 2 <= kMaxSeg && per_block * seg * 2 <= kMlpWarps && chunks / (seg * 2) >= 32) seg *= 2;
  ka.seg = seg;
  if (a.B == 1) return mlp_launch_nb<1>(ka, 1, sm_count, s);
  if (a.B == 2) return mlp_launch_nb<2>(ka, 1, sm_count, s);
  return mlp_launch_nb<4>(ka, (a.B + 3) / 4, sm_count, s);
}

}  // namespace npi
