// Stage 4 over a run of consecutive layers in ONE persistent kernel (B = 1).
//
//   x_{l+1} = x_l + sum_{i in act_l} silu(gate_l[s_i].x_l) * (up_l[s_i].x_l) * downT_l[s_i]
//
// (Section 3.4: the sparse MLP reads each active row through the slot map;
// Section 3.1: the sparse suffix runs once its delta rows are in place.)
//
// A layer moves only ~27 MB at the 7B shape, a few microseconds of HBM time, so
// separate launches spend as long on launch latency and on the dependency
// between layers as on the rows.  Here one block per SM stays resident for the
// whole run of layers (cooperative launch).  Each block owns a ring of
// shared-memory stages, one 3*D*2-byte record each, filled by 1-D bulk copies;
// the rows of layer l+1 are requested as soon as a tile of layer l has been
// read, i.e. before layer l's partial sums are reduced and before the grid-wide
// barrier that publishes x_{l+1}.  The HBM pipe therefore stays busy across
// layer boundaries and the only exposed latency per layer is the barrier.
//
// Every wait (mbarrier, grid barrier) is bounded; on expiry the block records
// kStatTimeout and leaves, and the other blocks follow at their next barrier.
#include <algorithm>

#include "np_device.cuh"
#include "np_internal.h"
#include "np_pipe.cuh"

namespace npi {
using namespace npd;

constexpr int kChainThreads = 512;
constexpr int kChainWarps = kChainThreads / 32;
constexpr int kChainMaxStages = 16;
constexpr int kChainMaxLayers = 128;  // layers per launch (longer runs are split by the host)

struct ChainKernelArgs {
  const unsigned char* gate;   // layer 0 of each buffer; layer stride = C * D * 2 bytes
  const unsigned char* up;
  const unsigned char* downT;
  const int32_t* slots;        // active_slots [L][C]
  const int32_t* counters;     // [L][NP_N_COUNTERS]
  float* xbuf[2];              // x_l is stored to xbuf[l & 1]
  float* zbuf[3];              // MLP_l(x_l) accumulates into zbuf[l % 3]
  unsigned int* grid_bar;      // zeroed by the host before the launch
  int32_t* status;
  int l_begin, l_end, D, C, n_stages, tile_rows, check;
};

__device__ __forceinline__ float4 ldcg4(const float* p) {
  return __ldcg(reinterpret_cast<const float4*>(p));
}

template <int XJ, int COLS>
__global__ void __launch_bounds__(kChainThreads, 1) k_mlp_chain(ChainKernelArgs a) {
  extern __shared__ __align__(128) unsigned char csm[];
  __shared__ __align__(8) uint64_t full_bar[kChainMaxStages];
  __shared__ float part[kChainWarps][2];
  __shared__ float act[kChainWarps];
  __shared__ int s_ok;
  __shared__ int lay_rb[kChainMaxLayers];       // first active-list index of this block, per layer
  __shared__ int lay_pre[kChainMaxLayers + 1];  // rows of this block before each layer (virtual row index)

  const int D = a.D, chunks = D >> 3;
  const uint32_t row_bytes = (uint32_t)D * 2u;
  const uint32_t rec_bytes = 3u * row_bytes;
  const size_t layer_bytes = (size_t)a.C * row_bytes;
  const int n_stages = a.n_stages, TR = a.tile_rows, SEG = kChainWarps / TR;
  const int seg_chunks = (chunks + SEG - 1) / SEG;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int G = gridDim.x, nl = a.l_end - a.l_begin;

  // ---- this block's share of every layer of the run ----
  if (tid < nl) {
    int n = a.counters[(size_t)(a.l_begin + tid) * NP_N_COUNTERS + NP_CNT_ACTIVE];
    if (a.check && (n < 0 || n > a.C)) {
      atomicOr(a.status, kStatBadCount);
      n = 0;
    }
    const int rb = (int)(((long long)n * blockIdx.x) / G);
    const int re = (int)(((long long)n * (blockIdx.x + 1)) / G);
    lay_rb[tid] = rb;
    lay_pre[tid + 1] = re - rb;  // turned into a prefix sum below
  }
  if (tid == 0) {
    for (int s = 0; s < n_stages; ++s) npp::mbar_init(&full_bar[s], 1);
    npp::fence_barrier_init();
    s_ok = 1;
  }
  __syncthreads();
  if (tid == 0) {
    lay_pre[0] = 0;
    for (int i = 0; i < nl; ++i) lay_pre[i + 1] += lay_pre[i];
  }
  __syncthreads();
  const int total_rows = lay_pre[nl];

  // ---- producer state (used by warp 0 only; identical in all its lanes) ----
  int issued = 0;    // virtual rows requested so far
  int consumed = 0;  // virtual rows whose stage has been read completely
  int issue_layer = 0;
  auto issue_more = [&]() {  // warp 0, all lanes
    const int limit = min(total_rows, consumed + n_stages);
    while (issued < limit) {
      const int v = issued + lane;
      if (v < limit) {
        int ll = issue_layer;
        while (v >= lay_pre[ll + 1]) ++ll;
        const int i = v - lay_pre[ll];
        int slot = a.slots[(size_t)(a.l_begin + ll) * a.C + lay_rb[ll] + i];
        if (a.check && (slot < 0 || slot >= a.C)) {
          atomicOr(a.status, kStatBadSlot);
          slot = 0;
        }
        const int s = v % n_stages;
        unsigned char* dst = csm + (size_t)s * rec_bytes;
        const size_t off = (size_t)(a.l_begin + ll) * layer_bytes + (size_t)slot * row_bytes;
        npp::mbar_expect_tx(&full_bar[s], rec_bytes);
        npp::bulk_g2s(dst, a.gate + off, row_bytes, &full_bar[s]);
        npp::bulk_g2s(dst + row_bytes, a.up + off, row_bytes, &full_bar[s]);
        npp::bulk_g2s(dst + 2 * row_bytes, a.downT + off, row_bytes, &full_bar[s]);
      }
      issued = min(limit, issued + 32);
    }
    while (issue_layer < nl && issued >= lay_pre[issue_layer + 1]) ++issue_layer;
    if (issue_layer >= nl) issue_layer = nl - 1;
  };
  if (wid == 0) issue_more();

  const int sg = wid % SEG, row_in_tile = wid / SEG;
  const int c_lo = sg * seg_chunks, c_hi = min(chunks, c_lo + seg_chunks);

  for (int li = 0; li < nl; ++li) {
    const int l = a.l_begin + li;
    // ---- wait until every block has added its part of layer l-1 (x_l is final) ----
    if (li > 0) {
      if (tid == 0) {
        const unsigned int target = (unsigned int)li * (unsigned int)G;
        bool ok = false;
        for (uint32_t spin = 0; spin < npp::kSpinLimit; ++spin) {
          unsigned int v;
          asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(a.grid_bar) : "memory");
          if (v >= target) {
            ok = true;
            break;
          }
        }
        if (!ok) {
          atomicOr(a.status, npp::kStatTimeout);
          s_ok = 0;
        }
      }
      __syncthreads();
      if (!s_ok) break;
    }

    // ---- x_l = xbuf[(l+1)&1] + zbuf[(l-1)%3]: this warp's slice, in registers ----
    const float* xa = a.xbuf[(l + 1) & 1];
    const float* xb = l > 0 ? a.zbuf[(l - 1) % 3] : nullptr;
    float xr[XJ][8];
#pragma unroll
    for (int j = 0; j < XJ; ++j) {
      const int c = c_lo + lane + 32 * j;
      if (c < c_hi) {
        float4 v0 = ldcg4(xa + (size_t)c * 8), v1 = ldcg4(xa + (size_t)c * 8 + 4);
        if (xb) {
          const float4 w0 = ldcg4(xb + (size_t)c * 8), w1 = ldcg4(xb + (size_t)c * 8 + 4);
          v0.x += w0.x; v0.y += w0.y; v0.z += w0.z; v0.w += w0.w;
          v1.x += w1.x; v1.y += w1.y; v1.z += w1.z; v1.w += w1.w;
        }
        xr[j][0] = v0.x; xr[j][1] = v0.y; xr[j][2] = v0.z; xr[j][3] = v0.w;
        xr[j][4] = v1.x; xr[j][5] = v1.y; xr[j][6] = v1.z; xr[j][7] = v1.w;
        if (blockIdx.x == 0 && row_in_tile == 0) {  // one warp per segment: store x_l, clear the next accumulator
          float4* ps = reinterpret_cast<float4*>(a.xbuf[l & 1] + (size_t)c * 8);
          ps[0] = v0;
          ps[1] = v1;
          float4* pz = reinterpret_cast<float4*>(a.zbuf[(l + 1) % 3] + (size_t)c * 8);
          pz[0] = make_float4(0.f, 0.f, 0.f, 0.f);
          pz[1] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) xr[j][e] = 0.f;
      }
    }

    float acc[COLS][8];
#pragma unroll
    for (int j = 0; j < COLS; ++j)
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[j][e] = 0.f;

    const int vbase = lay_pre[li], nrows = lay_pre[li + 1] - vbase;
    for (int t0 = 0; t0 < nrows; t0 += TR) {
      const int rows = min(TR, nrows - t0);
      // ---- phase 1: (row, segment) partial dot products from shared memory ----
      if (row_in_tile < rows) {
        const int v = vbase + t0 + row_in_tile;
        const int s = v % n_stages;
        if (!npp::mbar_wait(&full_bar[s], (uint32_t)(v / n_stages) & 1u)) {
          if (lane == 0) {
            atomicOr(a.status, npp::kStatTimeout);
            s_ok = 0;
          }
        }
        const uint4* gp = reinterpret_cast<const uint4*>(csm + (size_t)s * rec_bytes);
        const uint4* up = gp + chunks;
        float g = 0.f, u = 0.f;
#pragma unroll
        for (int j = 0; j < XJ; ++j) {
          const int c = c_lo + lane + 32 * j;
          if (c < c_hi) {
            const uint4 gw = gp[c], uw = up[c];
            const float4 x0 = make_float4(xr[j][0], xr[j][1], xr[j][2], xr[j][3]);
            const float4 x1 = make_float4(xr[j][4], xr[j][5], xr[j][6], xr[j][7]);
            g = dot8(gw, x0, x1, g);
            u = dot8(uw, x0, x1, u);
          }
        }
        g = warp_sum(g);
        u = warp_sum(u);
        if (lane == 0) {
          part[wid][0] = g;
          part[wid][1] = u;
        }
      }
      __syncthreads();
      if (!s_ok) break;
      if (tid < rows) {
        float gs = 0.f, us = 0.f;
        for (int q = 0; q < SEG; ++q) {
          gs += part[tid * SEG + q][0];
          us += part[tid * SEG + q][1];
        }
        act[tid] = gs / (1.f + __expf(-gs)) * us;
      }
      __syncthreads();
      // ---- phase 2: y[cols] += a_i * downT[s_i][cols] ----
#pragma unroll
      for (int j = 0; j < COLS; ++j) {
        const int c = tid + j * kChainThreads;
        if (c < chunks) {
          for (int q = 0; q < rows; ++q) {
            const int s = (vbase + t0 + q) % n_stages;
            const uint4 w = reinterpret_cast<const uint4*>(csm + (size_t)s * rec_bytes + 2 * row_bytes)[c];
            const float av = act[q];
            acc[j][0] = fmaf(av, bf16_lo(w.x), acc[j][0]);
            acc[j][1] = fmaf(av, bf16_hi(w.x), acc[j][1]);
            acc[j][2] = fmaf(av, bf16_lo(w.y), acc[j][2]);
            acc[j][3] = fmaf(av, bf16_hi(w.y), acc[j][3]);
            acc[j][4] = fmaf(av, bf16_lo(w.z), acc[j][4]);
            acc[j][5] = fmaf(av, bf16_hi(w.z), acc[j][5]);
            acc[j][6] = fmaf(av, bf16_lo(w.w), acc[j][6]);
            acc[j][7] = fmaf(av, bf16_hi(w.w), acc[j][7]);
          }
        }
      }
      __syncthreads();  // the tile's stages have been read: request the rows that come next,
      consumed += rows; // possibly those of the following layers
      if (wid == 0) issue_more();
    }
    if (!s_ok) break;

    // ---- add this block's partial MLP_l(x_l) to the layer's accumulator ----
    if (nrows > 0) {
      float* yacc = a.zbuf[l % 3];
#pragma unroll
      for (int j = 0; j < COLS; ++j) {
        const int c = tid + j * kChainThreads;
        if (c < chunks) {
          float4* yp = reinterpret_cast<float4*>(yacc + (size_t)c * 8);
          atomicAdd(yp, make_float4(acc[j][0], acc[j][1], acc[j][2], acc[j][3]));
          atomicAdd(yp + 1, make_float4(acc[j][4], acc[j][5], acc[j][6], acc[j][7]));
        }
      }
    }
    if (li + 1 < nl) {  // publish: every thread's adds and stores precede the arrival
      __syncthreads();
      if (tid == 0) {
        __threadfence();
        atomicAdd(a.grid_bar, 1u);
      }
    }
  }
}

template <int XJ, int COLS>
static cudaError_t chain_launch(const ChainKernelArgs& ka, size_t sm, int grid_x, cudaStream_t s) {
  auto kfn = k_mlp_chain<XJ, COLS>;
  cudaError_t e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
  if (e != cudaSuccess) return e;
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kfn, kChainThreads, sm);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorCooperativeLaunchTooLarge;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid_x);
  cfg.blockDim = dim3(kChainThreads);
  cfg.dynamicSmemBytes = sm;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;  // all blocks co-resident: the grid barrier cannot starve
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kfn, ka);
}

bool mlp_chain_supported(const Dims& d, int sm_count) {
  ChainPlan p;
  return mlp_chain_plan(d, sm_count, &p);
}

bool mlp_chain_plan(const Dims& d, int sm_count, ChainPlan* p) {
  const int chunks = d.D >> 3;
  const size_t rec = (size_t)d.D * 6;
  const size_t budget = 200 * 1024;
  int n_stages = (int)std::min<size_t>(kChainMaxStages, budget / rec);
  if (n_stages < 2) return false;
  const long long expect = std::min<long long>(d.C, d.k);
  const int per_block = (int)std::max<long long>(1, (expect + sm_count - 1) / sm_count);
  int tr = 1;
  const int tr_cap = std::max(1, std::min(per_block, n_stages) / 2);
  while (tr * 2 <= tr_cap && tr * 2 <= kChainWarps) tr *= 2;
  while (tr < kChainWarps && chunks / (kChainWarps / tr) < 32) tr *= 2;
  if (tr > n_stages) return false;
  const int seg = kChainWarps / tr;
  const int seg_chunks = (chunks + seg - 1) / seg;
  p->xj = (seg_chunks + 31) / 32;
  const int need_cols = (chunks + kChainThreads - 1) / kChainThreads;
  if (p->xj > 8 || need_cols > 4) return false;
  p->cols = need_cols <= 1 ? 1 : (need_cols <= 2 ? 2 : 4);
  p->n_stages = n_stages;
  p->tile_rows = tr;
  p->smem = (size_t)n_stages * rec;
  return true;
}

cudaError_t launch_mlp_chain(const Dims& d, const ChainArgs& a, cudaStream_t s, int sm_count) {
  ChainPlan p;
  if (!mlp_chain_plan(d, sm_count, &p)) return cudaErrorInvalidValue;
  cudaError_t e = cudaSuccess;
  for (int l0 = a.l_begin; l0 < a.l_end; l0 += kChainMaxLayers) {
    ChainKernelArgs ka;
    ka.gate = static_cast<const unsigned char*>(a.gate);
    ka.up = static_cast<const unsigned char*>(a.up);
    ka.downT = static_cast<const unsigned char*>(a.downT);
    ka.slots = a.active_slots;
    ka.counters = a.counters;
    for (int i = 0; i < 2; ++i) ka.xbuf[i] = a.xbuf[i];
    for (int i = 0; i < 3; ++i) ka.zbuf[i] = a.zbuf[i];
    ka.grid_bar = a.grid_bar;
    ka.status = a.status;
    ka.l_begin = l0;
    ka.l_end = std::min(a.l_end, l0 + kChainMaxLayers);
    ka.D = d.D;
    ka.C = d.C;
    ka.n_stages = p.n_stages;
    ka.tile_rows = p.tile_rows;
    ka.check = a.check;
    e = cudaMemsetAsync(a.grid_bar, 0, sizeof(unsigned int), s);
    if (e != cudaSuccess) return e;
#define NP_CHAIN(XJV)                                                        \
  do {                                                                       \
    if (p.cols == 1) e = chain_launch<XJV, 1>(ka, p.smem, sm_count, s);      \
    else if (p.cols == 2) e = chain_launch<XJV, 2>(ka, p.smem, sm_count, s); \
    else e = chain_launch<XJV, 4>(ka, p.smem, sm_count, s);                  \
  } while (0)
    switch (p.xj) {
      case 1: NP_CHAIN(1); break;
      case 2: NP_CHAIN(2); break;
      case 3: NP_CHAIN(3); break;
      case 4: NP_CHAIN(4); break;
      case 5: NP_CHAIN(5); break;
      case 6: NP_CHAIN(6); break;
      default: NP_CHAIN(8); break;
    }
#undef NP_CHAIN
    if (e != cudaSuccess) return e;
  }
  return e;
}

}  // namespace npi
