// Stage 4 over a run of layers in one resident kernel, rows dealt whole to the blocks (B = 1).
//
//   x_{l+1} = x_l + sum_{i in act_l} silu(gate_l[s_i].n_l) * (up_l[s_i].n_l) * downT_l[s_i],
//   n_l = x_l / sqrt(mean(x_l^2) + 1e-6)
//
// (Section 3.4: the sparse MLP reads each active row through the slot map.)  One block per SM
// stays resident over the run (cooperative launch); every block owns a share of a layer's
// active rows and a ring of shared-memory stages of one record each, filled by 1-D bulk copies
// from a producer lane; the gate/up dot products run on the ALUs with a (row, segment) item per
// warp and x_l in shared memory as fp32; every block adds its partial vector of all D outputs to
// one of kZRep accumulator copies and a grid-wide counter barrier publishes x_{l+1}.
// It takes any row width, and is what runs where the column-sliced kernel (np_mlp_slices.cu)
// does not apply: row widths that are not a multiple of 64, dense layers without the
// direct-load kernel, and NP_F_ROW_CHAIN.  Every wait is bounded (kStatTimeout on expiry).
#include <algorithm>

#include "np_device.cuh"
#include "np_internal.h"
#include "np_pipe.cuh"

namespace npi {
namespace chain_alu {
using namespace npd;

constexpr int kChainWarps = 16;                      // consumer warps
constexpr int kChainThreads = kChainWarps * 32;      // consumer threads
constexpr int kChainBlock = kChainThreads + 32;      // plus one producer warp
constexpr int kChainMaxStages = 16;
constexpr int kChainMaxRpw = 2;   // rows a warp may take per tile in phase 1
constexpr int kChainMaxLayers = 128;  // layers per launch (longer runs are split by the host)

struct AluPlan {
  int n_stages, tile_rows, rows_per_warp, xj, cols;
  int run_layers, slot_cache_rows, window_rows;
  size_t smem;
};

struct ChainKernelArgs {
  const unsigned char* gate;   // layer 0 of each buffer; layer stride = C * D * 2 bytes
  const unsigned char* up;
  const unsigned char* downT;
  const int32_t* slots;        // active_slots [L][C]
  const int32_t* counters;     // [L][NP_N_COUNTERS]
  float* xbuf[2];              // x_l is stored to xbuf[l & 1]
  float* zbuf[3];              // MLP_l(x_l) accumulates into zbuf[l % 3]: kZRep copies of [D], block g adds
                               // into copy g % kZRep (fewer adds per address), readers sum the copies
  unsigned int* grid_bar;      // zeroed by the host before the launch
  int32_t* status;
  int l_begin, l_end, D, C, n_stages, tile_rows, rows_per_warp, check;
  int dense_rows;              // > 0: dense layers.  Each layer is dense_rows whole records ([row][gate|up|down][D],
                               // `gate` points at layer 0's first record), every row is active, `slots` is one
                               // identity list shared by all layers and `counters` is not read
  int slot_cache_rows;         // capacity of the per-block slot cache (rows)
  int window_rows;             // records in flight per block (< n_stages)
};

__device__ __forceinline__ float4 ldcg4(const float* p) {
  return __ldcg(reinterpret_cast<const float4*>(p));
}

// barrier among the consumer warps only (the producer warp never joins it)
__device__ __forceinline__ void consumer_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(kChainWarps * 32) : "memory");
}

// 16-byte floating-point reduction to global memory, no return value
__device__ __forceinline__ void red_add_v4(float* p, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d)
               : "memory");
}

template <int XJ, int COLS>
__global__ void __launch_bounds__(kChainBlock, 1) k_mlp_chain(ChainKernelArgs a) {
  extern __shared__ __align__(128) unsigned char csm[];
  __shared__ __align__(8) uint64_t full_bar[kChainMaxStages];   // a stage's record has landed
  __shared__ __align__(8) uint64_t empty_bar[kChainMaxStages];  // every consumer warp is done with it
  __shared__ float part[kChainMaxRpw * kChainWarps][2];  // (g, u) partial sums of the tile's (row, segment) items
  __shared__ float act[kChainMaxRpw * kChainWarps];      // a_i of the tile's rows
  __shared__ float ssq_part[kChainWarps];       // per-warp sums of x_l^2 (for the RMS normalisation)
  __shared__ int s_ok;
  __shared__ int lay_rb[kChainMaxLayers];       // first active-list index of this block, per layer
  __shared__ int lay_pre[kChainMaxLayers + 1];  // rows of this block before each layer (virtual row index)

  const int D = a.D, chunks = D >> 3;
  const uint32_t row_bytes = (uint32_t)D * 2u;
  const uint32_t rec_bytes = 3u * row_bytes;
  // resident slot buffers: one row per slot and projection; dense layers: whole records
  const int cap = a.dense_rows > 0 ? a.dense_rows : a.C;               // rows a layer can hold
  const uint32_t row_pitch = a.dense_rows > 0 ? rec_bytes : row_bytes;  // bytes from one row to the next
  const size_t layer_bytes = (size_t)cap * row_pitch;
  // a tile is TR = RPW * (16 / SEG) rows: phase 1 gives every warp RPW (row, segment) items
  const int n_stages = a.n_stages, RPW = a.rows_per_warp, TR = a.tile_rows, SEG = kChainWarps * RPW / TR;
  const int seg_chunks = (chunks + SEG - 1) / SEG;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int G = gridDim.x, nl = a.l_end - a.l_begin;
  float* xs = reinterpret_cast<float*>(csm + (size_t)n_stages * rec_bytes);  // x_l, fp32 [D], kept across layers
  int* slot_cache = reinterpret_cast<int*>(xs + D);                         // this block's slots, virtual row order

  // ---- this block's share of every layer of the run ----
  if (tid < nl) {
    int n = a.dense_rows > 0 ? a.dense_rows : a.counters[(size_t)(a.l_begin + tid) * NP_N_COUNTERS + NP_CNT_ACTIVE];
    if (a.check && (n < 0 || n > cap)) {
      atomicOr(a.status, kStatBadCount);
      n = 0;
    }
    const int rb = (int)(((long long)n * blockIdx.x) / G);
    const int re = (int)(((long long)n * (blockIdx.x + 1)) / G);
    lay_rb[tid] = rb;
    lay_pre[tid + 1] = re - rb;  // turned into a prefix sum below
  }
  if (tid == 0) {
    for (int s = 0; s < n_stages; ++s) {
      npp::mbar_init(&full_bar[s], 1);
      npp::mbar_init(&empty_bar[s], kChainWarps);
    }
    npp::fence_barrier_init();
    s_ok = 1;
  }
  __syncthreads();
  if (tid == 0) {
    lay_pre[0] = 0;
    for (int i = 0; i < nl; ++i) lay_pre[i + 1] += lay_pre[i];
  }
  __syncthreads();
  const int total_rows = min(lay_pre[nl], a.slot_cache_rows);
  // slots of all this block's rows, so that no request waits on a global load later
  for (int li = 0; li < nl; ++li) {
    const int nr = lay_pre[li + 1] - lay_pre[li];
    for (int i = tid; i < nr; i += blockDim.x) {
      const int v = lay_pre[li] + i;
      if (v < total_rows) {
        int slot = a.slots[(a.dense_rows > 0 ? 0 : (size_t)(a.l_begin + li) * a.C) + lay_rb[li] + i];
        if (a.check && (slot < 0 || slot >= cap)) {
          atomicOr(a.status, kStatBadSlot);
          slot = 0;
        }
        slot_cache[v] = slot;
      }
    }
  }
  __syncthreads();

  if (wid == kChainWarps) {
    // =========================== producer warp ===========================
    // One lane requests the block's virtual rows strictly in order: rows are consumed in
    // order, so stage v % n_stages is always the next one to be released.  (Lanes that wait
    // on different barriers must not be used here: the compiler may reconverge the warp
    // after the wait, and a lane whose stage is free would then be held back by a lane whose
    // stage is released only after the first lane's row has been consumed.)
    if (lane == 0) {
      int ll = 0, s = 0;
      uint32_t use = 0;
      const int window = a.window_rows;
      for (int v = 0; v < total_rows; ++v) {
        // pacing: at most `window` records in flight per block.  A deeper burst moves no more
        // bytes (HBM is shared by all blocks) but queues in front of the short loads on the
        // layer's critical path (barrier counter, accumulator vectors).
        if (v >= window) {
          const int vv = v - window;
          if (!npp::mbar_wait(&full_bar[vv % n_stages], (uint32_t)(vv / n_stages) & 1u)) {
            atomicOr(a.status, npp::kStatTimeout);
            break;
          }
        }
        if (!npp::mbar_wait(&empty_bar[s], (use & 1u) ^ 1u)) {
          atomicOr(a.status, npp::kStatTimeout);
          break;
        }
        while (v >= lay_pre[ll + 1]) ++ll;
        const size_t off = (size_t)(a.l_begin + ll) * layer_bytes + (size_t)slot_cache[v] * row_pitch;
        unsigned char* dst = csm + (size_t)s * rec_bytes;
        npp::mbar_expect_tx(&full_bar[s], rec_bytes);
        const uint64_t pol = npp::policy_evict_first();  // weight rows are read once per token
        npp::bulk_g2s_stream(dst, a.gate + off, row_bytes, &full_bar[s], pol);
        npp::bulk_g2s_stream(dst + row_bytes, a.up + off, row_bytes, &full_bar[s], pol);
        npp::bulk_g2s_stream(dst + 2 * row_bytes, a.downT + off, row_bytes, &full_bar[s], pol);
        if (++s == n_stages) {
          s = 0;
          ++use;
        }
      }
    }
    return;
  }

  // =========================== consumer warps ===========================
  const int sg = wid % SEG, row_in_tile = wid / SEG;
  const int c_lo = sg * seg_chunks, c_hi = min(chunks, c_lo + seg_chunks);
  const int l_last = a.l_end - 1;

  for (int li = 0; li < nl; ++li) {
    const int l = a.l_begin + li;
    // ---- wait until every block has added its part of layer l-1 ----
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
      consumer_sync();
      if (!s_ok) break;
    }
    // ---- x_l: first layer of the run from global, afterwards x_l = x_{l-1} + MLP_{l-1} ----
    {
      const float* xa = a.xbuf[(l + 1) & 1];
      const float* zb = l > 0 ? a.zbuf[(l - 1) % 3] : nullptr;
      float* xst = a.xbuf[l & 1];
      const int nf4 = chunks * 2;  // float4 granules of one vector
      float ssq = 0.f;
      for (int c0 = tid; c0 < nf4; c0 += 2 * kChainThreads) {
        // all loads of two granules (and of every accumulator copy) are issued before any is used
        const int c1 = c0 + kChainThreads;
        const bool has1 = c1 < nf4;
        float4 w0[kZRep], w1[kZRep];
        if (zb) {
#pragma unroll
          for (int r = 0; r < kZRep; ++r) {
            w0[r] = ldcg4(zb + (size_t)r * D + (size_t)c0 * 4);
            w1[r] = has1 ? ldcg4(zb + (size_t)r * D + (size_t)c1 * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
          }
        }
        float4 v0, v1 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (li == 0) {
          v0 = ldcg4(xa + (size_t)c0 * 4);
          if (has1) v1 = ldcg4(xa + (size_t)c1 * 4);
        } else {
          v0 = reinterpret_cast<float4*>(xs)[c0];
          if (has1) v1 = reinterpret_cast<float4*>(xs)[c1];
        }
        if (zb) {
#pragma unroll
          for (int r = 0; r < kZRep; ++r) {
            v0.x += w0[r].x; v0.y += w0[r].y; v0.z += w0[r].z; v0.w += w0[r].w;
            v1.x += w1[r].x; v1.y += w1[r].y; v1.z += w1[r].z; v1.w += w1[r].w;
          }
        }
        reinterpret_cast<float4*>(xs)[c0] = v0;
        if (has1) reinterpret_cast<float4*>(xs)[c1] = v1;
        ssq += v0.x * v0.x + v0.y * v0.y + v0.z * v0.z + v0.w * v0.w;
        ssq += v1.x * v1.x + v1.y * v1.y + v1.z * v1.z + v1.w * v1.w;  // zeros when there is no second granule
        if (blockIdx.x == 0 && l == l_last) {  // x for the next launch
          reinterpret_cast<float4*>(xst)[c0] = v0;
          if (has1) reinterpret_cast<float4*>(xst)[c1] = v1;
        }
      }
      ssq = warp_sum(ssq);
      if (lane == 0) ssq_part[wid] = ssq;
      // clear the next layer's accumulator copies: every block takes a slice
      float4* znext = reinterpret_cast<float4*>(a.zbuf[(l + 1) % 3]);
      const int ztotal = nf4 * kZRep;
      const int zlo = (int)(((long long)ztotal * blockIdx.x) / G), zhi = (int)(((long long)ztotal * (blockIdx.x + 1)) / G);
      for (int c = zlo + tid; c < zhi; c += kChainThreads) znext[c] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    consumer_sync();
    float xr[XJ][8];
#pragma unroll
    for (int j = 0; j < XJ; ++j) {
      const int c = c_lo + lane + 32 * j;
      if (c < c_hi) {
        const float4 v0 = reinterpret_cast<const float4*>(xs)[2 * c], v1 = reinterpret_cast<const float4*>(xs)[2 * c + 1];
        xr[j][0] = v0.x; xr[j][1] = v0.y; xr[j][2] = v0.z; xr[j][3] = v0.w;
        xr[j][4] = v1.x; xr[j][5] = v1.y; xr[j][6] = v1.z; xr[j][7] = v1.w;
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

    const int vbase = lay_pre[li], nrows = min(lay_pre[li + 1], total_rows) - vbase;
    for (int t0 = 0; t0 < nrows; t0 += TR) {
      const int rows = min(TR, nrows - t0);
      const int s0 = (vbase + t0) % n_stages;  // stage of the tile's first row; the rest follow, wrapping
      const uint32_t use0 = (uint32_t)((vbase + t0) / n_stages);
      // ---- phase 1: (row, segment) partial dot products from shared memory ----
      for (int rr = 0; rr < RPW; ++rr) {
        const int row = row_in_tile + rr * (TR / RPW);
        if (row >= rows) break;
        int s = s0 + row;
        uint32_t use = use0;
        if (s >= n_stages) {
          s -= n_stages;
          ++use;
        }
        if (!npp::mbar_wait(&full_bar[s], use & 1u)) {
          if (lane == 0) {
            atomicOr(a.status, npp::kStatTimeout);
            s_ok = 0;
          }
        }
        const uint4* gp = reinterpret_cast<const uint4*>(csm + (size_t)s * rec_bytes);
        const uint4* up = gp + chunks;
        float g0 = 0.f, g1 = 0.f, u0 = 0.f, u1 = 0.f;  // two chains each: the FMAs of a dot product are dependent
#pragma unroll
        for (int j = 0; j < XJ; ++j) {
          const int c = c_lo + lane + 32 * j;
          if (c < c_hi) {
            const uint4 gw = gp[c], uw = up[c];
            const float4 x0 = make_float4(xr[j][0], xr[j][1], xr[j][2], xr[j][3]);
            const float4 x1 = make_float4(xr[j][4], xr[j][5], xr[j][6], xr[j][7]);
            if (j & 1) {
              g1 = dot8(gw, x0, x1, g1);
              u1 = dot8(uw, x0, x1, u1);
            } else {
              g0 = dot8(gw, x0, x1, g0);
              u0 = dot8(uw, x0, x1, u0);
            }
          }
        }
        float g = g0 + g1, u = u0 + u1;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          g += __shfl_xor_sync(0xffffffffu, g, o);
          u += __shfl_xor_sync(0xffffffffu, u, o);
        }
        if (lane == 0) {
          part[row * SEG + sg][0] = g;
          part[row * SEG + sg][1] = u;
        }
      }
      consumer_sync();
      if (!s_ok) break;
      if (tid < rows) {
        float gs = 0.f, us = 0.f;
        for (int w = 0; w < SEG; ++w) {
          gs += part[tid * SEG + w][0];
          us += part[tid * SEG + w][1];
        }
        // the MLP's input is x_l scaled to unit RMS; the dot products are linear in it
        float ss = 0.f;
        for (int w = 0; w < kChainWarps; ++w) ss += ssq_part[w];
        const float inv_rms = rsqrtf(ss / (float)D + kRmsEps);
        gs *= inv_rms;
        us *= inv_rms;
        act[tid] = gs / (1.f + __expf(-gs)) * us;
      }
      consumer_sync();
      // ---- phase 2: y[cols] += a_i * downT[s_i][cols] ----
      {
        int s = s0;
        for (int q = 0; q < rows; ++q) {
          const float av = act[q];
          const uint4* dp = reinterpret_cast<const uint4*>(csm + (size_t)s * rec_bytes + 2 * row_bytes);
#pragma unroll
          for (int j = 0; j < COLS; ++j) {
            const int c = tid + j * kChainThreads;
            if (c < chunks) {
              const uint4 w = dp[c];
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
          if (++s == n_stages) s = 0;
        }
        // this warp is done with the tile's stages.  (`part` is rewritten only after every warp
        // has passed the barrier above, `act` only after the next tile's first barrier.)
        __syncwarp();
        if (lane == 0) {
          s = s0;
          for (int q = 0; q < rows; ++q) {
            npp::mbar_arrive(&empty_bar[s]);
            if (++s == n_stages) s = 0;
          }
        }
      }
    }
    if (!s_ok) break;

    // ---- add this block's partial MLP_l(x_l) to the layer's accumulator ----
    if (nrows > 0) {
      float* yacc = a.zbuf[l % 3] + (size_t)(blockIdx.x % kZRep) * D;
#pragma unroll
      for (int j = 0; j < COLS; ++j) {
        const int c = tid + j * kChainThreads;
        if (c < chunks) {
          red_add_v4(yacc + (size_t)c * 8, acc[j][0], acc[j][1], acc[j][2], acc[j][3]);
          red_add_v4(yacc + (size_t)c * 8 + 4, acc[j][4], acc[j][5], acc[j][6], acc[j][7]);
        }
      }
    }
    if (li + 1 < nl) {  // publish: every thread's adds and stores precede the arrival
      consumer_sync();
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
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kfn, kChainBlock, sm);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorCooperativeLaunchTooLarge;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid_x);
  cfg.blockDim = dim3(kChainBlock);
  cfg.dynamicSmemBytes = sm;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;  // all blocks co-resident: the grid barrier cannot starve
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kfn, ka);
}

static bool alu_plan(const Dims& d, int sm_count, AluPlan* p) {
  const int chunks = d.D >> 3;
  const size_t rec = (size_t)d.D * 6;
  // shared memory: ring + x (fp32 [D]) + slot cache, under the 227 KB per-block limit
  const long long expect = std::min<long long>(d.C, d.k);
  const int per_block = (int)std::max<long long>(1, (expect + sm_count - 1) / sm_count);
  const int max_per_block = d.C / sm_count + 2;   // whatever the active count turns out to be
  p->run_layers = std::max(1, std::min(kChainMaxLayers, 16384 / (4 * max_per_block)));
  p->slot_cache_rows = p->run_layers * max_per_block;
  const size_t fixed = (size_t)d.D * 4 + (size_t)p->slot_cache_rows * 4;
  const size_t budget = 227 * 1024 - 4096;  // static shared memory and the driver's reserve
  if (fixed + 2 * rec > budget) return false;
  int n_stages = (int)std::min<size_t>(kChainMaxStages, (budget - fixed) / rec);
  if (d.ring_stages >= 2) n_stages = std::min(n_stages, d.ring_stages);
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
  // when the whole share of a layer fits the ring, take it as one tile: two rows per warp
  // in phase 1, half the block-wide barriers
  p->rows_per_warp = 1;
  if (2 * tr <= n_stages && 2 * tr >= per_block) {
    p->rows_per_warp = 2;
    tr *= 2;
  }
  p->n_stages = n_stages;
  p->tile_rows = tr;
  p->window_rows = 2;
  p->smem = (size_t)n_stages * rec + fixed;
  return true;
}

bool supported(const Dims& d, int sm_count) {
  AluPlan p;
  return alu_plan(d, sm_count, &p);
}

cudaError_t launch(const Dims& d_in, const ChainArgs& a, cudaStream_t s, int sm_count) {
  Dims d = d_in;
  if (a.dense_rows > 0) d.k = d.C = a.dense_rows;  // plan for layers whose every row is active
  AluPlan p;
  if (!alu_plan(d, sm_count, &p)) return cudaErrorInvalidValue;
  cudaError_t e = cudaSuccess;
  for (int l0 = a.l_begin; l0 < a.l_end; l0 += p.run_layers) {
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
    ka.l_end = std::min(a.l_end, l0 + p.run_layers);
    ka.slot_cache_rows = p.slot_cache_rows;
    ka.window_rows = std::max(1, std::min(p.n_stages - 1, p.window_rows));
    ka.D = d.D;
    ka.C = d_in.C;
    ka.dense_rows = a.dense_rows;
    ka.n_stages = p.n_stages;
    ka.tile_rows = p.tile_rows;
    ka.rows_per_warp = p.rows_per_warp;
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

}  // namespace chain_alu
}  // namespace npi
