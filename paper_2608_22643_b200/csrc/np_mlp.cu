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
#include "np_pipe.cuh"

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
  int B, D, C, seg, check, normalize;
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
  // optional pre-MLP RMS normalisation: the dot products are linear in x, so only their
  // sums are scaled
  __shared__ float s_ssq[NB][kMlpWarps];
  __shared__ float s_inv[NB];
  if (a.normalize) {
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      float ss = 0.f;
      if (b < nb)
        for (int i = tid; i < D; i += kMlpThreads) ss += xs[(size_t)b * D + i] * xs[(size_t)b * D + i];
      ss = warp_sum(ss);
      if (lane == 0) s_ssq[b][wid] = ss;
    }
    __syncthreads();
    if (tid < NB) {
      float ss = 0.f;
      for (int w = 0; w < kMlpWarps; ++w) ss += s_ssq[tid][w];
      s_inv[tid] = rsqrtf(ss / (float)D + kRmsEps);
    }
  } else if (tid < NB) {
    s_inv[tid] = 1.f;
  }
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
      gs *= s_inv[b];
      us *= s_inv[b];
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

// ---------------------------------------------------------------------------
// One sequence (B = 1): the same computation with the rows staged in shared
// memory by the bulk-copy engine.
//
// A block's share of a layer is only a handful of 3*D*2-byte records, so the
// whole share (or a ring of kStages records when it is larger) is requested up
// front: one thread issues three bulk copies per record (gate, up and down rows
// of the slot) against one mbarrier per stage.  All of a block's bytes are then
// in flight at once, no registers are spent on loads, and the requests go out
// before the kernel waits for the previous layer's output (programmatic
// dependent launch), so a layer's row traffic overlaps the previous layer's tail.
//
// Phase 1: 16 warps = TR rows x SEG segments; a warp's slice of x lives in
// registers (its segment never changes), rows are read from shared memory.
// Phase 2: thread c owns output columns [8c, 8c+8) and walks the tile's down rows.
// ---------------------------------------------------------------------------
constexpr int kPipeMaxStages = 16;

struct MlpPipeArgs {
  MlpKernelArgs k;
  int n_stages;   // records the ring holds
  int tile_rows;  // TR; TR * SEG == kMlpWarps
};

template <int XJ, int COLS>
__global__ void __launch_bounds__(kMlpThreads, 1) k_sparse_mlp_pipe(MlpPipeArgs pa) {
  const MlpKernelArgs& a = pa.k;
  extern __shared__ __align__(128) unsigned char psm[];
  __shared__ __align__(8) uint64_t full_bar[kPipeMaxStages];
  __shared__ float part[kMlpWarps][2];
  __shared__ float act[kMlpWarps];
  __shared__ int s_ok;
  __shared__ float ssq_part[kMlpWarps];  // sums of x^2 per segment (optional RMS normalisation)

  const int D = a.D, chunks = D >> 3;
  const uint32_t row_bytes = (uint32_t)D * 2u;
  const uint32_t rec_bytes = 3u * row_bytes;
  const int n_stages = pa.n_stages, TR = pa.tile_rows, SEG = kMlpWarps / TR;
  const int seg_chunks = (chunks + SEG - 1) / SEG;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;

  int n = *a.n_ptr;  // written by the delta kernel, many launches ago
  if (a.check && (n < 0 || n > a.C)) {
    if (tid == 0) atomicOr(a.status, kStatBadCount);
    n = 0;
  }
  const int G = gridDim.x;
  const int r_begin = (int)(((long long)n * blockIdx.x) / G);
  const int r_end = (int)(((long long)n * (blockIdx.x + 1)) / G);
  const int nrows = r_end - r_begin;

  auto issue_row = [&](int i) {  // local row i -> stage i % n_stages (one lane per row)
    int slot = a.slots[r_begin + i];
    if (a.check && (slot < 0 || slot >= a.C)) {
      atomicOr(a.status, kStatBadSlot);
      slot = 0;
    }
    const int s = i % n_stages;
    unsigned char* dst = psm + (size_t)s * rec_bytes;
    const size_t off = (size_t)slot * row_bytes;
    npp::mbar_expect_tx(&full_bar[s], rec_bytes);
    const uint64_t pol = npp::policy_evict_first();  // weight rows are read once per token
    npp::bulk_g2s_stream(dst, reinterpret_cast<const unsigned char*>(a.gate) + off, row_bytes, &full_bar[s], pol);
    npp::bulk_g2s_stream(dst + row_bytes, reinterpret_cast<const unsigned char*>(a.up) + off, row_bytes, &full_bar[s], pol);
    npp::bulk_g2s_stream(dst + 2 * row_bytes, reinterpret_cast<const unsigned char*>(a.downT) + off, row_bytes,
                         &full_bar[s], pol);
  };

  if (tid == 0) {
    for (int s = 0; s < n_stages; ++s) npp::mbar_init(&full_bar[s], 1);
    npp::fence_barrier_init();
    s_ok = 1;
  }
  __syncthreads();
  // rows are resident before this kernel is launched (the stream is ordered after the
  // layer's install mark), so they can be requested before the previous layer is done;
  // one lane per row, so the slot lookups overlap
  if (wid == 0 && lane < min(nrows, n_stages)) issue_row(lane);
  npp::pdl_launch_dependents();
  npp::pdl_wait_prior();  // x (and the accumulators this kernel adds into) are final from here on

  // this warp's slice of x, in registers: chunks c_lo + lane + 32*j of segment wid % SEG
  const int sg = wid % SEG, row_in_tile = wid / SEG;
  const int c_lo = sg * seg_chunks, c_hi = min(chunks, c_lo + seg_chunks);
  float xr[XJ][8];
#pragma unroll
  for (int j = 0; j < XJ; ++j) {
    const int c = c_lo + lane + 32 * j;
    if (c < c_hi) {
      const float4* pa4 = reinterpret_cast<const float4*>(a.xa + (size_t)c * 8);
      float4 v0 = pa4[0], v1 = pa4[1];
      if (a.xb) {
        const float4* pb4 = reinterpret_cast<const float4*>(a.xb + (size_t)c * 8);
        const float4 w0 = pb4[0], w1 = pb4[1];
        v0.x += w0.x; v0.y += w0.y; v0.z += w0.z; v0.w += w0.w;
        v1.x += w1.x; v1.y += w1.y; v1.z += w1.z; v1.w += w1.w;
      }
      xr[j][0] = v0.x; xr[j][1] = v0.y; xr[j][2] = v0.z; xr[j][3] = v0.w;
      xr[j][4] = v1.x; xr[j][5] = v1.y; xr[j][6] = v1.z; xr[j][7] = v1.w;
      if (blockIdx.x == 0 && row_in_tile == 0) {  // one warp per segment keeps the chain's side effects
        if (a.x_store) {
          float4* ps = reinterpret_cast<float4*>(a.x_store + (size_t)c * 8);
          ps[0] = v0;
          ps[1] = v1;
        }
        if (a.zero_out) {
          float4* pz = reinterpret_cast<float4*>(a.zero_out + (size_t)c * 8);
          pz[0] = make_float4(0.f, 0.f, 0.f, 0.f);
          pz[1] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
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
  if (row_in_tile == 0) {  // one warp per segment covers x exactly once
    float ss = 0.f;
#pragma unroll
    for (int j = 0; j < XJ; ++j)
#pragma unroll
      for (int e = 0; e < 8; ++e) ss += xr[j][e] * xr[j][e];
    ss = warp_sum(ss);
    if (lane == 0) ssq_part[sg] = ss;
  }
  __syncthreads();  // barrier init, s_ok and ssq_part visible to all

  for (int t0 = 0; t0 < nrows; t0 += TR) {
    const int rows = min(TR, nrows - t0);
    // ---- phase 1: this warp's (row, segment) partial dot products ----
    if (row_in_tile < rows) {
      const int i = t0 + row_in_tile;
      const int s = i % n_stages;
      if (!npp::mbar_wait(&full_bar[s], (uint32_t)(i / n_stages) & 1u)) {
        if (lane == 0) {
          atomicOr(a.status, npp::kStatTimeout);
          s_ok = 0;
        }
      }
      const uint4* gp = reinterpret_cast<const uint4*>(psm + (size_t)s * rec_bytes);
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
    if (!s_ok) break;  // a copy never arrived: leave without touching the output
    if (tid < rows) {
      float gs = 0.f, us = 0.f;
      for (int q = 0; q < SEG; ++q) {
        gs += part[tid * SEG + q][0];
        us += part[tid * SEG + q][1];
      }
      if (a.normalize) {
        float ss = 0.f;
        for (int q = 0; q < SEG; ++q) ss += ssq_part[q];
        const float inv_rms = rsqrtf(ss / (float)D + kRmsEps);
        gs *= inv_rms;
        us *= inv_rms;
      }
      act[tid] = gs / (1.f + __expf(-gs)) * us;
    }
    __syncthreads();
    // ---- phase 2: y[cols] += a_i * downT[s_i][cols] from shared memory ----
#pragma unroll
    for (int j = 0; j < COLS; ++j) {
      const int c = tid + j * kMlpThreads;
      if (c < chunks) {
        for (int q = 0; q < rows; ++q) {
          const int s = (t0 + q) % n_stages;
          const uint4 w = reinterpret_cast<const uint4*>(psm + (size_t)s * rec_bytes + 2 * row_bytes)[c];
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
    __syncthreads();  // every read of this tile's stages is done
    // refill the stages this tile used with the rows that map to them next
    if (wid == 0 && lane < rows && t0 + lane + n_stages < nrows) issue_row(t0 + lane + n_stages);
  }

  if (nrows > 0 && s_ok) {
#pragma unroll
    for (int j = 0; j < COLS; ++j) {
      const int c = tid + j * kMlpThreads;
      if (c < chunks) {
        float4* yp = reinterpret_cast<float4*>(a.yacc + (size_t)c * 8);
        atomicAdd(yp, make_float4(acc[j][0], acc[j][1], acc[j][2], acc[j][3]));
        atomicAdd(yp + 1, make_float4(acc[j][4], acc[j][5], acc[j][6], acc[j][7]));
      }
    }
  }
}

template <int XJ, int COLS>
static cudaError_t mlp_pipe_launch(const MlpPipeArgs& pa, size_t sm, int grid_x, cudaStream_t s) {
  auto kfn = k_sparse_mlp_pipe<XJ, COLS>;
  cudaError_t e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid_x);
  cfg.blockDim = dim3(kMlpThreads);
  cfg.dynamicSmemBytes = sm;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kfn, pa);
}

// Picks the ring and tile shape for one sequence; false if the shape is outside what the
// staged kernel covers (the direct-load kernel handles it then).
static bool mlp_pipe_plan(const Dims& d, int sm_count, MlpPipeArgs* pa, size_t* sm, int* xj, int* cols) {
  const int chunks = d.D >> 3;
  const size_t rec = (size_t)d.D * 6;
  const size_t budget = 200 * 1024;
  int n_stages = (int)std::min<size_t>(kPipeMaxStages, budget / rec);
  if (n_stages < 2) return false;
  if (d.ring_stages >= 2) n_stages = std::min(n_stages, d.ring_stages);
  const long long expect = std::min<long long>(d.C, d.k);
  const int per_block = (int)std::max<long long>(1, (expect + sm_count - 1) / sm_count);
  // tile rows: a power of two, about half the block's share (or half the ring), so that the
  // first tile is computed while the second is still arriving
  int tr = 1;
  const int tr_cap = std::max(1, std::min(per_block, n_stages) / 2);
  while (tr * 2 <= tr_cap && tr * 2 <= kMlpWarps) tr *= 2;
  // a segment must give every lane at least one chunk
  while (tr < kMlpWarps && chunks / (kMlpWarps / tr) < 32) tr *= 2;
  if (tr > n_stages) return false;
  const int seg = kMlpWarps / tr;
  const int seg_chunks = (chunks + seg - 1) / seg;
  const int need_xj = (seg_chunks + 31) / 32;
  const int need_cols = (chunks + kMlpThreads - 1) / kMlpThreads;
  if (need_xj > 8 || need_cols > 4) return false;
  pa->n_stages = n_stages;
  pa->tile_rows = tr;
  *sm = (size_t)n_stages * rec;
  *xj = need_xj;
  *cols = need_cols <= 1 ? 1 : (need_cols <= 2 ? 2 : 4);
  return true;
}

static cudaError_t mlp_pipe_dispatch(const MlpPipeArgs& pa, size_t sm, int xj, int cols, int grid_x,
                                     cudaStream_t s) {
#define NP_PIPE(XJV)                                                       \
  do {                                                                     \
    if (cols == 1) return mlp_pipe_launch<XJV, 1>(pa, sm, grid_x, s);      \
    if (cols == 2) return mlp_pipe_launch<XJV, 2>(pa, sm, grid_x, s);      \
    return mlp_pipe_launch<XJV, 4>(pa, sm, grid_x, s);                     \
  } while (0)
  switch (xj) {
    case 1: NP_PIPE(1);
    case 2: NP_PIPE(2);
    case 3: NP_PIPE(3);
    case 4: NP_PIPE(4);
    case 5: NP_PIPE(5);
    case 6: NP_PIPE(6);
    default: NP_PIPE(8);
  }
#undef NP_PIPE
}

template <int NB, int COLS>
static cudaError_t mlp_launch_cols(const MlpKernelArgs& ka, int groups, int grid_x, cudaStream_t s) {
  const size_t sm = ((size_t)NB * ka.D + (size_t)NB * kTileRows * kMaxSeg * 2 + NB * kTileRows) * 4;
  auto kfn = k_sparse_mlp<NB, COLS>;
  // set on every launch: the attribute belongs to the current device's context, and a cache in
  // this function would be shared by all devices and threads of the process
  if (sm > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (e != cudaSuccess) return e;
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
  ka.normalize = a.normalize;
  // warps per row in phase 1: spread the block's expected share of rows over its warps,
  // but keep at least one 16-byte chunk per lane in a segment
  const int chunks = d.D >> 3;
  const long long expect = std::min<long long>(d.C, (long long)d.k * a.B);
  const int per_block = (int)std::max<long long>(1, (expect + sm_count - 1) / sm_count);
  int seg = 1;
  while (seg * 2 <= kMaxSeg && per_block * seg * 2 <= kMlpWarps && chunks / (seg * 2) >= 32) seg *= 2;
  ka.seg = seg;
  if (a.B == 1 && !a.force_direct) {
    MlpPipeArgs pa;
    pa.k = ka;
    size_t sm = 0;
    int xj = 0, cols = 0;
    if (mlp_pipe_plan(d, sm_count, &pa, &sm, &xj, &cols)) return mlp_pipe_dispatch(pa, sm, xj, cols, sm_count, s);
  }
  // sequences per block: as many as keep their fp32 x vectors in shared memory (<= 200 KB)
  const size_t x_bytes = (size_t)d.D * 4;
  if (a.B == 1 || 2 * x_bytes > 200 * 1024) return mlp_launch_nb<1>(ka, a.B, sm_count, s);
  if (a.B == 2 || 4 * x_bytes > 200 * 1024) return mlp_launch_nb<2>(ka, (a.B + 1) / 2, sm_count, s);
  return mlp_launch_nb<4>(ka, (a.B + 3) / 4, sm_count, s);
}

}  // namespace npi
