// Dense layers of the residual chain for one sequence (the dense prefix of Section 3.1), a run
// of consecutive layers in one persistent kernel:
//
//   x_{l+1} = x_l + sum_{i < M} silu(gate_l[i].n_l) * (up_l[i].n_l) * downT_l[i],
//   n_l = x_l / sqrt(mean(x_l^2) + 1e-6)
//
// A dense layer is M whole records ([row][gate|up|downT][D] bf16), 270 MB at the 7B shape:
// a streaming job, bound by HBM alone if nothing else gets in the way.  The sparse layers'
// kernels stage rows in a shared-memory ring behind mbarriers and pay a block-wide hand-over
// per tile of 4-8 rows; over the 74 rows a block owns here that hand-over, not the memory,
// set the pace (0.70 of the copy bandwidth).  This kernel has no ring: every thread loads its
// 16-byte pieces straight from global memory into registers, several rows ahead, and the block
// meets only three times per layer.
//
//   phase A  warp w takes rows w, w + 16, ... of the block's share: gate and up dot products
//            against x_l (fp32, in shared memory), 16 pieces of 16 bytes in flight per lane,
//            a shuffle reduction, one activation per row into shared memory;
//   phase B  thread (half, c) adds a_i * downT[i][8c .. 8c+7] over the rows of its half
//            (even / odd), 8 rows in flight; the two halves meet in shared memory and the
//            block adds its partial vector to the layer's accumulator with 16-byte reductions.
//
// Layers hand x over as the other resident kernels do (accumulator copies in zbuf, a counter
// barrier, x_l kept in shared memory), so runs of this kernel and of the sparse kernels chain.
// The wait on the barrier is bounded; on expiry the block records kStatTimeout and leaves.
#include <algorithm>

#include "np_device.cuh"
#include "np_internal.h"
#include "np_pipe.cuh"

namespace npi {
using namespace npd;
namespace dense_chain {

constexpr int kWarps = 16;
constexpr int kThreads = kWarps * 32;
constexpr int kPiecesA = 8;           // 16-byte pieces per projection in flight per lane in phase A
constexpr int kRowsB = 12;            // rows in flight per thread in phase B (times COLS pieces)
constexpr int kMaxRows = 512;         // rows of a layer one block may own

struct KArgs {
  const unsigned char* rec0;  // record 0 of layer 0; layer stride = rows * 3 * D * 2 bytes
  float* xbuf[2];
  float* zbuf[3];
  unsigned int* grid_bar;     // zeroed by the host before the launch
  int32_t* status;
  int l_begin, l_end, D, rows;
};

__device__ __forceinline__ float4 ldcg4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }

__device__ __forceinline__ void red_add_v4(float* p, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d)
               : "memory");
}

__device__ __forceinline__ float dot8(const uint4& w, const float4& x0, const float4& x1, float acc) {
  acc = fmaf(bf16_lo(w.x), x0.x, acc);
  acc = fmaf(bf16_hi(w.x), x0.y, acc);
  acc = fmaf(bf16_lo(w.y), x0.z, acc);
  acc = fmaf(bf16_hi(w.y), x0.w, acc);
  acc = fmaf(bf16_lo(w.z), x1.x, acc);
  acc = fmaf(bf16_hi(w.z), x1.y, acc);
  acc = fmaf(bf16_lo(w.w), x1.z, acc);
  acc = fmaf(bf16_hi(w.w), x1.w, acc);
  return acc;
}

template <int COLS>
__global__ void __launch_bounds__(kThreads, 1) k_dense_chain(KArgs a) {
  extern __shared__ __align__(16) unsigned char dsm[];
  __shared__ float hs[kMaxRows];     // a_i of the block's rows
  __shared__ float ssq_part[kWarps];
  __shared__ int s_ok;

  const int D = a.D, chunks = D >> 3;
  const size_t row_bytes = (size_t)D * 2, rec_bytes = 3 * row_bytes;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int G = gridDim.x, nl = a.l_end - a.l_begin, l_last = a.l_end - 1;
  // x_l, fp32, kept across layers.  Granule c (4 floats) sits at xg(c): the even granules first,
  // then the odd ones, so that the lanes of a warp, which read granules 2p and 2p + 1 for
  // consecutive pieces p, touch consecutive 16-byte words (no bank conflicts)
  float* xs = reinterpret_cast<float*>(dsm);
  auto xg = [chunks](int c) { return (c & 1) * chunks + (c >> 1); };
  float* ys = xs + D;  // partial vectors of the row groups past the first, fp32 [RG - 1][D]
  const int rb = (int)(((long long)a.rows * blockIdx.x) / G), re = (int)(((long long)a.rows * (blockIdx.x + 1)) / G);
  const int nr = min(re - rb, kMaxRows);
  // phase B: cpt threads span the row's column pieces (COLS pieces each), RG such groups share the rows
  const int cpt = min(kThreads, (chunks + COLS - 1) / COLS), RG = kThreads / cpt;
  const int rg = tid / cpt, pc = tid - rg * cpt;
  const bool in_b = rg < RG;  // cpt need not divide the block: the threads left over sit phase B out
  if (tid == 0) s_ok = 1;
  __syncthreads();

  for (int li = 0; li < nl; ++li) {
    const int l = a.l_begin + li;
    const unsigned char* recs = a.rec0 + ((size_t)l * a.rows + rb) * rec_bytes;
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
      __syncthreads();
      if (!s_ok) break;
    }
    // ---- x_l: first layer of the run from global, afterwards x_l = x_{l-1} + MLP_{l-1} ----
    {
      const float* xa = a.xbuf[(l + 1) & 1];
      const float* zb = l > 0 ? a.zbuf[(l - 1) % 3] : nullptr;
      float* xst = a.xbuf[l & 1];
      const int nf4 = chunks * 2;  // float4 granules of one vector
      float ssq = 0.f;
      for (int c = tid; c < nf4; c += kThreads) {
        float4 w[kZRep];
        if (zb) {
#pragma unroll
          for (int r = 0; r < kZRep; ++r) w[r] = ldcg4(zb + (size_t)r * D + (size_t)c * 4);
        }
        float4 v = li == 0 ? ldcg4(xa + (size_t)c * 4) : reinterpret_cast<float4*>(xs)[xg(c)];
        if (zb) {
#pragma unroll
          for (int r = 0; r < kZRep; ++r) {
            v.x += w[r].x; v.y += w[r].y; v.z += w[r].z; v.w += w[r].w;
          }
        }
        reinterpret_cast<float4*>(xs)[xg(c)] = v;
        ssq += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        if (blockIdx.x == 0 && l == l_last) reinterpret_cast<float4*>(xst)[c] = v;  // x for the next launch
      }
      ssq = warp_sum(ssq);
      if (lane == 0) ssq_part[wid] = ssq;
      // clear the next layer's accumulator copies: every block takes a slice
      float4* znext = reinterpret_cast<float4*>(a.zbuf[(l + 1) % 3]);
      const int ztotal = nf4 * kZRep;
      const int zlo = (int)(((long long)ztotal * blockIdx.x) / G), zhi = (int)(((long long)ztotal * (blockIdx.x + 1)) / G);
      for (int c = zlo + tid; c < zhi; c += kThreads) znext[c] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    __syncthreads();
    float ss = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) ss += ssq_part[w];
    // the MLP's input is x_l scaled to unit RMS; the dot products are linear in it
    const float inv_rms = rsqrtf(ss / (float)D + kRmsEps);

    // ---- phase A: one row per warp at a time ----
    for (int r = wid; r < nr; r += kWarps) {
      const unsigned char* grow = recs + (size_t)r * rec_bytes;
      const unsigned char* urow = grow + row_bytes;
      float g = 0.f, u = 0.f;
      for (int p0 = lane; p0 < chunks; p0 += 32 * kPiecesA) {
        // every load is issued, unconditionally, before any is used; a piece past the row's end
        // re-reads the last one and is skipped in the sums
        uint4 wg[kPiecesA], wu[kPiecesA];
#pragma unroll
        for (int i = 0; i < kPiecesA; ++i) {
          const int p = min(p0 + 32 * i, chunks - 1);
          wg[i] = ldg_stream(grow + (size_t)p * 16);
          wu[i] = ldg_stream(urow + (size_t)p * 16);
        }
#pragma unroll
        for (int i = 0; i < kPiecesA; ++i) {
          const int p = p0 + 32 * i;
          if (p < chunks) {
            const float4 x0 = reinterpret_cast<const float4*>(xs)[p];
            const float4 x1 = reinterpret_cast<const float4*>(xs)[chunks + p];
            g = dot8(wg[i], x0, x1, g);
            u = dot8(wu[i], x0, x1, u);
          }
        }
      }
      g = warp_sum(g) * inv_rms;
      u = warp_sum(u) * inv_rms;
      if (lane == 0) hs[r] = g / (1.f + __expf(-g)) * u;
    }
    __syncthreads();

    // ---- phase B: y[cols] += a_i * downT[i][cols]; thread (rg, c): row group rg takes rows
    //      rg, rg + RG, ..., c is the 16-byte column piece ----
    float acc[COLS][8];
#pragma unroll
    for (int j = 0; j < COLS; ++j)
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[j][e] = 0.f;
    for (int r0 = rg; in_b && r0 < nr; r0 += RG * kRowsB) {
      // unconditional loads again: a row past the share's end re-reads the last row with weight 0
      uint4 w[COLS][kRowsB];
#pragma unroll
      for (int j = 0; j < COLS; ++j) {
        const int c = min(pc + j * cpt, chunks - 1);
#pragma unroll
        for (int i = 0; i < kRowsB; ++i) {
          const int r = min(r0 + RG * i, nr - 1);
          w[j][i] = ldg_stream(recs + 2 * row_bytes + (size_t)c * 16 + (size_t)r * rec_bytes);
        }
      }
#pragma unroll
      for (int i = 0; i < kRowsB; ++i) {
        const int r = r0 + RG * i;
        {
          const float av = r < nr ? hs[r] : 0.f;
#pragma unroll
          for (int j = 0; j < COLS; ++j) {
            {
              acc[j][0] = fmaf(av, bf16_lo(w[j][i].x), acc[j][0]);
              acc[j][1] = fmaf(av, bf16_hi(w[j][i].x), acc[j][1]);
              acc[j][2] = fmaf(av, bf16_lo(w[j][i].y), acc[j][2]);
              acc[j][3] = fmaf(av, bf16_hi(w[j][i].y), acc[j][3]);
              acc[j][4] = fmaf(av, bf16_lo(w[j][i].z), acc[j][4]);
              acc[j][5] = fmaf(av, bf16_hi(w[j][i].z), acc[j][5]);
              acc[j][6] = fmaf(av, bf16_lo(w[j][i].w), acc[j][6]);
              acc[j][7] = fmaf(av, bf16_hi(w[j][i].w), acc[j][7]);
            }
          }
        }
      }
    }
    // the row groups meet in shared memory: group rg > 0 leaves its vector in ys[rg - 1]
    if (rg > 0 && in_b) {
#pragma unroll
      for (int j = 0; j < COLS; ++j) {
        const int c = pc + j * cpt;
        if (c < chunks) {
          float4* o = reinterpret_cast<float4*>(ys + (size_t)(rg - 1) * D) + 2 * c;
          o[0] = make_float4(acc[j][0], acc[j][1], acc[j][2], acc[j][3]);
          o[1] = make_float4(acc[j][4], acc[j][5], acc[j][6], acc[j][7]);
        }
      }
    }
    if (RG > 1) __syncthreads();
    if (rg == 0 && nr > 0) {
      float* yacc = a.zbuf[l % 3] + (size_t)(blockIdx.x % kZRep) * D;
#pragma unroll
      for (int j = 0; j < COLS; ++j) {
        const int c = pc + j * cpt;
        if (c < chunks) {
          for (int g2 = 1; g2 < RG; ++g2) {
            const float4* o = reinterpret_cast<const float4*>(ys + (size_t)(g2 - 1) * D) + 2 * c;
            const float4 o0 = o[0], o1 = o[1];
            acc[j][0] += o0.x; acc[j][1] += o0.y; acc[j][2] += o0.z; acc[j][3] += o0.w;
            acc[j][4] += o1.x; acc[j][5] += o1.y; acc[j][6] += o1.z; acc[j][7] += o1.w;
          }
          red_add_v4(yacc + (size_t)c * 8, acc[j][0], acc[j][1], acc[j][2], acc[j][3]);
          red_add_v4(yacc + (size_t)c * 8 + 4, acc[j][4], acc[j][5], acc[j][6], acc[j][7]);
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

template <int COLS>
static cudaError_t launch_k(const KArgs& ka, size_t sm, int grid_x, cudaStream_t s) {
  auto kfn = k_dense_chain<COLS>;
  cudaError_t e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
  if (e != cudaSuccess) return e;
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kfn, kThreads, sm);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorCooperativeLaunchTooLarge;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid_x);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = sm;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;  // all blocks co-resident: the grid barrier cannot starve
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kfn, ka);
}

static int cols_of(const Dims& d) { return ((d.D >> 3) + kThreads - 1) / kThreads; }
static size_t smem_bytes(const Dims& d) {
  const int chunks = d.D >> 3, cols = cols_of(d);
  const int cpt = std::min(kThreads, (chunks + cols - 1) / cols), rgroups = kThreads / cpt;
  return (size_t)d.D * 4 * rgroups;  // x_l and the partial vectors of the other row groups
}

bool supported(const Dims& d, int sm_count) {
  const int chunks = d.D >> 3;
  if (d.D % 8 || chunks > 2 * kThreads) return false;
  if ((d.M + sm_count - 1) / sm_count > kMaxRows) return false;
  return smem_bytes(d) <= 200 * 1024;
}

cudaError_t launch(const Dims& d, const void* rec0, int rows, float* const xbuf[2], float* const zbuf[3],
                   unsigned int* grid_bar, int32_t* status, int l_begin, int l_end, cudaStream_t s, int sm_count) {
  if (!supported(d, sm_count)) return cudaErrorInvalidValue;
  KArgs ka;
  ka.rec0 = static_cast<const unsigned char*>(rec0);
  for (int i = 0; i < 2; ++i) ka.xbuf[i] = xbuf[i];
  for (int i = 0; i < 3; ++i) ka.zbuf[i] = zbuf[i];
  ka.grid_bar = grid_bar;
  ka.status = status;
  ka.l_begin = l_begin;
  ka.l_end = l_end;
  ka.D = d.D;
  ka.rows = rows;
  cudaError_t e = cudaMemsetAsync(grid_bar, 0, sizeof(unsigned int), s);
  if (e != cudaSuccess) return e;
  const size_t sm = smem_bytes(d);
  return cols_of(d) <= 1 ? launch_k<1>(ka, sm, sm_count, s) : launch_k<2>(ka, sm, sm_count, s);
}

}  // namespace dense_chain
}  // namespace npi
