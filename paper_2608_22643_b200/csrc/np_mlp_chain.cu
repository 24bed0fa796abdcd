// Stage 4 over a run of consecutive layers in ONE persistent kernel (B = 1).
//
//   x_{l+1} = x_l + sum_{i in act_l} silu(gate_l[s_i].n_l) * (up_l[s_i].n_l) * downT_l[s_i],
//   n_l = x_l / sqrt(mean(x_l^2) + 1e-6)   (pre-MLP RMS normalisation, unit gain)
//
// (Section 3.4: the sparse MLP reads each active row through the slot map;
// Section 3.1: the sparse suffix runs once its delta rows are in place.)
//
// A layer moves only ~27 MB at the 7B shape, a few microseconds of HBM time, so
// separate launches spend as long on launch latency and on the dependency
// between layers as on the rows.  Here one block per SM stays resident for the
// whole run of layers (cooperative launch).  Each block owns a ring of
// shared-memory stages, one 3*D*2-byte record each, filled by 1-D bulk copies
// from a producer lane; the rows of layer l+1 are requested as soon as a tile of
// layer l has been read, i.e. before layer l's partial sums are reduced and
// before the grid-wide barrier that publishes x_{l+1}, so the row traffic of the
// next layer overlaps this layer's reduction.  What stays exposed per layer is
// the all-reduce of the 4*D-byte output across the blocks (flush of the
// reductions, barrier, re-read of the accumulators) and the two compute phases.
//
// Phase 1 (gate and up dot products of the tile's rows) is on the layer's critical path and
// was issue-bound on the ALUs (an unpack and an FMA per bf16 element), so it runs as
// mma.sync m16n8k16: A = 8 gate rows + 8 up rows read with ldmatrix from the ring (stages are
// staggered by 16 bytes against bank conflicts), B = x_l as three truncated bf16 terms
// (exact to 2^-24), K split over the 16 consumer warps.  Phase 2 (down rows) stays on the
// ALUs: thread c owns 8 output columns.  x_l itself lives in registers, 8 floats per thread.
//
// Every wait (mbarrier, grid barrier) is bounded; on expiry the block records
// kStatTimeout and leaves, and the other blocks follow at their next barrier.
#include <algorithm>

#include "np_device.cuh"
#include "np_internal.h"
#include "np_pipe.cuh"

namespace npi {
using namespace npd;

constexpr int kChainWarps = 16;                      // consumer warps
constexpr int kChainThreads = kChainWarps * 32;      // consumer threads
constexpr int kChainBlock = kChainThreads + 32;      // plus one producer warp
constexpr int kChainMaxStages = 16;
constexpr int kChainTileRows = 8;  // rows per tile: with their gate and up rows, the 16 rows of one MMA
constexpr int kChainMaxLayers = 128;  // layers per launch (longer runs are split by the host)

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
  int l_begin, l_end, D, C, n_stages, tile_rows, check;
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

// mma.sync m16n8k16, bf16 x bf16 -> fp32 (the 16 x 16 A tile holds 8 gate rows and 8 up rows)
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* smem_row) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(npp::smem_addr(smem_row)));
}

// fp32 -> three bf16 terms by truncation: v = t0 + t1 + t2 up to 2^-24 |v|; returns the terms
// as fp32 values whose low 16 bits are zero
__device__ __forceinline__ void split3(float v, uint32_t& t0, uint32_t& t1, uint32_t& t2) {
  t0 = __float_as_uint(v) & 0xffff0000u;
  const float r1 = v - __uint_as_float(t0);
  t1 = __float_as_uint(r1) & 0xffff0000u;
  const float r2 = r1 - __uint_as_float(t1);
  t2 = __float_as_uint(r2) & 0xffff0000u;
}
// two truncated terms -> one packed bf16x2 word (first element in the low half)
__device__ __forceinline__ uint32_t pack_hi16(uint32_t first, uint32_t second) {
  return __byte_perm(first, second, 0x7632);
}

template <int COLS>
__global__ void __launch_bounds__(kChainBlock, 1) k_mlp_chain(ChainKernelArgs a) {
  extern __shared__ __align__(128) unsigned char csm[];
  __shared__ __align__(8) uint64_t full_bar[kChainMaxStages];   // a stage's record has landed
  __shared__ __align__(8) uint64_t empty_bar[kChainMaxStages];  // the consumers are done with it
  __shared__ float part[kChainWarps][16];       // per warp: partial gate (0-7) and up (8-15) sums of the tile's rows
  __shared__ float act[kChainTileRows];         // a_i of the tile's rows
  __shared__ float ssq_part[kChainWarps];       // per-warp sums of x_l^2 (for the RMS normalisation)
  __shared__ int s_ok;
  __shared__ int lay_rb[kChainMaxLayers];       // first active-list index of this block, per layer
  __shared__ int lay_pre[kChainMaxLayers + 1];  // rows of this block before each layer (virtual row index)

  const int D = a.D, chunks = D >> 3;
  const uint32_t row_bytes = (uint32_t)D * 2u;
  const uint32_t rec_bytes = 3u * row_bytes;
  // stages are 16 bytes further apart than a record, so that the same column of the rows of
  // consecutive stages falls into different shared-memory banks (ldmatrix reads 8 rows at once)
  const uint32_t stage_stride = rec_bytes + 16u;
  const uint32_t term_stride = row_bytes + 16u;  // the three bf16 terms of x, staggered the same way
  const size_t layer_bytes = (size_t)a.C * row_bytes;
  const int n_stages = a.n_stages, TR = a.tile_rows;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int G = gridDim.x, nl = a.l_end - a.l_begin;
  unsigned char* xsp = csm + (size_t)n_stages * stage_stride;               // x_l as 3 bf16 terms, [3][D] (+ stagger)
  int* slot_cache = reinterpret_cast<int*>(xsp + 3 * (size_t)term_stride);  // this block's slots, virtual row order

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
    for (int s = 0; s < n_stages; ++s) {
      npp::mbar_init(&full_bar[s], 1);
      npp::mbar_init(&empty_bar[s], 1);
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
        int slot = a.slots[(size_t)(a.l_begin + li) * a.C + lay_rb[li] + i];
        if (a.check && (slot < 0 || slot >= a.C)) {
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
        const size_t off = (size_t)(a.l_begin + ll) * layer_bytes + (size_t)slot_cache[v] * row_bytes;
        unsigned char* dst = csm + (size_t)s * stage_stride;
        npp::mbar_expect_tx(&full_bar[s], rec_bytes);
        npp::bulk_g2s(dst, a.gate + off, row_bytes, &full_bar[s]);
        npp::bulk_g2s(dst + row_bytes, a.up + off, row_bytes, &full_bar[s]);
        npp::bulk_g2s(dst + 2 * row_bytes, a.downT + off, row_bytes, &full_bar[s]);
        if (++s == n_stages) {
          s = 0;
          ++use;
        }
      }
    }
    return;
  }

  // =========================== consumer warps ===========================
  const int l_last = a.l_end - 1;
  const int g8 = lane >> 2, t4 = lane & 3;  // mma fragment coordinates of this lane
  // phase 1 splits the K dimension (D, in blocks of 16) evenly over the consumer warps
  const int kblocks = D >> 4;
  const int kb_lo = (int)(((long long)kblocks * wid) / kChainWarps), kb_hi = (int)(((long long)kblocks * (wid + 1)) / kChainWarps);
  // x_l lives in registers: this thread owns float4 granules tid, tid + 512, ... for the whole run
  float4 xown[2 * COLS];

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
    // ---- x_l: first layer of the run from global, afterwards x_l = x_{l-1} + MLP_{l-1};
    //      each thread updates its own granules and publishes them as three bf16 terms ----
    {
      const float* xa = a.xbuf[(l + 1) & 1];
      const float* zb = l > 0 ? a.zbuf[(l - 1) % 3] : nullptr;
      float* xst = a.xbuf[l & 1];
      const int nf4 = chunks * 2;  // float4 granules of one vector
      float ssq = 0.f;
      float4 w[2 * COLS][kZRep];
      // every load of the pass is issued before any is used
#pragma unroll
      for (int i = 0; i < 2 * COLS; ++i) {
        const int c = tid + i * kChainThreads;
        if (c < nf4) {
          if (li == 0) xown[i] = ldcg4(xa + (size_t)c * 4);
          if (zb) {
#pragma unroll
            for (int r = 0; r < kZRep; ++r) w[i][r] = ldcg4(zb + (size_t)r * D + (size_t)c * 4);
          }
        } else {
          xown[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
#pragma unroll
      for (int i = 0; i < 2 * COLS; ++i) {
        const int c = tid + i * kChainThreads;
        if (c < nf4) {
          float4 v = xown[i];
          if (zb) {
#pragma unroll
            for (int r = 0; r < kZRep; ++r) {
              v.x += w[i][r].x; v.y += w[i][r].y; v.z += w[i][r].z; v.w += w[i][r].w;
            }
          }
          xown[i] = v;
          ssq += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
          uint32_t p0[3], p1[3], p2[3], p3[3];
          split3(v.x, p0[0], p0[1], p0[2]);
          split3(v.y, p1[0], p1[1], p1[2]);
          split3(v.z, p2[0], p2[1], p2[2]);
          split3(v.w, p3[0], p3[1], p3[2]);
#pragma unroll
          for (int term = 0; term < 3; ++term) {
            uint2 packed;
            packed.x = pack_hi16(p0[term], p1[term]);
            packed.y = pack_hi16(p2[term], p3[term]);
            *reinterpret_cast<uint2*>(xsp + (size_t)term * term_stride + (size_t)c * 8) = packed;
          }
          if (blockIdx.x == 0 && l == l_last) reinterpret_cast<float4*>(xst)[c] = v;  // x for the next launch
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
    // this warp's share of the wait for the layer's first tile rides on the same barrier
    const int vbase = lay_pre[li], nrows = min(lay_pre[li + 1], total_rows) - vbase;
    auto poll_tile_row = [&](int t0, int rows) {
      // every warp reads all rows of a tile, but each polls only one row's barrier (an mbarrier
      // poll costs ~0.1 us even when the phase is complete); a block-wide barrier publishes them
      const int v = vbase + t0 + wid % rows;
      if (!npp::mbar_wait(&full_bar[v % n_stages], (uint32_t)(v / n_stages) & 1u)) {
        if (lane == 0) {
          atomicOr(a.status, npp::kStatTimeout);
          s_ok = 0;
        }
      }
    };
    if (nrows > 0) poll_tile_row(0, min(TR, nrows));
    consumer_sync();

    float acc[COLS][8];
#pragma unroll
    for (int j = 0; j < COLS; ++j)
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[j][e] = 0.f;

    for (int t0 = 0; t0 < nrows; t0 += TR) {
      const int rows = min(TR, nrows - t0);
      const int s0 = (vbase + t0) % n_stages;  // stage of the tile's first row; the rest follow, wrapping
      // ---- phase 1 on the tensor cores: [8 gate rows; 8 up rows] x [x as 3 bf16 terms] over this
      //      warp's K range.  Every warp reads all rows of the tile, so it waits for all of them. ----
      if (t0 > 0) {
        poll_tile_row(t0, rows);
        consumer_sync();
      }
      {
        // ldmatrix: lanes 8m..8m+7 give the row addresses of 8x8 matrix m; m & 1 picks up
        // (rows 8-15 of A) over gate, m >> 1 the second 8 columns of the 16-wide K block
        const int m = lane >> 3;
        int r = lane & 7;
        if (r >= rows) r = 0;  // rows past the tile's end: any valid address, results unused
        int sr = s0 + r;
        if (sr >= n_stages) sr -= n_stages;
        const unsigned char* arow = csm + (size_t)sr * stage_stride + (size_t)(m & 1) * row_bytes + (size_t)(m >> 1) * 16;
        const unsigned char* brow = xsp + (size_t)(g8 < 3 ? g8 : 0) * term_stride + (size_t)t4 * 4;
        float c4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
        for (int kb = kb_lo; kb < kb_hi; ++kb) {
          uint32_t af[4];
          ldmatrix_x4(af, arow + (size_t)kb * 32);
          uint32_t b0 = 0u, b1 = 0u;
          if (g8 < 3) {  // column n of B is term n of x; columns 3-7 are zero
            b0 = *reinterpret_cast<const uint32_t*>(brow + (size_t)kb * 32);
            b1 = *reinterpret_cast<const uint32_t*>(brow + (size_t)kb * 32 + 16);
          }
          mma_bf16_16816(c4, af, b0, b1);
        }
        // C: c4[0], c4[1] = (row g8, columns 2*t4, 2*t4+1); c4[2], c4[3] = (row g8 + 8, same columns).
        // The three terms sit in columns 0, 1 (lane t4 = 0) and 2 (lane t4 = 1).
        float lo = t4 == 0 ? c4[0] + c4[1] : (t4 == 1 ? c4[0] : 0.f);
        float hi = t4 == 0 ? c4[2] + c4[3] : (t4 == 1 ? c4[2] : 0.f);
        lo += __shfl_xor_sync(0xffffffffu, lo, 1);
        hi += __shfl_xor_sync(0xffffffffu, hi, 1);
        if (t4 == 0) {
          part[wid][g8] = lo;      // gate . x over this warp's K range, tile row g8
          part[wid][8 + g8] = hi;  // up . x
        }
      }
      consumer_sync();
      if (!s_ok) break;
      if (tid < rows) {
        float gs = 0.f, us = 0.f;
#pragma unroll
        for (int w = 0; w < kChainWarps; ++w) {
          gs += part[w][tid];
          us += part[w][8 + tid];
        }
        // the MLP's input is x_l scaled to unit RMS; the dot products are linear in it
        float ss = 0.f;
#pragma unroll
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
          const uint4* dp = reinterpret_cast<const uint4*>(csm + (size_t)s * stage_stride + 2 * row_bytes);
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
      }
      // every warp is done with the tile's stages: one thread per row releases its stage (a single
      // arrival per stage instead of one per warp keeps the barrier unit out of the way).  The
      // layer's last tile is released after the reductions below, on their barrier.
      if (t0 + TR < nrows) {
        consumer_sync();
        if (tid < rows) {
          int s = s0 + tid;
          if (s >= n_stages) s -= n_stages;
          npp::mbar_arrive(&empty_bar[s]);
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
      if (nrows > 0) {  // release the stages of the layer's last tile
        const int t_last = ((nrows - 1) / TR) * TR;
        if (tid < nrows - t_last) npp::mbar_arrive(&empty_bar[(vbase + t_last + tid) % n_stages]);
      }
      if (tid == 0) {
        __threadfence();
        atomicAdd(a.grid_bar, 1u);
      }
    }
  }
}

template <int COLS>
static cudaError_t chain_launch(const ChainKernelArgs& ka, size_t sm, int grid_x, cudaStream_t s) {
  auto kfn = k_mlp_chain<COLS>;
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

bool mlp_chain_supported(const Dims& d, int sm_count) {
  ChainPlan p;
  return mlp_chain_plan(d, sm_count, &p) || chain_alu::supported(d, sm_count);
}

bool mlp_chain_plan(const Dims& d, int sm_count, ChainPlan* p) {
  if (d.D % 16) return false;  // phase 1 walks D in MMA K blocks of 16
  const int chunks = d.D >> 3;
  const size_t stage = (size_t)d.D * 6 + 16;      // record + stagger
  const size_t terms = 3 * ((size_t)d.D * 2 + 16);  // x as three bf16 terms
  const long long expect = std::min<long long>(d.C, d.k);
  const int per_block = (int)std::max<long long>(1, (expect + sm_count - 1) / sm_count);
  const int max_per_block = d.C / sm_count + 2;  // whatever the active count turns out to be
  // slot cache: up to 4 KB of it, which bounds the layers one launch can span
  p->run_layers = std::max(1, std::min(kChainMaxLayers, 4096 / (4 * max_per_block)));
  p->slot_cache_rows = p->run_layers * max_per_block;
  const size_t fixed = terms + (size_t)p->slot_cache_rows * 4;
  const size_t budget = 227 * 1024 - 3072;  // static shared memory of the kernel
  if (fixed + 2 * stage > budget) return false;
  int n_stages = (int)std::min<size_t>(kChainMaxStages, (budget - fixed) / stage);
  if (d.ring_stages >= 2) n_stages = std::min(n_stages, d.ring_stages);
  // one tile per layer when the block's share fits the ring, else half-ring tiles so that the
  // next tile's rows arrive while this one is computed
  int tr = per_block <= n_stages ? std::min(n_stages, kChainTileRows) : std::max(1, std::min(kChainTileRows, n_stages / 2));
  const int need_cols = (chunks + kChainThreads - 1) / kChainThreads;
  if (need_cols > 4) return false;
  p->cols = need_cols <= 1 ? 1 : (need_cols <= 2 ? 2 : 4);
  p->single_tile = per_block <= std::min(n_stages, kChainTileRows) ? 1 : 0;
  p->n_stages = n_stages;
  p->tile_rows = tr;
  p->window_rows = 2;
  p->smem = (size_t)n_stages * stage + fixed;
  return true;
}

cudaError_t launch_mlp_chain(const Dims& d, const ChainArgs& a, cudaStream_t s, int sm_count) {
  ChainPlan p;
  const bool mma_ok = mlp_chain_plan(d, sm_count, &p);
  // the tensor-core form pays a fixed price per tile: keep it for shares that are one tile
  if ((!mma_ok || !p.single_tile) && chain_alu::supported(d, sm_count)) return chain_alu::launch(d, a, s, sm_count);
  if (!mma_ok) return cudaErrorInvalidValue;
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
    ka.C = d.C;
    ka.n_stages = p.n_stages;
    ka.tile_rows = p.tile_rows;
    ka.check = a.check;
    e = cudaMemsetAsync(a.grid_bar, 0, sizeof(unsigned int), s);
    if (e != cudaSuccess) return e;
    if (p.cols == 1) e = chain_launch<1>(ka, p.smem, sm_count, s);
    else if (p.cols == 2) e = chain_launch<2>(ka, p.smem, sm_count, s);
    else e = chain_launch<4>(ka, p.smem, sm_count, s);
    if (e != cudaSuccess) return e;
  }
  return e;
}

}  // namespace npi
