// Stage 4 for batches: the sparse SwiGLU MLP of one layer on tensor cores.
//
//   y[b] = sum_{i in act} silu(gate[s_i] . x[b]) * (up[s_i] . x[b]) * downT[s_i]      (Section 3.4)
//
// With several sequences every weight row is used once per sequence, so the
// dot products are small matrix products: bf16 weights times activations that
// are kept in fp32 and split, on the fly, into three truncated bf16 terms
// (x = t0 + t1 + t2 up to 2^-24 |x|; one MMA per term, fp32 accumulation).
//
// Two kernels per layer, no block ever waits for another block:
//
//   k_mlp_tc_up    grid (row blocks, K slices).  A block streams the K slice of
//                  its rows' gate and up vectors through a ring of bulk copies
//                  and adds its partial dot products (for all sequences) into
//                  GU[row][gate|up][sequence] in global memory.  Slicing K keeps
//                  the block's piece of x small (16 sequences x 1024 columns),
//                  so shared memory goes to rows in flight.
//   k_mlp_tc_down  grid (row blocks, column slices).  A block turns the finished
//                  dot products of its rows into activations h, streams the
//                  column slice of the rows' down vectors and accumulates
//                  y[:, slice] += h^T . down in registers; one vector reduction
//                  per output element and block at the end.
//
// Every weight byte is read once.  The kernels are chained by programmatic
// dependent launch: weight copies are issued before the wait for the previous
// kernel, everything that depends on it after.
#include <algorithm>

#include "np_device.cuh"
#include "np_internal.h"
#include "np_pipe.cuh"

namespace npi {
using namespace npd;
using namespace npp;

namespace {

constexpr int kSeq = 16;  // sequence columns of the MMA tiles (= kMaxBatch)
static_assert(kSeq == kMaxBatch, "tile width follows the batch limit");

constexpr int kUpWarps = 16;  // consumer warps: four per tile slot (all sixteen build the B fragments)
constexpr int kUpSlots = 4;   // tiles in flight, at most
constexpr int kUpBatch = 8;  // prologue items whose loads a thread keeps in flight
constexpr int kUpTile = 8;    // records per tile: 8 gate rows + 8 up rows = the 16 rows of one MMA
constexpr int kUpThreads = (kUpWarps + 1) * 32;

constexpr int kDownWarps = 16;  // consumer warps: each owns up to 8 n-tiles (64 columns) of the slice
constexpr int kDownTile = 16;   // records per tile = the K extent of one MMA
constexpr int kDownMaxSlots = 8;
constexpr int kDownChunk = 128;  // rows whose activations sit in shared memory at a time
constexpr int kDownThreads = (kDownWarps + 1) * 32;
constexpr int kSlotCache = 512;  // slot indices of a block's first rows, fetched in one batch
constexpr int kXPad = 8;  // floats between sequences / activation rows: conflict-free fragment reads

struct TcArgs {
  const unsigned char* gate;  // this layer's row buffers
  const unsigned char* up;
  const unsigned char* downT;
  const int32_t* slots;
  const int32_t* n_ptr;
  const float* xa;
  const float* xb;
  float* yacc;
  float* x_store;
  float* zero_out;
  float* gu;        // [C][2][kSeq] dot products of this layer, zero on entry
  float* gu_next;   // cleared for the next layer by the down kernel (may be NULL)
  float* ssq;       // [kSeq] sum of x^2 per sequence, zero on entry
  float* ssq_next;  // may be NULL
  int32_t* status;
  int B, D, C, SW, check, normalize, up_slots, down_slots;
};

__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
  asm(  // a pure function of its register operands: the compiler may schedule it freely
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}

__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}

// fp32 -> three truncated bf16 terms, returned as fp32 bit patterns with a zero low half
__device__ __forceinline__ void split3(float v, uint32_t& t0, uint32_t& t1, uint32_t& t2) {
  t0 = __float_as_uint(v) & 0xffff0000u;
  const float r1 = v - __uint_as_float(t0);
  t1 = __float_as_uint(r1) & 0xffff0000u;
  const float r2 = r1 - __uint_as_float(t1);
  t2 = __float_as_uint(r2) & 0xffff0000u;
}
// two such terms -> one bf16x2 word, `first` in the low half
__device__ __forceinline__ uint32_t pack2(uint32_t first, uint32_t second) {
  return __byte_perm(first, second, 0x7632);
}

__device__ __forceinline__ void red_add_v4(float* p, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d)
               : "memory");
}

template <int kThreads>
__device__ __forceinline__ void consumer_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");
}

__device__ __forceinline__ int checked_slot(const TcArgs& a, int r) {
  int s = a.slots[r];
  if (a.check && (s < 0 || s >= a.C)) {
    atomicOr(a.status, kStatBadSlot);
    s = 0;
  }
  return s;
}

__device__ __forceinline__ int checked_count(const TcArgs& a) {
  int n = *a.n_ptr;
  if (a.check && (n < 0 || n > a.C)) {
    if (threadIdx.x == 0) atomicOr(a.status, kStatBadCount);
    n = 0;
  }
  return n;
}

// ---------------------------------------------------------------------------
// Phase 1: GU[r][0][b] += gate[s_r][slice] . x[b][slice], GU[r][1][b] likewise for up.
//
// MMA shape: rows = 8 gate rows + 8 up rows of a tile, K = 16 columns of the slice, columns =
// 8 sequences; one MMA per term of x and per group of 8 sequences.  The split of x is the
// same for every tile, so it is done once per block: the prologue leaves the B fragments of
// every K step in shared memory in register layout (a lane's b0/b1 words side by side).
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(kUpThreads, 1) k_mlp_tc_up(TcArgs a) {
  extern __shared__ __align__(128) unsigned char tsm[];
  __shared__ __align__(8) uint64_t full_bar[kUpSlots];
  __shared__ __align__(8) uint64_t empty_bar[kUpSlots];
  __shared__ int s_slots[kSlotCache];

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int rb = blockIdx.x, RB = gridDim.x, ks = blockIdx.y;
  const int D = a.D, SW = a.SW, NS = a.up_slots;
  const int NJ = a.B > 8 ? 2 : 1;                          // groups of 8 sequences
  const int n_ksteps = SW >> 4;
  const uint32_t slice_bytes = (uint32_t)SW * 2u;
  const uint32_t row_stride = slice_bytes + 16u;          // consecutive rows fall into different banks
  uint2* xf = reinterpret_cast<uint2*>(tsm);              // [n_ksteps][NJ][3 terms][32 lanes]
  unsigned char* ring = tsm + (size_t)n_ksteps * NJ * 3 * 32 * 8;  // [NS][16 rows][row_stride]
  const uint32_t slot_bytes = 16u * row_stride;
  constexpr int kQ = 4;                                    // warps per tile; they interleave the K steps

  if (tid == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(&full_bar[i], 1);
      mbar_init(&empty_bar[i], kQ);
    }
    fence_barrier_init();
  }
  __syncthreads();
  pdl_launch_dependents();

  const int n = checked_count(a);
  const int r_begin = (int)(((long long)n * rb) / RB);
  const int r_end = (int)(((long long)n * (rb + 1)) / RB);
  const int n_tiles = (r_end - r_begin + kUpTile - 1) / kUpTile;

  if (wid == kUpWarps) {
    // ---- producer warp: weight rows do not depend on the previous kernel ----
    const size_t slice_off = (size_t)ks * slice_bytes;
    for (int i = lane; i < min(r_end - r_begin, kSlotCache); i += 32) s_slots[i] = checked_slot(a, r_begin + i);
    __syncwarp();
    for (int t = 0; t < n_tiles; ++t) {
      const int slot = t % NS;
      if (t >= NS && !mbar_wait(&empty_bar[slot], (uint32_t)((t / NS - 1) & 1))) {
        if (lane == 0) atomicOr(a.status, kStatTimeout);
        break;
      }
      const int r0 = r_begin + t * kUpTile;
      const int rows = min(kUpTile, r_end - r0);
      if (lane == 0) mbar_expect_tx(&full_bar[slot], (uint32_t)rows * 2u * slice_bytes);
      __syncwarp();
      if (lane < rows) {
        const int ri = r0 - r_begin + lane;
        const size_t src = (size_t)(ri < kSlotCache ? s_slots[ri] : checked_slot(a, r0 + lane)) * D * 2 + slice_off;
        unsigned char* dst = ring + (size_t)slot * slot_bytes + (size_t)lane * row_stride;
        bulk_g2s(dst, a.gate + src, slice_bytes, &full_bar[slot]);
        bulk_g2s(dst + (size_t)kUpTile * row_stride, a.up + src, slice_bytes, &full_bar[slot]);
      }
    }
    return;
  }

  // ---- consumers: B fragments of the x slice (depends on the previous kernel) ----
  pdl_wait_prior();
  constexpr int kC = kUpWarps * 32;
  {
    // item = (K step, sequence group, lane): the four x values behind that lane's b0/b1.
    // A thread's items all belong to one sequence (kC / 32 is a multiple of NJ).
    const int items = n_ksteps * NJ * 32;
    const bool has_b = a.xb != nullptr;
    const int g = lane >> 2, q = lane & 3;
    float ss = 0.f;
    for (int base = tid; base < items; base += kC * kUpBatch) {
      float2 va[kUpBatch][2], vb[kUpBatch][2];
#pragma unroll
      for (int u = 0; u < kUpBatch; ++u) {
        const int it = base + u * kC, pair = it >> 5;
        const int b = 8 * (pair % NJ) + g;
        va[u][0] = va[u][1] = vb[u][0] = vb[u][1] = make_float2(0.f, 0.f);
        if (it < items && b < a.B) {
          const size_t gi = (size_t)b * D + (size_t)ks * SW + (size_t)(pair / NJ) * 16 + 2 * q;
          va[u][0] = __ldcg(reinterpret_cast<const float2*>(a.xa + gi));
          va[u][1] = __ldcg(reinterpret_cast<const float2*>(a.xa + gi + 8));
          if (has_b) {
            vb[u][0] = __ldcg(reinterpret_cast<const float2*>(a.xb + gi));
            vb[u][1] = __ldcg(reinterpret_cast<const float2*>(a.xb + gi + 8));
          }
        }
      }
#pragma unroll
      for (int u = 0; u < kUpBatch; ++u) {
        const int it = base + u * kC, pair = it >> 5;
        if (it < items) {
          const float2 lo = make_float2(va[u][0].x + vb[u][0].x, va[u][0].y + vb[u][0].y);
          const float2 hi = make_float2(va[u][1].x + vb[u][1].x, va[u][1].y + vb[u][1].y);
          uint32_t l0[3], l1[3], h0[3], h1[3];
          split3(lo.x, l0[0], l0[1], l0[2]);
          split3(lo.y, l1[0], l1[1], l1[2]);
          split3(hi.x, h0[0], h0[1], h0[2]);
          split3(hi.y, h1[0], h1[1], h1[2]);
#pragma unroll
          for (int e = 0; e < 3; ++e)
            xf[((size_t)pair * 3 + e) * 32 + lane] = make_uint2(pack2(l0[e], l1[e]), pack2(h0[e], h1[e]));
          ss += lo.x * lo.x + lo.y * lo.y + hi.x * hi.x + hi.y * hi.y;
          const int b = 8 * (pair % NJ) + g;
          if (rb == 0 && b < a.B) {
            const size_t gi = (size_t)b * D + (size_t)ks * SW + (size_t)(pair / NJ) * 16 + 2 * q;
            if (a.x_store) {
              *reinterpret_cast<float2*>(a.x_store + gi) = lo;
              *reinterpret_cast<float2*>(a.x_store + gi + 8) = hi;
            }
            if (a.zero_out) {
              *reinterpret_cast<float2*>(a.zero_out + gi) = make_float2(0.f, 0.f);
              *reinterpret_cast<float2*>(a.zero_out + gi + 8) = make_float2(0.f, 0.f);
            }
          }
        }
      }
    }
    if (rb == 0 && a.normalize) {
      // this slice's share of sum(x^2): lanes 4g..4g+3 hold parts of the same sequence
      ss += __shfl_xor_sync(0xffffffffu, ss, 1);
      ss += __shfl_xor_sync(0xffffffffu, ss, 2);
      const int b = 8 * (wid % NJ) + g;
      if (q == 0 && b < a.B) atomicAdd(a.ssq + b, ss);
    }
  }
  consumer_sync<kC>();
  if (wid >= kQ * NS) return;  // warps beyond the tile slots only helped with the prologue

  const int slot = wid % NS, kq = wid / NS;
  const int g = lane >> 2, q = lane & 3;
  const bool two = NJ == 2;
  const uint32_t a_lane = (uint32_t)(lane & 15) * row_stride + (uint32_t)(lane >> 4) * 16u;
  const uint32_t ring_addr = smem_addr(ring);
  const uint2* xf_lane = xf + lane;
  const int kstep_stride = NJ * 3 * 32;  // uint2 units

  for (int t = slot; t < n_tiles; t += NS) {
    if (!__all_sync(0xffffffffu, mbar_wait(&full_bar[slot], (uint32_t)((t / NS) & 1)))) {
      if (lane == 0) atomicOr(a.status, kStatTimeout);
      break;
    }
    float acc[2][3][4];
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
      for (int e = 0; e < 3; ++e)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[j][e][i] = 0.f;
    const uint32_t a_base = ring_addr + (uint32_t)slot * slot_bytes + a_lane;
#pragma unroll 2
    for (int kstep = kq; kstep < n_ksteps; kstep += kQ) {
      uint32_t af[4];
      ldsm_x4(af, a_base + (uint32_t)kstep * 32u);
      const uint2* xp = xf_lane + (size_t)kstep * kstep_stride;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        if (j == 0 || two) {
#pragma unroll
          for (int e = 0; e < 3; ++e) {
            const uint2 b = xp[(j * 3 + e) * 32];
            mma_16816(acc[j][e], af[0], af[1], af[2], af[3], b.x, b.y);
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty_bar[slot]);  // this warp is done with the tile's rows

    // Rows g (gate of record g) and g + 8 (up of record g); columns = sequences 8j + 2q, +1.
    // Lane pairs trade halves so that even-q lanes add four consecutive sequences of the gate
    // row and odd-q lanes the same four of the up row: every reduction is 16 bytes wide.
    const int r0 = r_begin + t * kUpTile;
    const bool odd = q & 1;
    const bool row_ok = g < min(kUpTile, r_end - r0);
    float* dst = a.gu + ((size_t)(r0 + g) * 2 + (odd ? 1 : 0)) * kSeq + (q & ~1) * 2;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      if (j == 0 || two) {
        const float g0 = acc[j][0][0] + acc[j][1][0] + acc[j][2][0], g1 = acc[j][0][1] + acc[j][1][1] + acc[j][2][1];
        const float u0 = acc[j][0][2] + acc[j][1][2] + acc[j][2][2], u1 = acc[j][0][3] + acc[j][1][3] + acc[j][2][3];
        const float ra = __shfl_xor_sync(0xffffffffu, odd ? g0 : u0, 1);
        const float rbv = __shfl_xor_sync(0xffffffffu, odd ? g1 : u1, 1);
        if (row_ok && 8 * j + (q & ~1) * 2 < a.B) {
          if (odd)
            red_add_v4(dst + 8 * j, ra, rbv, u0, u1);
          else
            red_add_v4(dst + 8 * j, g0, g1, ra, rbv);
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------
// Phase 2: h[b][r] = silu(inv_b * GU[r][0][b]) * inv_b * GU[r][1][b];
//          y[b][slice] += sum_r h[b][r] * downT[s_r][slice].
// MMA shape: rows = sequences, K = 16 records, columns = 8 output columns.  The three terms of
// h share one accumulator: a first MMA carries t0 in rows 0-7 and t1 in rows 8-15 (both of
// sequence g), a second one t2 in rows 0-7; rows g and g + 8 are added at the end.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(kDownThreads, 1) k_mlp_tc_down(TcArgs a) {
  extern __shared__ __align__(128) unsigned char tsm[];
  __shared__ __align__(8) uint64_t full_bar[kDownMaxSlots];
  __shared__ __align__(8) uint64_t empty_bar[kDownMaxSlots];
  __shared__ float s_inv[kSeq];
  __shared__ int s_slots[kSlotCache];

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int rb = blockIdx.x, RB = gridDim.x, cs = blockIdx.y;
  const int D = a.D, SW = a.SW, NS = a.down_slots;
  constexpr int hs_stride = kDownChunk + kXPad;             // floats per sequence
  const uint32_t slice_bytes = (uint32_t)SW * 2u;
  const uint32_t row_stride = slice_bytes + 16u;
  float* hs = reinterpret_cast<float*>(tsm);                // [kSeq][kDownChunk + kXPad]
  unsigned char* ring = tsm + (size_t)kSeq * hs_stride * 4;  // [NS][16 rows][row_stride]
  const uint32_t slot_bytes = (uint32_t)kDownTile * row_stride;

  if (tid == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(&full_bar[i], 1);
      mbar_init(&empty_bar[i], kDownWarps);
    }
    fence_barrier_init();
  }
  __syncthreads();
  pdl_launch_dependents();

  const int n = checked_count(a);
  const int r_begin = (int)(((long long)n * rb) / RB);
  const int r_end = (int)(((long long)n * (rb + 1)) / RB);
  const int n_tiles = (r_end - r_begin + kDownTile - 1) / kDownTile;

  if (wid == kDownWarps) {
    // ---- producer warp ----
    const size_t slice_off = (size_t)cs * slice_bytes;
    for (int i = lane; i < min(r_end - r_begin, kSlotCache); i += 32) s_slots[i] = checked_slot(a, r_begin + i);
    __syncwarp();
    for (int t = 0; t < n_tiles; ++t) {
      const int slot = t % NS;
      if (t >= NS && !mbar_wait(&empty_bar[slot], (uint32_t)((t / NS - 1) & 1))) {
        if (lane == 0) atomicOr(a.status, kStatTimeout);
        break;
      }
      const int r0 = r_begin + t * kDownTile;
      const int rows = min(kDownTile, r_end - r0);
      if (lane == 0) mbar_expect_tx(&full_bar[slot], (uint32_t)kDownTile * slice_bytes);
      __syncwarp();
      if (lane < kDownTile) {
        // a short last tile repeats its last record: those rows meet h = 0, and the shared
        // memory they would otherwise leave stale could hold anything
        const int r = r0 + min(lane, rows - 1);
        const int ri = r - r_begin;
        const size_t src = (size_t)(ri < kSlotCache ? s_slots[ri] : checked_slot(a, r)) * D * 2 + slice_off;
        bulk_g2s(ring + (size_t)slot * slot_bytes + (size_t)lane * row_stride, a.downT + src, slice_bytes,
                 &full_bar[slot]);
      }
    }
    return;
  }

  // ---- consumers ----
  pdl_wait_prior();
  constexpr int kC = kDownWarps * 32;
  if (tid < kSeq) s_inv[tid] = a.normalize ? rsqrtf(__ldcg(a.ssq + tid) / (float)D + kRmsEps) : 1.f;
  {
    // clear the next layer's accumulators (every block a share)
    const int nblk = RB * gridDim.y, bid = cs * RB + rb;
    if (a.gu_next) {
      const size_t total = (size_t)a.C * 2 * kSeq / 4;  // float4 units
      const size_t lo = total * bid / nblk, hi = total * (bid + 1) / nblk;
      float4* p = reinterpret_cast<float4*>(a.gu_next);
      for (size_t i = lo + tid; i < hi; i += kC) p[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (a.ssq_next && bid == 0 && tid < kSeq) a.ssq_next[tid] = 0.f;
  }
  consumer_sync<kC>();

  const int g = lane >> 2, q = lane & 3;
  const int n_mt = a.B > 8 ? 2 : 1;
  const int nt0 = wid * 8;                        // this warp's first n-tile of the slice
  const int my_nt = max(0, min(8, SW / 8 - nt0));  // n-tiles it owns (even: SW % 16 == 0)
  float acc[2][8][4];
#pragma unroll
  for (int m = 0; m < 2; ++m)
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[m][j][i] = 0.f;
  // ldmatrix.trans lane address: matrices 0/1 = records 0-7 / 8-15 of n-tile j, 2/3 = the same of n-tile j + 1
  const uint32_t b_lane = (uint32_t)((lane & 7) + ((lane >> 3) & 1) * 8) * row_stride +
                          (uint32_t)(nt0 + (lane >> 4)) * 16u;
  const uint32_t ring_addr = smem_addr(ring);
  bool ok = true;

  for (int c0 = r_begin; c0 < r_end; c0 += kDownChunk) {
    const int rows_c = min(kDownChunk, r_end - c0);
    const int rows_pad = (rows_c + kDownTile - 1) / kDownTile * kDownTile;
    for (int i = tid; i < rows_pad * kSeq; i += kC) {
      const int rec = i / kSeq, b = i % kSeq;
      float h = 0.f;
      if (rec < rows_c && b < a.B) {
        const float* p = a.gu + (size_t)(c0 + rec) * 2 * kSeq + b;
        const float gs = __ldcg(p) * s_inv[b], us = __ldcg(p + kSeq) * s_inv[b];
        h = gs / (1.f + __expf(-gs)) * us;
      }
      hs[(size_t)b * hs_stride + rec] = h;
    }
    consumer_sync<kC>();

    for (int rl = 0; rl < rows_c; rl += kDownTile) {
      const int t = (c0 - r_begin + rl) / kDownTile;
      const int slot = t % NS;
      // a wait that runs out is reported once; the warp then keeps the loop's barrier
      // structure but neither waits nor computes any more
      if (ok && !__all_sync(0xffffffffu, mbar_wait(&full_bar[slot], (uint32_t)((t / NS) & 1)))) {
        if (lane == 0) atomicOr(a.status, kStatTimeout);
        ok = false;
      }
      if (!ok) continue;
      // A fragments: the three terms of h[8m + g][rl + 2q, +1, +8, +9]
      uint32_t a1[2][4], a2[2][2];
#pragma unroll
      for (int m = 0; m < 2; ++m) {
        if (m < n_mt) {
          const float* hp = hs + (size_t)(8 * m + g) * hs_stride + rl + 2 * q;
          const float2 lo = *reinterpret_cast<const float2*>(hp);
          const float2 hi = *reinterpret_cast<const float2*>(hp + 8);
          uint32_t l0[3], l1[3], h0[3], h1[3];
          split3(lo.x, l0[0], l0[1], l0[2]);
          split3(lo.y, l1[0], l1[1], l1[2]);
          split3(hi.x, h0[0], h0[1], h0[2]);
          split3(hi.y, h1[0], h1[1], h1[2]);
          a1[m][0] = pack2(l0[0], l1[0]);  // row g:     t0, records 2q, 2q+1
          a1[m][1] = pack2(l0[1], l1[1]);  // row g + 8: t1
          a1[m][2] = pack2(h0[0], h1[0]);  // row g:     t0, records 2q+8, 2q+9
          a1[m][3] = pack2(h0[1], h1[1]);  // row g + 8: t1
          a2[m][0] = pack2(l0[2], l1[2]);  // row g:     t2
          a2[m][1] = pack2(h0[2], h1[2]);
        }
      }
      const uint32_t b_base = ring_addr + (uint32_t)slot * slot_bytes + b_lane;
      // two halves of four n-tiles: fragment loads first, then a round of MMAs with (t0 | t1)
      // and a round with t2, eight independent accumulators per round
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        if (4 * hf < my_nt) {
          uint32_t bf[2][4];
#pragma unroll
          for (int p2 = 0; p2 < 2; ++p2)
            if (4 * hf + 2 * p2 < my_nt) ldsm_x4_trans(bf[p2], b_base + (uint32_t)(2 * hf + p2) * 32u);
#pragma unroll
          for (int p2 = 0; p2 < 2; ++p2) {
            if (4 * hf + 2 * p2 < my_nt) {
              const int j = 4 * hf + 2 * p2;
#pragma unroll
              for (int m = 0; m < 2; ++m) {
                if (m < n_mt) {
                  mma_16816(acc[m][j], a1[m][0], a1[m][1], a1[m][2], a1[m][3], bf[p2][0], bf[p2][1]);
                  mma_16816(acc[m][j + 1], a1[m][0], a1[m][1], a1[m][2], a1[m][3], bf[p2][2], bf[p2][3]);
                }
              }
            }
          }
#pragma unroll
          for (int p2 = 0; p2 < 2; ++p2) {
            if (4 * hf + 2 * p2 < my_nt) {
              const int j = 4 * hf + 2 * p2;
#pragma unroll
              for (int m = 0; m < 2; ++m) {
                if (m < n_mt) {
                  mma_16816(acc[m][j], a2[m][0], 0u, a2[m][1], 0u, bf[p2][0], bf[p2][1]);
                  mma_16816(acc[m][j + 1], a2[m][0], 0u, a2[m][1], 0u, bf[p2][2], bf[p2][3]);
                }
              }
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty_bar[slot]);
    }
    consumer_sync<kC>();  // hs is rewritten by the next chunk
  }

  // y[seq][slice columns]: rows g and g + 8 of an accumulator belong to the same sequence.
  // Even-q lanes end up with four consecutive columns of sequence g, odd-q lanes with the
  // same four columns of sequence 8 + g, so every reduction is 16 bytes wide.
  if (r_end > r_begin && ok) {
    const bool odd = q & 1;
    const int seq = odd ? 8 + g : g;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (j < my_nt) {
        const float m0a = acc[0][j][0] + acc[0][j][2], m0b = acc[0][j][1] + acc[0][j][3];
        const float m1a = acc[1][j][0] + acc[1][j][2], m1b = acc[1][j][1] + acc[1][j][3];
        const float ra = __shfl_xor_sync(0xffffffffu, odd ? m0a : m1a, 1);
        const float rbv = __shfl_xor_sync(0xffffffffu, odd ? m0b : m1b, 1);
        if (seq < a.B) {
          float* dst = a.yacc + (size_t)seq * D + (size_t)cs * SW + (size_t)(nt0 + j) * 8 + (q & ~1) * 2;
          if (odd)
            red_add_v4(dst, ra, rbv, m1a, m1b);
          else
            red_add_v4(dst, m0a, m0b, ra, rbv);
        }
      }
    }
  }
}

struct TcPlan {
  int KS, SW, RB, up_slots, down_slots;
  size_t smem_up, smem_down;
};

bool tc_plan(const Dims& d, int sm_count, int B, TcPlan* p) {
  // slices of at most 1024 columns, each a multiple of 16 columns (one K step); four or more
  // slices where the width allows, so that the grid has row blocks x slices ~ SMs
  int ks = std::max(4, (d.D + 1023) / 1024);
  while (ks <= 64 && d.D % (ks * 16) != 0) ++ks;
  if (ks > 64) {
    ks = std::max(1, (d.D + 1023) / 1024);
    while (ks <= 64 && d.D % (ks * 16) != 0) ++ks;
    if (ks > 64) return false;
  }
  p->KS = ks;
  p->SW = d.D / ks;
  p->RB = std::max(1, sm_count / ks);
  const size_t row_stride = (size_t)p->SW * 2 + 16;
  const size_t budget = 220 * 1024;
  const size_t xf_bytes = (size_t)(p->SW / 16) * (B > 8 ? 2 : 1) * 3 * 32 * 8;
  if (xf_bytes + 16 * row_stride > budget) return false;
  p->up_slots = (int)std::min<size_t>(kUpSlots, (budget - xf_bytes) / (16 * row_stride));
  if (d.ring_stages > 0) p->up_slots = std::min(p->up_slots, d.ring_stages);
  p->smem_up = xf_bytes + (size_t)p->up_slots * 16 * row_stride;
  const size_t hs_bytes = (size_t)kSeq * (kDownChunk + kXPad) * 4;
  int ns = (int)std::min<size_t>(kDownMaxSlots, (budget - hs_bytes) / (kDownTile * row_stride));
  if (d.ring_stages > 0) ns = std::min(ns, std::max(2, d.ring_stages));
  if (ns < 1) return false;
  p->down_slots = ns;
  p->smem_down = hs_bytes + (size_t)ns * kDownTile * row_stride;
  return true;
}

template <typename K>
cudaError_t tc_launch(K kfn, dim3 grid, int threads, size_t smem, const TcArgs& ka, cudaStream_t s) {
  cudaError_t e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kfn, ka);
}

}  // namespace

bool mlp_tc_supported(const Dims& d, int sm_count) {
  TcPlan p;
  return tc_plan(d, sm_count, kMaxBatch, &p);
}

size_t mlp_tc_gu_floats(const Dims& d) { return (size_t)d.C * 2 * kSeq; }

cudaError_t launch_sparse_mlp_tc(const Dims& d, const MlpArgs& a, cudaStream_t s, int sm_count) {
  TcPlan p;
  if (!tc_plan(d, sm_count, a.B, &p) || !a.gu || (a.normalize && !a.ssq)) return cudaErrorInvalidValue;
  TcArgs ka;
  ka.gate = static_cast<const unsigned char*>(a.gate_l);
  ka.up = static_cast<const unsigned char*>(a.up_l);
  ka.downT = static_cast<const unsigned char*>(a.downT_l);
  ka.slots = a.active_slots;
  ka.n_ptr = a.n_active_ptr;
  ka.xa = a.xa;
  ka.xb = a.xb;
  ka.yacc = a.yacc;
  ka.x_store = a.x_store;
  ka.zero_out = a.zero_out;
  ka.gu = a.gu;
  ka.gu_next = a.gu_next;
  ka.ssq = a.ssq;
  ka.ssq_next = a.ssq_next;
  ka.status = a.status;
  ka.B = a.B;
  ka.D = d.D;
  ka.C = a.C;
  ka.SW = p.SW;
  ka.check = a.check;
  ka.normalize = a.normalize;
  ka.up_slots = p.up_slots;
  ka.down_slots = p.down_slots;
  const dim3 grid(p.RB, p.KS);
  cudaError_t e = tc_launch(k_mlp_tc_up, grid, kUpThreads, p.smem_up, ka, s);
  if (e != cudaSuccess) return e;
  return tc_launch(k_mlp_tc_down, grid, kDownThreads, p.smem_down, ka, s);
}

}  // namespace npi
