// Stage 4 on tensor cores: the sparse SwiGLU MLP through the slot map,
//
//   y[b] = sum_{i in act} silu(gate[s_i] . x[b]) * (up[s_i] . x[b]) * downT[s_i]      (Section 3.4)
//
// for one to sixteen sequences.  The dot products are small matrix products of bf16 weights
// with activations that stay in fp32 and are split into three truncated bf16 terms
// (v = t0 + t1 + t2 up to 2^-24 |v|; one MMA per term, fp32 accumulation).
//
// The work of a layer is cut twice, and no step needs a vector-wide all-reduce:
//
//   phase "up"    grid (row blocks, K slices).  A block streams the K slice of its rows' gate
//                 and up vectors through a ring of bulk copies and adds its partial dot
//                 products, for all sequences, into GU[row][gate|up][sequence] in global
//                 memory.  Slicing K keeps the block's piece of x small, so shared memory
//                 goes to rows in flight; the split of x is done once per block and layer.
//   phase "down"  grid (row blocks, column slices).  A block turns the finished dot products of
//                 its rows into activations h, streams the column slice of the rows' down
//                 vectors and accumulates y[:, slice] += h^T . down in registers; one 16-byte
//                 reduction per four output elements and block at the end.
//
// Every weight byte is read once.  The two kernels of a layer (k_mlp_tc_up, k_mlp_tc_down) are
// chained by programmatic dependent launch: weight copies are issued before the wait for the
// previous kernel, everything that depends on it after.  (A resident form with two grid
// barriers per layer was measured and was slower at every batch size: the barriers cost as
// much as the kernel boundaries they replace.)
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

constexpr int kWarps = 16;                   // consumer warps of every kernel here
constexpr int kC = kWarps * 32;              // consumer threads
constexpr int kThreads = kC + 32;            // plus one producer warp
constexpr int kQ = 4;                        // warps that share one up tile (they interleave its K steps)
constexpr int kMaxSlots = 8;                 // tiles in flight, at most
constexpr int kTileRows = 16;                // rows of a ring slot: 8 gate + 8 up rows, or 16 down rows
constexpr int kUpTile = 8;                   // records per up tile
constexpr int kDownTile = 16;                // records per down tile = the K extent of one MMA
constexpr int kDownChunk = 128;              // rows whose activations sit in shared memory at a time
constexpr int kSlotCache = 512;              // slot indices of a block's first rows, fetched in one batch
constexpr int kHsStride = kDownChunk + 8;    // floats per sequence in hs: conflict-free fragment reads
constexpr size_t kHsBytes = (size_t)kSeq * kHsStride * 4;

// Block geometry and the few scalars every helper needs.
struct Blk {
  int D, SW, B, NJ, n_ksteps, C, check;
  uint32_t slice_bytes;  // SW * 2
  uint32_t row_stride;   // slice_bytes + 16: consecutive rows of a tile fall into different banks
  uint32_t slot_bytes;   // kTileRows * row_stride
  size_t slice_off;      // byte offset of this block's slice within a row
  size_t row_pitch;      // bytes from one row to the next in the row buffers (D * 2, or a whole record for dense layers)
  int32_t* status;
};

__device__ __forceinline__ Blk make_blk(int B, int D, int C, int SW, int slice, int check, int32_t* status,
                                        int dense_rows) {
  Blk k;
  k.D = D, k.SW = SW, k.B = B, k.C = C, k.check = check;
  k.NJ = B > 8 ? 2 : 1;
  k.n_ksteps = SW >> 4;
  k.slice_bytes = (uint32_t)SW * 2u;
  k.row_stride = k.slice_bytes + 16u;
  k.slot_bytes = (uint32_t)kTileRows * k.row_stride;
  k.slice_off = (size_t)slice * k.slice_bytes;
  k.row_pitch = dense_rows > 0 ? (size_t)D * 6 : (size_t)D * 2;
  if (dense_rows > 0) k.C = dense_rows;  // bound of the slot checks
  k.status = status;
  return k;
}

__device__ __forceinline__ size_t xf_bytes(const Blk& k) { return (size_t)k.n_ksteps * k.NJ * 3 * 32 * 8; }

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

// barrier among the consumer warps only (the producer warp never joins it)
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kC) : "memory"); }

__device__ __forceinline__ int checked_slot(const Blk& k, const int32_t* slots, int r) {
  int s = slots[r];
  if (k.check && (s < 0 || s >= k.C)) {
    atomicOr(k.status, kStatBadSlot);
    s = 0;
  }
  return s;
}

__device__ __forceinline__ int checked_count(const Blk& k, const int32_t* n_ptr) {
  int n = *n_ptr;
  if (k.check && (n < 0 || n > k.C)) {
    if (threadIdx.x == 0) atomicOr(k.status, kStatBadCount);
    n = 0;
  }
  return n;
}

// ---------------------------------------------------------------------------
// Producer side (one warp): slot indices of the block's rows, then one bulk copy per row.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void fill_slot_cache(const Blk& k, const int32_t* slots, int* s_slots, int r_begin,
                                                int r_end, int lane) {
  for (int i = lane; i < min(r_end - r_begin, kSlotCache); i += 32) s_slots[i] = checked_slot(k, slots, r_begin + i);
  __syncwarp();
}

__device__ __forceinline__ int slot_of(const Blk& k, const int32_t* slots, const int* s_slots, int r_begin, int r) {
  const int ri = r - r_begin;
  return ri < kSlotCache ? s_slots[ri] : checked_slot(k, slots, r);
}

// gate rows into tile rows 0-7, up rows into 8-15
__device__ __forceinline__ void issue_up_tile(const Blk& k, const unsigned char* gate, const unsigned char* up,
                                              const int32_t* slots, const int* s_slots, int r_begin, int r0,
                                              int rows, unsigned char* tile, uint64_t* full, int lane) {
  if (lane == 0) mbar_expect_tx(full, (uint32_t)rows * 2u * k.slice_bytes);
  __syncwarp();
  if (lane < rows) {
    const size_t src = (size_t)slot_of(k, slots, s_slots, r_begin, r0 + lane) * k.row_pitch + k.slice_off;
    unsigned char* dst = tile + (size_t)lane * k.row_stride;
    const uint64_t pol = policy_evict_first();  // weight rows are read once per token
    bulk_g2s_stream(dst, gate + src, k.slice_bytes, full, pol);
    bulk_g2s_stream(dst + (size_t)kUpTile * k.row_stride, up + src, k.slice_bytes, full, pol);
  }
}

// A short last tile repeats its last record: those rows meet h = 0, and the shared memory
// they would otherwise leave stale could hold anything (0 * NaN).
__device__ __forceinline__ void issue_down_tile(const Blk& k, const unsigned char* downT, const int32_t* slots,
                                                const int* s_slots, int r_begin, int r0, int rows,
                                                unsigned char* tile, uint64_t* full, int lane) {
  if (lane == 0) mbar_expect_tx(full, (uint32_t)kDownTile * k.slice_bytes);
  __syncwarp();
  if (lane < kDownTile) {
    const int r = r0 + min(lane, rows - 1);
    const size_t src = (size_t)slot_of(k, slots, s_slots, r_begin, r) * k.row_pitch + k.slice_off;
    bulk_g2s_stream(tile + (size_t)lane * k.row_stride, downT + src, k.slice_bytes, full, policy_evict_first());
  }
}

// ---------------------------------------------------------------------------
// Up phase, consumer side.
//
// MMA shape: rows = 8 gate rows + 8 up rows of a tile, K = 16 columns of the slice, columns =
// 8 sequences; one MMA per term of x and per group of 8 sequences.  The split of x is the
// same for every tile, so it is done once: build_x_fragments leaves the B fragments of every
// K step in shared memory in register layout (a lane's b0/b1 words side by side).
// ---------------------------------------------------------------------------

// x = xa (+ xb) of this block's slice -> xf[K step][sequence group][term][lane].  The block
// with `side` set also keeps the chain's side effects for its slice: x is stored, the
// accumulator one layer ahead is cleared, and the slice's share of sum(x^2) is added to ssq.
template <int kBatch>  // items whose loads a thread keeps in flight
__device__ __forceinline__ void build_x_fragments(const Blk& k, int slice, const float* xa, const float* xb,
                                                  float* x_store, float* zero_out, float* ssq, bool side,
                                                  uint2* xf, int tid) {
  // item = (K step, sequence group, lane): the four x values behind that lane's b0/b1.
  // A thread's items all belong to one sequence (kC / 32 is a multiple of NJ).
  const int lane = tid & 31, wid = tid >> 5;
  const int g = lane >> 2, q = lane & 3;
  const int items = k.n_ksteps * k.NJ * 32;
  const bool has_b = xb != nullptr;
  float ss = 0.f;
  for (int base = tid; base < items; base += kC * kBatch) {
    float2 va[kBatch][2], vb[kBatch][2];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int it = base + u * kC, pair = it >> 5;
      const int b = 8 * (pair % k.NJ) + g;
      va[u][0] = va[u][1] = vb[u][0] = vb[u][1] = make_float2(0.f, 0.f);
      if (it < items && b < k.B) {
        const size_t gi = (size_t)b * k.D + (size_t)slice * k.SW + (size_t)(pair / k.NJ) * 16 + 2 * q;
        va[u][0] = __ldcg(reinterpret_cast<const float2*>(xa + gi));
        va[u][1] = __ldcg(reinterpret_cast<const float2*>(xa + gi + 8));
        if (has_b) {
          vb[u][0] = __ldcg(reinterpret_cast<const float2*>(xb + gi));
          vb[u][1] = __ldcg(reinterpret_cast<const float2*>(xb + gi + 8));
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
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
        const int b = 8 * (pair % k.NJ) + g;
        if (side && b < k.B) {
          const size_t gi = (size_t)b * k.D + (size_t)slice * k.SW + (size_t)(pair / k.NJ) * 16 + 2 * q;
          if (x_store) {
            *reinterpret_cast<float2*>(x_store + gi) = lo;
            *reinterpret_cast<float2*>(x_store + gi + 8) = hi;
          }
          if (zero_out) {
            *reinterpret_cast<float2*>(zero_out + gi) = make_float2(0.f, 0.f);
            *reinterpret_cast<float2*>(zero_out + gi + 8) = make_float2(0.f, 0.f);
          }
        }
      }
    }
  }
  if (side && ssq) {
    // lanes 4g..4g+3 hold parts of the same sequence
    ss += __shfl_xor_sync(0xffffffffu, ss, 1);
    ss += __shfl_xor_sync(0xffffffffu, ss, 2);
    const int b = 8 * (wid % k.NJ) + g;
    if (q == 0 && b < k.B) atomicAdd(ssq + b, ss);
  }
}

// One warp's part of an up tile: K steps kq, kq + nw, ... of the tile at shared address
// `tile`; afterwards the partial dot products go to GU.  Rows g (gate of record g) and g + 8
// (up of record g) of the accumulator; columns = sequences 8j + 2q, +1.  Lane pairs trade
// halves so that even-q lanes add four consecutive sequences of the gate row and odd-q lanes
// the same four of the up row: every reduction is 16 bytes wide.
template <int NJ>
__device__ __forceinline__ void up_tile_mma_n(const Blk& k, const uint2* xf, uint32_t tile, int kq, int nw,
                                              int lane, float (&acc)[NJ][3][4]) {
#pragma unroll
  for (int j = 0; j < NJ; ++j)
#pragma unroll
    for (int e = 0; e < 3; ++e)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[j][e][i] = 0.f;
  const uint32_t a_base = tile + (uint32_t)(lane & 15) * k.row_stride + (uint32_t)(lane >> 4) * 16u;
  const uint2* xf_lane = xf + lane;
  constexpr int kstep_stride = NJ * 3 * 32;  // uint2 units
#pragma unroll 2
  for (int kstep = kq; kstep < k.n_ksteps; kstep += nw) {
    uint32_t af[4];
    ldsm_x4(af, a_base + (uint32_t)kstep * 32u);
    const uint2* xp = xf_lane + (size_t)kstep * kstep_stride;
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
#pragma unroll
      for (int e = 0; e < 3; ++e) {
        const uint2 b = xp[(j * 3 + e) * 32];
        mma_16816(acc[j][e], af[0], af[1], af[2], af[3], b.x, b.y);
      }
    }
  }
}

template <int NJ>
__device__ __forceinline__ void up_tile_reds(const Blk& k, const float (&acc)[NJ][3][4], float* gu, int r0,
                                             int rows, int lane) {
  const int g = lane >> 2, q = lane & 3;
  const bool odd = q & 1;
  const bool row_ok = g < rows;
  float* dst = gu + ((size_t)(r0 + g) * 2 + (odd ? 1 : 0)) * kSeq + (q & ~1) * 2;
#pragma unroll
  for (int j = 0; j < NJ; ++j) {
    {
      const float g0 = acc[j][0][0] + acc[j][1][0] + acc[j][2][0], g1 = acc[j][0][1] + acc[j][1][1] + acc[j][2][1];
      const float u0 = acc[j][0][2] + acc[j][1][2] + acc[j][2][2], u1 = acc[j][0][3] + acc[j][1][3] + acc[j][2][3];
      const float ra = __shfl_xor_sync(0xffffffffu, odd ? g0 : u0, 1);
      const float rb = __shfl_xor_sync(0xffffffffu, odd ? g1 : u1, 1);
      if (row_ok && 8 * j + (q & ~1) * 2 < k.B) {
        if (odd)
          red_add_v4(dst + 8 * j, ra, rb, u0, u1);
        else
          red_add_v4(dst + 8 * j, g0, g1, ra, rb);
      }
    }
  }
}

// ---------------------------------------------------------------------------
// Down phase, consumer side.
//
// MMA shape: rows = sequences, K = 16 records, columns = 8 output columns.  The three terms of
// h share one accumulator: a first MMA carries t0 in rows 0-7 and t1 in rows 8-15 (both of
// sequence g), a second one t2 in rows 0-7; rows g and g + 8 are added at the end.
// ---------------------------------------------------------------------------

// h[b][rec] = silu(inv_b * GU[rec][0][b]) * inv_b * GU[rec][1][b] for the chunk's rows; rows up
// to the next multiple of the tile get h = 0.
__device__ __forceinline__ void down_activations(const Blk& k, const float* gu, const float* s_inv, float* hs,
                                                 int c0, int rows_c, int tid) {
  const int rows_pad = (rows_c + kDownTile - 1) / kDownTile * kDownTile;
  for (int i = tid; i < rows_pad * kSeq; i += kC) {
    const int rec = i / kSeq, b = i % kSeq;
    float h = 0.f;
    if (rec < rows_c && b < k.B) {
      const float* p = gu + (size_t)(c0 + rec) * 2 * kSeq + b;
      const float gs = __ldcg(p) * s_inv[b], us = __ldcg(p + kSeq) * s_inv[b];
      h = gs / (1.f + __expf(-gs)) * us;
    }
    hs[(size_t)b * kHsStride + rec] = h;
  }
}

// One warp's part of a down tile: its n-tiles [nt0, nt0 + my_nt) of the slice, records
// rl .. rl + 15 of the chunk.
template <int NJ>
__device__ __forceinline__ void down_tile_mma(const Blk& k, const float* hs, int rl, uint32_t tile, int nt0,
                                              int my_nt, int lane, float (&acc)[NJ][8][4]) {
  const int g = lane >> 2, q = lane & 3;
  // A fragments: the three terms of h[8m + g][rl + 2q, +1, +8, +9]
  uint32_t a1[NJ][4], a2[NJ][2];
#pragma unroll
  for (int m = 0; m < NJ; ++m) {
    {
      const float* hp = hs + (size_t)(8 * m + g) * kHsStride + rl + 2 * q;
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
  // ldmatrix.trans lane address: matrices 0/1 = records 0-7 / 8-15 of n-tile j, 2/3 = the same of n-tile j + 1
  const uint32_t b_base = tile + (uint32_t)((lane & 7) + ((lane >> 3) & 1) * 8) * k.row_stride +
                          (uint32_t)(nt0 + (lane >> 4)) * 16u;
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
          for (int m = 0; m < NJ; ++m) {
            mma_16816(acc[m][j], a1[m][0], a1[m][1], a1[m][2], a1[m][3], bf[p2][0], bf[p2][1]);
            mma_16816(acc[m][j + 1], a1[m][0], a1[m][1], a1[m][2], a1[m][3], bf[p2][2], bf[p2][3]);
          }
        }
      }
#pragma unroll
      for (int p2 = 0; p2 < 2; ++p2) {
        if (4 * hf + 2 * p2 < my_nt) {
          const int j = 4 * hf + 2 * p2;
#pragma unroll
          for (int m = 0; m < NJ; ++m) {
            mma_16816(acc[m][j], a2[m][0], 0u, a2[m][1], 0u, bf[p2][0], bf[p2][1]);
            mma_16816(acc[m][j + 1], a2[m][0], 0u, a2[m][1], 0u, bf[p2][2], bf[p2][3]);
          }
        }
      }
    }
  }
}

// y[seq][slice columns] += acc.  Rows g and g + 8 of an accumulator belong to the same
// sequence.  Even-q lanes end up with four consecutive columns of sequence g, odd-q lanes with
// the same four columns of sequence 8 + g, so every reduction is 16 bytes wide.
template <int NJ>
__device__ __forceinline__ void down_reds(const Blk& k, const float (&acc)[NJ][8][4], float* y_slice, int nt0,
                                          int my_nt, int lane) {
  const int g = lane >> 2, q = lane & 3;
  const bool odd = q & 1;
  const int seq = odd ? 8 + g : g;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    if (j < my_nt) {
      const float m0a = acc[0][j][0] + acc[0][j][2], m0b = acc[0][j][1] + acc[0][j][3];
      const float m1a = NJ == 2 ? acc[NJ - 1][j][0] + acc[NJ - 1][j][2] : 0.f;
      const float m1b = NJ == 2 ? acc[NJ - 1][j][1] + acc[NJ - 1][j][3] : 0.f;
      const float ra = __shfl_xor_sync(0xffffffffu, odd ? m0a : m1a, 1);
      const float rb = __shfl_xor_sync(0xffffffffu, odd ? m0b : m1b, 1);
      if (seq < k.B) {
        float* dst = y_slice + (size_t)seq * k.D + (size_t)(nt0 + j) * 8 + (q & ~1) * 2;
        if (odd)
          red_add_v4(dst, ra, rb, m1a, m1b);
        else
          red_add_v4(dst, m0a, m0b, ra, rb);
      }
    }
  }
}

// every block clears its share of the next layer's accumulators
__device__ __forceinline__ void clear_next(float* gu_next, float* ssq_next, int rows, int bid, int nblk, int tid) {
  if (gu_next) {
    const size_t total = (size_t)rows * 2 * kSeq / 4;  // float4 units
    const size_t lo = total * bid / nblk, hi = total * (bid + 1) / nblk;
    float4* p = reinterpret_cast<float4*>(gu_next);
    for (size_t i = lo + tid; i < hi; i += kC) p[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  if (ssq_next && bid == 0 && tid < kSeq) ssq_next[tid] = 0.f;
}

// ---------------------------------------------------------------------------
// Per-layer form: two kernels, chained by programmatic dependent launch.
// ---------------------------------------------------------------------------
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
  int gu_rows;      // rows the GU buffers hold (all of them are cleared for the next layer)
  void* xterms;     // tcgen05 up phase: x as three bf16 terms, [D / 8][48][8] (may be NULL: legacy up kernel)
  int up_rp;        // tcgen05 up phase: rows of a chunk plane (the most rows a block can have, rounded up to 8)
  int dense_rows;   // > 0: a dense layer.  gate / up / downT point at the three rows of its first record (row
                    // pitch = one record), every one of its dense_rows rows is active, slots = an identity list
};

template <int NJ>
__global__ void __launch_bounds__(kThreads, 1) k_mlp_tc_up(TcArgs a) {
  extern __shared__ __align__(128) unsigned char tsm[];
  __shared__ __align__(8) uint64_t full_bar[kMaxSlots];
  __shared__ __align__(8) uint64_t empty_bar[kMaxSlots];
  __shared__ int s_slots[kSlotCache];

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int rb = blockIdx.x, RB = gridDim.x, ks = blockIdx.y;
  const int NS = a.up_slots;
  const Blk k = make_blk(a.B, a.D, a.C, a.SW, ks, a.check, a.status, a.dense_rows);
  uint2* xf = reinterpret_cast<uint2*>(tsm);  // [n_ksteps][NJ][3 terms][32 lanes]
  unsigned char* ring = tsm + xf_bytes(k);    // [NS][kTileRows][row_stride]

  if (tid == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(&full_bar[i], 1);
      mbar_init(&empty_bar[i], kQ);
    }
    fence_barrier_init();
  }
  __syncthreads();
  pdl_launch_dependents();

  const int n = a.dense_rows > 0 ? a.dense_rows : checked_count(k, a.n_ptr);
  const int r_begin = (int)(((long long)n * rb) / RB);
  const int r_end = (int)(((long long)n * (rb + 1)) / RB);
  const int n_tiles = (r_end - r_begin + kUpTile - 1) / kUpTile;

  if (wid == kWarps) {
    // ---- producer warp: weight rows do not depend on the previous kernel ----
    fill_slot_cache(k, a.slots, s_slots, r_begin, r_end, lane);
    for (int t = 0; t < n_tiles; ++t) {
      const int slot = t % NS;
      if (t >= NS && !mbar_wait(&empty_bar[slot], (uint32_t)((t / NS - 1) & 1))) {
        if (lane == 0) atomicOr(a.status, kStatTimeout);
        break;
      }
      const int r0 = r_begin + t * kUpTile;
      issue_up_tile(k, a.gate, a.up, a.slots, s_slots, r_begin, r0, min(kUpTile, r_end - r0),
                    ring + (size_t)slot * k.slot_bytes, &full_bar[slot], lane);
    }
    return;
  }

  // ---- consumers: everything that depends on the previous kernel ----
  pdl_wait_prior();
  build_x_fragments<4 * NJ>(k, ks, a.xa, a.xb, a.x_store, a.zero_out, a.normalize ? a.ssq : nullptr, rb == 0, xf, tid);
  consumer_sync();
  if (wid >= kQ * NS) return;  // warps beyond the tile slots only helped with the fragments

  const int slot = wid % NS, kq = wid / NS;
  const uint32_t ring_addr = smem_addr(ring);
  for (int t = slot; t < n_tiles; t += NS) {
    if (!__all_sync(0xffffffffu, mbar_wait(&full_bar[slot], (uint32_t)((t / NS) & 1)))) {
      if (lane == 0) atomicOr(a.status, kStatTimeout);
      break;
    }
    float acc[NJ][3][4];
    up_tile_mma_n<NJ>(k, xf, ring_addr + (uint32_t)slot * k.slot_bytes, kq, kQ, lane, acc);
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty_bar[slot]);  // this warp is done with the tile's rows
    const int r0 = r_begin + t * kUpTile;
    up_tile_reds<NJ>(k, acc, a.gu, r0, min(kUpTile, r_end - r0), lane);
  }
}

template <int NJ>
__global__ void __launch_bounds__(kThreads, 1) k_mlp_tc_down(TcArgs a) {
  extern __shared__ __align__(128) unsigned char tsm[];
  __shared__ __align__(8) uint64_t full_bar[kMaxSlots];
  __shared__ __align__(8) uint64_t empty_bar[kMaxSlots];
  __shared__ float s_inv[kSeq];
  __shared__ int s_slots[kSlotCache];

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int rb = blockIdx.x, RB = gridDim.x, cs = blockIdx.y;
  const int NS = a.down_slots;
  const Blk k = make_blk(a.B, a.D, a.C, a.SW, cs, a.check, a.status, a.dense_rows);
  float* hs = reinterpret_cast<float*>(tsm);  // [kSeq][kHsStride]
  unsigned char* ring = tsm + kHsBytes;       // [NS][kTileRows][row_stride]

  if (tid == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(&full_bar[i], 1);
      mbar_init(&empty_bar[i], kWarps);
    }
    fence_barrier_init();
  }
  __syncthreads();
  pdl_launch_dependents();

  const int n = a.dense_rows > 0 ? a.dense_rows : checked_count(k, a.n_ptr);
  const int r_begin = (int)(((long long)n * rb) / RB);
  const int r_end = (int)(((long long)n * (rb + 1)) / RB);
  const int n_tiles = (r_end - r_begin + kDownTile - 1) / kDownTile;

  if (wid == kWarps) {
    fill_slot_cache(k, a.slots, s_slots, r_begin, r_end, lane);
    for (int t = 0; t < n_tiles; ++t) {
      const int slot = t % NS;
      if (t >= NS && !mbar_wait(&empty_bar[slot], (uint32_t)((t / NS - 1) & 1))) {
        if (lane == 0) atomicOr(a.status, kStatTimeout);
        break;
      }
      const int r0 = r_begin + t * kDownTile;
      issue_down_tile(k, a.downT, a.slots, s_slots, r_begin, r0, min(kDownTile, r_end - r0),
                      ring + (size_t)slot * k.slot_bytes, &full_bar[slot], lane);
    }
    return;
  }

  pdl_wait_prior();
  if (tid < kSeq) s_inv[tid] = a.normalize ? rsqrtf(__ldcg(a.ssq + tid) / (float)a.D + kRmsEps) : 1.f;
  clear_next(a.gu_next, a.ssq_next, a.gu_rows, cs * RB + rb, RB * gridDim.y, tid);
  consumer_sync();

  const int nt0 = wid * 8;                           // this warp's first n-tile of the slice
  const int my_nt = max(0, min(8, a.SW / 8 - nt0));  // n-tiles it owns (even: SW % 16 == 0)
  float acc[NJ][8][4];
#pragma unroll
  for (int m = 0; m < NJ; ++m)
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[m][j][i] = 0.f;
  const uint32_t ring_addr = smem_addr(ring);
  bool ok = true;

  for (int c0 = r_begin; c0 < r_end; c0 += kDownChunk) {
    const int rows_c = min(kDownChunk, r_end - c0);
    down_activations(k, a.gu, s_inv, hs, c0, rows_c, tid);
    consumer_sync();
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
      down_tile_mma<NJ>(k, hs, rl, ring_addr + (uint32_t)slot * k.slot_bytes, nt0, my_nt, lane, acc);
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty_bar[slot]);
    }
    consumer_sync();  // hs is rewritten by the next chunk
  }
  if (r_end > r_begin && ok) down_reds<NJ>(k, acc, a.yacc + (size_t)cs * a.SW, nt0, my_nt, lane);
}

// ---------------------------------------------------------------------------
// Up phase on the 5th-generation tensor cores (B >= 2, sparse layers): GU[row][gate|up][b] += W[row][K slice] . x_b.
//
// M = 128 rows of a row block, N = 48 = 16 sequences x 3 bf16 terms of x, K = 16 per MMA, fp32 accumulators in
// tensor memory (gate in columns 0-47, up in 64-111).  The rows are scattered over the slot buffers, so no tiled
// TMA copy can fetch a tile; four warps gather them with 16-byte cp.async into the layout the MMA reads without
// swizzling: 8 x 16-byte core matrices, here simply [16-byte chunk of K][row] (row r of chunk j at 2048 j + 16 r:
// groups of 8 rows 128 bytes apart, K-adjacent core matrices 2048 bytes apart).  Eight consecutive threads copy
// the 128 bytes a row has in a K block, so every 32-byte sector that is read is used.  x comes as one bulk copy:
// k_x_terms has split it once per layer, already in this layout ([chunk][48][8]), where the legacy kernel's blocks
// each rebuilt their slice (5 us of the 17).  One lane issues the MMAs; a commit per stage hands the stage back to
// the gathering warps, which at the end read the accumulators (tcgen05.ld), add the three terms and reduce into GU.
// ---------------------------------------------------------------------------
constexpr int kUpRows = 128;                         // MMA M
constexpr int kUpN = 48;                             // MMA N
constexpr int kUpKb = 64;                            // K per stage
constexpr int kUpStages = 6;                         // five stages in flight: a gather is bound by what it has in flight
constexpr int kUpLoaders = 256;                      // gathering threads (eight warps: one warp alone issues a copy every 13
                                                     // clocks or so); the first four warps also read the accumulators back
constexpr int kUpThreads = kUpLoaders + 32;          // plus the MMA warp
// A stage holds, per matrix (gate, up), 8 chunk planes of `rp` rows x 16 bytes, rp = the most rows a block can have,
// rounded up to 8: a plane is as long as the block's rows need, not 128 rows (the MMA still reads 128 rows per plane:
// those past rp are the next planes' bytes, and their results are not used).
__host__ __device__ constexpr uint32_t up_stage_bytes(int rp) { return 2u * 8u * (uint32_t)rp * 16u; }
constexpr uint32_t kUpChunkN = kUpN * 16;                // bytes of x per 16-byte K chunk: 48 x 16

__device__ __forceinline__ void tc5_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc5_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc5_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_addr(bar)) : "memory");
}
// K-major operand without swizzle: core matrices of 8 rows x 16 bytes; lbo = bytes between K-adjacent core
// matrices, sbo = bytes between groups of 8 rows
__device__ __forceinline__ uint64_t tc5_desc(const void* p, uint32_t lbo, uint32_t sbo) {
  const uint64_t addr = (uint64_t)(smem_addr(p) & 0x3ffffu) >> 4;
  return addr | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) | (1ull << 46);
}
__device__ __forceinline__ void tc5_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}
__device__ __forceinline__ void tc5_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}
__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_smem), "l"(src) : "memory");
}

// x = xa (+ xb) of a layer, once: three bf16 terms per value in the up kernel's operand layout [D / 8][48][8]
// (row 16 t + b of chunk j = term t of x_b[8 j .. 8 j + 7]; rows of sequences past B are zero), and the chain's side
// effects: x is stored, the accumulator one layer ahead is cleared, sum(x^2) per sequence is added to ssq.
__global__ void __launch_bounds__(256) k_x_terms(const float* __restrict__ xa, const float* __restrict__ xb, float* __restrict__ x_store,
                                                 float* __restrict__ zero_out, float* __restrict__ ssq, uint4* __restrict__ xt, int B, int D) {
  pdl_launch_dependents();
  pdl_wait_prior();
  const int chunks = D >> 3;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= kSeq * chunks) return;
  const int b = i / chunks, j = i - b * chunks;  // a warp's threads share b (chunks is a multiple of 32)
  float v[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) v[e] = 0.f;
  if (b < B) {
    const size_t gi = (size_t)b * D + (size_t)j * 8;
    const float4 a0 = __ldcg(reinterpret_cast<const float4*>(xa + gi)), a1 = __ldcg(reinterpret_cast<const float4*>(xa + gi + 4));
    v[0] = a0.x, v[1] = a0.y, v[2] = a0.z, v[3] = a0.w, v[4] = a1.x, v[5] = a1.y, v[6] = a1.z, v[7] = a1.w;
    if (xb) {
      const float4 b0 = __ldcg(reinterpret_cast<const float4*>(xb + gi)), b1 = __ldcg(reinterpret_cast<const float4*>(xb + gi + 4));
      v[0] += b0.x, v[1] += b0.y, v[2] += b0.z, v[3] += b0.w, v[4] += b1.x, v[5] += b1.y, v[6] += b1.z, v[7] += b1.w;
    }
    if (x_store) {
      *reinterpret_cast<float4*>(x_store + gi) = make_float4(v[0], v[1], v[2], v[3]);
      *reinterpret_cast<float4*>(x_store + gi + 4) = make_float4(v[4], v[5], v[6], v[7]);
    }
    if (zero_out) {
      *reinterpret_cast<float4*>(zero_out + gi) = make_float4(0.f, 0.f, 0.f, 0.f);
      *reinterpret_cast<float4*>(zero_out + gi + 4) = make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
  uint32_t t[8][3];
#pragma unroll
  for (int e = 0; e < 8; ++e) split3(v[e], t[e][0], t[e][1], t[e][2]);
#pragma unroll
  for (int k = 0; k < 3; ++k)
    xt[(size_t)j * kUpN + k * kSeq + b] = make_uint4(pack2(t[0][k], t[1][k]), pack2(t[2][k], t[3][k]), pack2(t[4][k], t[5][k]), pack2(t[6][k], t[7][k]));
  if (ssq) {
    float ss = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) ss += v[e] * v[e];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0 && b < B) atomicAdd(ssq + b, ss);
  }
}

#ifdef NP_TRACE  // development builds only
__device__ long long np_up5_clk[64];
#define UK(ev) do { if (blockIdx.x == 3 && blockIdx.y == 1 && (threadIdx.x & 31) == 0) np_up5_clk[ev] = clock64(); } while (0)
#else
#define UK(ev) do { } while (0)
#endif

__global__ void __launch_bounds__(kUpThreads, 1) k_mlp_up5(TcArgs a) {
  extern __shared__ __align__(128) unsigned char tsm[];
  __shared__ __align__(8) uint64_t full_bar[kUpStages];   // a stage's rows have landed (every gathering thread arrives)
  __shared__ __align__(8) uint64_t empty_bar[kUpStages];  // the MMAs that read the stage are done
  __shared__ __align__(8) uint64_t x_bar, acc_bar;
  __shared__ uint32_t s_tmem_base;
  __shared__ uint32_t rowoff[kUpRows];                    // byte offset of a row's K slice in the slot buffers, in 16-byte units

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int rb = blockIdx.x, RB = gridDim.x, ks = blockIdx.y;
  const int SW = a.SW, nkb = SW / kUpKb;
  const size_t row_pitch = (size_t)a.D * 2;
  unsigned char* xsm = tsm;                                        // [SW / 8][48][16 bytes]
  unsigned char* stages = tsm + (size_t)(SW / 8) * kUpChunkN;      // [kUpStages][gate | up][8 chunks][rp rows][16 bytes]
  const uint32_t plane = (uint32_t)a.up_rp * 16u, tile_bytes = 8u * plane, stage_bytes = 2u * tile_bytes;

  if (tid == 0) UK(0);
  if (tid == 0) {
    for (int i = 0; i < kUpStages; ++i) {
      mbar_init(&full_bar[i], kUpLoaders);
      mbar_init(&empty_bar[i], 1);
    }
    mbar_init(&x_bar, 1);
    mbar_init(&acc_bar, 1);
    fence_barrier_init();
  }
  if (wid == kUpLoaders / 32) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&s_tmem_base)), "r"(128) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  int n = *a.n_ptr;
  if (a.check && (n < 0 || n > a.C)) {
    if (tid == 0) atomicOr(a.status, kStatBadCount);
    n = 0;
  }
  const int r_begin = (int)(((long long)n * rb) / RB);
  int nrows = (int)(((long long)n * (rb + 1)) / RB) - r_begin;
  if (nrows > kUpRows) {  // more rows than a tile: the launch code does not choose this kernel for such shapes
    if (tid == 0) atomicOr(a.status, kStatBadCount);
    nrows = kUpRows;
  }
  if (tid < nrows) {
    int slot = a.slots[r_begin + tid];
    if (a.check && (slot < 0 || slot >= a.C)) {
      atomicOr(a.status, kStatBadSlot);
      slot = 0;
    }
    rowoff[tid] = (uint32_t)(((size_t)slot * row_pitch + (size_t)ks * SW * 2) >> 4);
  }
  tc5_fence_before();
  __syncthreads();
  tc5_fence_after();
  pdl_launch_dependents();
  const uint32_t tmem_base = s_tmem_base;
  if (tid == 0) UK(1);

  if (wid < kUpLoaders / 32) {
    // ---------------- gathering warps: the weight rows do not depend on the previous kernel ----------------
    const int chunk = tid & 7, row0 = tid >> 3;  // 8 threads per row, 32 rows per round
    constexpr int kRounds = kUpRows / (kUpLoaders / 8);
    size_t src_off[kRounds];   // this thread's rows: byte offset of its chunk of K block 0 (the same in gate and up)
    uint32_t dst_off[kRounds]; // ... and where it goes inside a stage
#pragma unroll
    for (int i = 0; i < kRounds; ++i) {
      const int row = row0 + (kUpLoaders / 8) * i;
      src_off[i] = row < nrows ? ((size_t)rowoff[row] << 4) + (size_t)chunk * 16 : 0;
      dst_off[i] = (uint32_t)chunk * plane + (uint32_t)row * 16u;
    }
    bool ok = true;
    for (int kb = 0; kb < nkb; ++kb) {
      const int s = kb % kUpStages;
      if (kb >= kUpStages && ok && !mbar_wait(&empty_bar[s], (uint32_t)((kb / kUpStages - 1) & 1))) {
        atomicOr(a.status, kStatTimeout);
        ok = false;
      }
      const uint32_t dst0 = smem_addr(stages + (size_t)s * stage_bytes);
      const size_t koff = (size_t)kb * (kUpKb * 2);
#pragma unroll
      for (int i = 0; i < kRounds; ++i) {
        if (row0 + (kUpLoaders / 8) * i < nrows) {
          cp_async16(dst0 + dst_off[i], a.gate + src_off[i] + koff);
          cp_async16(dst0 + tile_bytes + dst_off[i], a.up + src_off[i] + koff);
        }
      }
      // the thread's arrival on the stage's barrier happens when its copies above have landed: nothing here waits,
      // so a stage is announced as soon as it is complete, whatever the thread is doing by then
      asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_addr(&full_bar[s])) : "memory");
      if (tid == 0 && kb < 16) UK(8 + kb);
    }
    if (wid >= 4) goto done;  // the other four warps read the accumulators
    // ---------------- epilogue: the same warps read the accumulators of their 32 rows ----------------
    const int q = wid & 3;
    if (mbar_wait(&acc_bar, 0)) {
      tc5_fence_after();
      if (tid == 0) UK(2);
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
      uint32_t g0[16], g1[16], g2[16];
      tc5_ld16(taddr, g0);
      tc5_ld16(taddr + 16, g1);
      tc5_ld16(taddr + 32, g2);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      const int row = q * 32 + lane;
      float* dst = a.gu + (size_t)(r_begin + row) * 2 * kSeq;
      if (row < nrows) {
#pragma unroll
        for (int b4 = 0; b4 < kSeq; b4 += 4)
          if (b4 < a.B)
            red_add_v4(dst + b4, (__uint_as_float(g2[b4]) + __uint_as_float(g1[b4])) + __uint_as_float(g0[b4]),
                       (__uint_as_float(g2[b4 + 1]) + __uint_as_float(g1[b4 + 1])) + __uint_as_float(g0[b4 + 1]),
                       (__uint_as_float(g2[b4 + 2]) + __uint_as_float(g1[b4 + 2])) + __uint_as_float(g0[b4 + 2]),
                       (__uint_as_float(g2[b4 + 3]) + __uint_as_float(g1[b4 + 3])) + __uint_as_float(g0[b4 + 3]));
      }
      tc5_ld16(taddr + 64, g0);
      tc5_ld16(taddr + 80, g1);
      tc5_ld16(taddr + 96, g2);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      if (row < nrows) {
#pragma unroll
        for (int b4 = 0; b4 < kSeq; b4 += 4)
          if (b4 < a.B)
            red_add_v4(dst + kSeq + b4, (__uint_as_float(g2[b4]) + __uint_as_float(g1[b4])) + __uint_as_float(g0[b4]),
                       (__uint_as_float(g2[b4 + 1]) + __uint_as_float(g1[b4 + 1])) + __uint_as_float(g0[b4 + 1]),
                       (__uint_as_float(g2[b4 + 2]) + __uint_as_float(g1[b4 + 2])) + __uint_as_float(g0[b4 + 2]),
                       (__uint_as_float(g2[b4 + 3]) + __uint_as_float(g1[b4 + 3])) + __uint_as_float(g0[b4 + 3]));
      }
    } else if (lane == 0) {
      atomicOr(a.status, kStatTimeout);
    }
    if (tid == 0) UK(3);
  } else if (lane == 0) {
    // ---------------- MMA lane ----------------
    pdl_wait_prior();  // the terms of x are the previous kernel's
    UK(4);
    const uint32_t x_bytes = (uint32_t)(SW / 8) * kUpChunkN;
    mbar_expect_tx(&x_bar, x_bytes);
    bulk_g2s(xsm, static_cast<const unsigned char*>(a.xterms) + (size_t)ks * x_bytes, x_bytes, &x_bar);
    // instruction descriptor: D fp32, A and B bf16, both K-major, N = 48, M = 128
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kUpN >> 3) << 17) | ((uint32_t)(kUpRows >> 4) << 24);
    bool ok = mbar_wait(&x_bar, 0);
    if (!ok) atomicOr(a.status, kStatTimeout);
    UK(5);
    for (int kb = 0; kb < nkb && ok; ++kb) {
      const int s = kb % kUpStages;
      if (!mbar_wait(&full_bar[s], (uint32_t)(kb / kUpStages) & 1u)) {
        atomicOr(a.status, kStatTimeout);
        ok = false;
        break;
      }
      fence_proxy_async();  // the rows were written by cp.async; the MMA reads shared memory through the async proxy
      tc5_fence_after();
      const unsigned char* st = stages + (size_t)s * stage_bytes;
#pragma unroll
      for (int k = 0; k < kUpKb / 16; ++k) {  // 16 K values = two 16-byte chunks
        const uint64_t bd = tc5_desc(xsm + (size_t)(kb * 8 + k * 2) * kUpChunkN, kUpChunkN, 128);
        tc5_mma(tmem_base, tc5_desc(st + (size_t)k * 2 * plane, plane, 128), bd, idesc, (kb | k) != 0 ? 1u : 0u);
        tc5_mma(tmem_base + 64, tc5_desc(st + tile_bytes + (size_t)k * 2 * plane, plane, 128), bd, idesc, (kb | k) != 0 ? 1u : 0u);
      }
      tc5_commit(&empty_bar[s]);
      if (kb < 16) UK(32 + kb);
    }
    tc5_commit(&acc_bar);
    UK(6);  // also after a timeout: the epilogue must not wait in vain
  }
done:
  tc5_fence_before();
  __syncthreads();
  if (wid == kUpLoaders / 32) {
    tc5_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(128) : "memory");
  }
}

struct TcPlan {
  int KS, SW, RB;
  int up_slots, down_slots;
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
  const size_t slot_bytes = (size_t)kTileRows * ((size_t)p->SW * 2 + 16);
  const size_t budget = 220 * 1024;
  const size_t xf = (size_t)(p->SW / 16) * (B > 8 ? 2 : 1) * 3 * 32 * 8;
  if (std::max(xf, kHsBytes) + slot_bytes > budget) return false;
  const int cap = d.ring_stages > 0 ? std::min(kMaxSlots, d.ring_stages) : kMaxSlots;
  p->up_slots = (int)std::min<size_t>(std::min(cap, kWarps / kQ), (budget - xf) / slot_bytes);
  p->down_slots = (int)std::min<size_t>(cap, (budget - kHsBytes) / slot_bytes);
  p->smem_up = xf + (size_t)p->up_slots * slot_bytes;
  p->smem_down = kHsBytes + (size_t)p->down_slots * slot_bytes;
  return true;
}

template <typename K>
cudaError_t tc_launch(K kfn, dim3 grid, size_t smem, const TcArgs& ka, cudaStream_t s) {
  cudaError_t e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kThreads);
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

size_t mlp_tc_xterms_bytes(const Dims& d) { return (size_t)d.D / 8 * kUpChunkN; }

// The tcgen05 up kernel applies to sparse layers whose K slices are whole stages and whose row blocks fit one tile.
static int up5_rp(const Dims& d, const TcPlan& p) { return ((d.C + p.RB - 1) / p.RB + 7) & ~7; }
// x terms | stages | slack for the rows the MMA reads past the last plane
static size_t up5_smem(const Dims& d, const TcPlan& p) {
  return (size_t)(p.SW / 8) * kUpChunkN + (size_t)kUpStages * up_stage_bytes(up5_rp(d, p)) + kUpRows * 16;
}
static bool up5_shape_ok(const Dims& d, const TcPlan& p) {
  return p.SW % kUpKb == 0 && d.D % 256 == 0 && up5_rp(d, p) <= kUpRows && up5_smem(d, p) <= 224 * 1024;
}
static bool up5_applies(const Dims& d, const TcPlan& p, const MlpArgs& a) {
  return a.xterms && a.dense_rows == 0 && a.C == d.C && up5_shape_ok(d, p);
}
bool mlp_tc_up_on_tcgen05(const Dims& d, int sm_count) {
  TcPlan p;
  return tc_plan(d, sm_count, kMaxBatch, &p) && up5_shape_ok(d, p);
}

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
  ka.dense_rows = a.dense_rows;
  ka.gu_rows = a.gu_rows > 0 ? a.gu_rows : a.C;
  ka.xterms = a.xterms;
  const dim3 grid(p.RB, p.KS);
  if (up5_applies(d, p, a)) {
    // x once per layer (split, side effects), the up phase on tcgen05, the down phase as before
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((kSeq * (d.D / 8) + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, k_x_terms, a.xa, a.xb, a.x_store, a.zero_out, a.normalize ? a.ssq : (float*)nullptr,
                                       static_cast<uint4*>(a.xterms), a.B, d.D);
    if (e != cudaSuccess) return e;
    const size_t smem_up5 = up5_smem(d, p);
    ka.up_rp = up5_rp(d, p);
    e = cudaFuncSetAttribute(k_mlp_up5, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_up5);
    if (e != cudaSuccess) return e;
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kUpThreads);
    cfg.dynamicSmemBytes = smem_up5;
    e = cudaLaunchKernelEx(&cfg, k_mlp_up5, ka);
    if (e != cudaSuccess) return e;
    return a.B > 8 ? tc_launch(k_mlp_tc_down<2>, grid, p.smem_down, ka, s) : tc_launch(k_mlp_tc_down<1>, grid, p.smem_down, ka, s);
  }
  if (a.B > 8) {
    cudaError_t e = tc_launch(k_mlp_tc_up<2>, grid, p.smem_up, ka, s);
    return e != cudaSuccess ? e : tc_launch(k_mlp_tc_down<2>, grid, p.smem_down, ka, s);
  }
  cudaError_t e = tc_launch(k_mlp_tc_up<1>, grid, p.smem_up, ka, s);
  return e != cudaSuccess ? e : tc_launch(k_mlp_tc_down<1>, grid, p.smem_down, ka, s);
}

}  // namespace npi

#ifdef NP_TRACE
extern "C" int np_debug_up5(void* out) { return (int)cudaMemcpyFromSymbol(out, npi::np_up5_clk, sizeof(npi::np_up5_clk)); }
#endif
