// Stage 1b for batched sequences (B > 4): the predictor's second layer as a real dense
// contraction on the 5th-generation tensor cores.
//
//   logits[b][r] = sum_m W2[r][m] * hidden[b][m]        r over all L*M rows, b < B <= 16
//
// (One predictor pass scores every FFN neuron of every downstream layer, Section 3.1 step 2;
// the batch is the workload's batch-16 case.)  With 16 sequences the ALU kernel needs
// 16 FMAs per weight element and becomes instruction-bound; here a 128-row tile of W2 is
// the M side of a tcgen05.mma (bf16 x bf16 -> fp32 in tensor memory) and the sequences are
// the N side.  The kernel is still bound by the single pass over W2:
//
//   * W2 tiles [128 rows x 64 k] come in by tiled TMA (128-byte swizzle, the layout the MMA
//     shared-memory descriptor expects) through a ring of 16 KB stages, one producer lane.
//   * hidden is fp32; to keep fp32 accuracy it is split into three bf16 terms
//     (h = h0 + h1 + h2 exactly up to 2^-24), which become 48 N-columns; the three partial
//     products are added in the epilogue.  The extra MMA work is free under the W2 stream.
//   * one lane issues the MMAs (4 per stage, K = 16 each) and commits each stage back to the
//     producer and each finished tile to the epilogue; two 64-column accumulators in tensor
//     memory let the epilogue of tile i overlap the MMAs of tile i+1.
//   * 4 epilogue warps read their 32 TMEM lanes (tcgen05.ld), add the three terms and store
//     coalesced fp32 logits.
//
// Every wait is bounded (np_pipe.cuh); on expiry the roles leave their loops, the block
// meets at the final barrier and tensor memory is released.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cstring>

#include "np_device.cuh"
#include "np_internal.h"
#include "np_pipe.cuh"

namespace npi {

constexpr int kTcTileRows = 128;   // MMA M
constexpr int kTcKBlock = 64;      // k elements per stage (128 bytes of bf16: one swizzle atom)
constexpr int kTcN = 48;           // 16 sequences x 3 bf16 terms
constexpr int kTcAccCols = 64;     // TMEM columns per accumulator (power-of-two allocation)
constexpr int kTcMaxStages = 12;
constexpr int kTcThreads = 192;    // warp 0 TMA, warp 1 MMA + TMEM, warps 2-5 epilogue
constexpr uint32_t kTcStageBytes = kTcTileRows * kTcKBlock * 2;

__device__ __forceinline__ void tma_load_2d(void* dst_smem, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::
          "r"(npp::smem_addr(dst_smem)),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(npp::smem_addr(bar))
      : "memory");
}

__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }

// commit: the mbarrier gets one arrival when all MMAs issued so far by this thread are done
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                   npp::smem_addr(bar))
               : "memory");
}

// K-major operand, 128-byte swizzle: rows of 128 bytes, groups of 8 rows 1024 bytes apart
__device__ __forceinline__ uint64_t tc_smem_desc(const void* p) {
  const uint64_t addr = (uint64_t)(npp::smem_addr(p) & 0x3ffffu) >> 4;
  return addr | (1ull << 16)              // leading byte offset (unused with swizzle): 16 B
         | ((uint64_t)(1024 >> 4) << 32)  // stride byte offset: 8 rows x 128 B
         | (1ull << 46)                   // descriptor version of this architecture
         | (2ull << 61);                  // 128-byte swizzle
}

__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}

__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}

// hidden fp32 [B][H] -> three bf16 terms, rows [term * 16 + b] of a [48][H] array (zero for b >= B).
// n_part > 0: `hidden` holds n_part partial sums [n_part][16][H] of layer 1 (one per K range of the tensor-core
// kernel below); they are added in a fixed order, the ReLU is applied, and the result is also stored to `sum_out`.
__global__ void k_split_hidden(const float* __restrict__ hidden, __nv_bfloat16* __restrict__ out, int H, int B, int n_part,
                               float* __restrict__ sum_out) {
  npp::pdl_launch_dependents();
  npp::pdl_wait_prior();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= 16 * H) return;
  const int b = i / H, m = i - b * H;
  float v = 0.f;
  if (b < B) {
    if (n_part > 0) {
      for (int p = 0; p < n_part; ++p) v += hidden[((size_t)p * 16 + b) * H + m];
      v = fmaxf(v, 0.f);
      sum_out[(size_t)b * H + m] = v;
    } else {
      v = hidden[(size_t)b * H + m];
    }
  }
  const __nv_bfloat16 t0 = __float2bfloat16_rn(v);
  v -= __bfloat162float(t0);
  const __nv_bfloat16 t1 = __float2bfloat16_rn(v);
  v -= __bfloat162float(t1);
  const __nv_bfloat16 t2 = __float2bfloat16_rn(v);
  out[(size_t)(0 * 16 + b) * H + m] = t0;
  out[(size_t)(1 * 16 + b) * H + m] = t1;
  out[(size_t)(2 * 16 + b) * H + m] = t2;
}

__global__ void __launch_bounds__(kTcThreads, 1)
k_pred_l2_tc(const __grid_constant__ CUtensorMap map_w2, const __grid_constant__ CUtensorMap map_h,
             float* __restrict__ logits, long long rows, int H, int B, int n_stages, int32_t* status) {
  extern __shared__ __align__(1024) unsigned char tsm[];
  __shared__ __align__(8) uint64_t full_bar[kTcMaxStages], empty_bar[kTcMaxStages];
  __shared__ __align__(8) uint64_t h_bar, acc_full[2], acc_empty[2];
  __shared__ uint32_t s_tmem_base;

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int n_kb = H / kTcKBlock;
  // shared memory: [ring of W2 stages][hidden terms: n_kb blocks of 48 rows x 128 B]
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tsm) + 1023) & ~(uintptr_t)1023);
  unsigned char* ring = base;
  unsigned char* hsm = base + (size_t)n_stages * kTcStageBytes;
  const uint32_t h_block_bytes = kTcN * kTcKBlock * 2;  // 6144, a multiple of 1024

  const long long n_tiles = (rows + kTcTileRows - 1) / kTcTileRows;
  const long long t_begin = n_tiles * blockIdx.x / gridDim.x, t_end = n_tiles * (blockIdx.x + 1) / gridDim.x;
  const int my_tiles = (int)(t_end - t_begin);

  if (tid == 0) {
    for (int s = 0; s < n_stages; ++s) {
      npp::mbar_init(&full_bar[s], 1);
      npp::mbar_init(&empty_bar[s], 1);
    }
    npp::mbar_init(&h_bar, 1);
    for (int i = 0; i < 2; ++i) {
      npp::mbar_init(&acc_full[i], 1);
      npp::mbar_init(&acc_empty[i], 4);  // one arrival per epilogue warp
    }
    npp::fence_barrier_init();
  }
  if (wid == 1) {  // tensor memory: two accumulators; the address lands in shared memory
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     npp::smem_addr(&s_tmem_base)),
                 "r"(2 * kTcAccCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = s_tmem_base;

  if (wid == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      // W2 does not depend on the previous kernels: start streaming at once; the hidden
      // terms are written by the kernel just before this one
      int it = 0;
      bool ok = true;
      const int prefill = min(n_stages, my_tiles * n_kb);
      for (; it < prefill; ++it) {
        const int kb = it % n_kb;
        const long long tile = t_begin + it / n_kb;
        npp::mbar_expect_tx(&full_bar[it], kTcStageBytes);
        tma_load_2d(ring + (size_t)it * kTcStageBytes, &map_w2, kb * kTcKBlock, (int)(tile * kTcTileRows), &full_bar[it]);
      }
      npp::pdl_wait_prior();
      npp::mbar_expect_tx(&h_bar, (uint32_t)n_kb * h_block_bytes);
      for (int kb = 0; kb < n_kb; ++kb) tma_load_2d(hsm + (size_t)kb * h_block_bytes, &map_h, kb * kTcKBlock, 0, &h_bar);
      const int total = my_tiles * n_kb;
      for (; it < total && ok; ++it) {
        const int s = it % n_stages;
        const uint32_t use = (uint32_t)(it / n_stages);
        if (!npp::mbar_wait(&empty_bar[s], (use & 1u) ^ 1u)) {
          atomicOr(status, npp::kStatTimeout);
          ok = false;
          break;
        }
        const int kb = it % n_kb;
        const long long tile = t_begin + it / n_kb;
        npp::mbar_expect_tx(&full_bar[s], kTcStageBytes);
        tma_load_2d(ring + (size_t)s * kTcStageBytes, &map_w2, kb * kTcKBlock, (int)(tile * kTcTileRows), &full_bar[s]);
      }
    }
  } else if (wid == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      // instruction descriptor: D fp32, A and B bf16, both K-major, N = 48, M = 128
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTcN >> 3) << 17) |
                             ((uint32_t)(kTcTileRows >> 4) << 24);
      bool ok = npp::mbar_wait(&h_bar, 0);
      if (!ok) atomicOr(status, npp::kStatTimeout);
      int it = 0;
      for (int i = 0; i < my_tiles && ok; ++i) {
        const int acc = i & 1;
        const uint32_t acc_use = (uint32_t)(i >> 1);
        if (!npp::mbar_wait(&acc_empty[acc], (acc_use & 1u) ^ 1u)) {
          atomicOr(status, npp::kStatTimeout);
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kTcAccCols);
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const int s = it % n_stages;
          if (!npp::mbar_wait(&full_bar[s], (uint32_t)(it / n_stages) & 1u)) {
            atomicOr(status, npp::kStatTimeout);
            ok = false;
            break;
          }
          tc_fence_after();
          const uint64_t a0 = tc_smem_desc(ring + (size_t)s * kTcStageBytes);
          const uint64_t b0 = tc_smem_desc(hsm + (size_t)kb * h_block_bytes);
#pragma unroll
          for (int k = 0; k < kTcKBlock / 16; ++k) {
            // 16 k-elements = 32 bytes further along the swizzled row: +2 in 16-byte units
            tc_mma(d_tmem, a0 + (uint64_t)(2 * k), b0 + (uint64_t)(2 * k), idesc, (kb | k) != 0 ? 1u : 0u);
          }
          tc_commit(&empty_bar[s]);  // the stage may be refilled once these MMAs have read it
        }
        if (ok) tc_commit(&acc_full[acc]);
      }
    }
  } else {
    // ------------------------------ epilogue warps ------------------------------
    const int q = wid & 3;  // the TMEM lane quarter this warp may read
    for (int i = 0; i < my_tiles; ++i) {
      const int acc = i & 1;
      if (!npp::mbar_wait(&acc_full[acc], (uint32_t)(i >> 1) & 1u)) {
        if (lane == 0) atomicOr(status, npp::kStatTimeout);
        break;
      }
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * kTcAccCols);
      uint32_t t0[16], t1[16], t2[16];
      tc_ld16(taddr, t0);
      tc_ld16(taddr + 16, t1);
      tc_ld16(taddr + 32, t2);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      tc_fence_before();
      __syncwarp();
      if (lane == 0) npp::mbar_arrive(&acc_empty[acc]);  // the accumulator may be overwritten
      const long long r = (t_begin + i) * kTcTileRows + q * 32 + lane;
      if (r < rows) {
#pragma unroll
        for (int b = 0; b < 16; ++b) {
          if (b < B)
            logits[(size_t)b * rows + r] = (__uint_as_float(t2[b]) + __uint_as_float(t1[b])) + __uint_as_float(t0[b]);
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (wid == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * kTcAccCols)
                 : "memory");
  }
}

// ---------------------------------------------------------------------------------------
// Layer 1 for batches on the same tensor cores: raw[b][r] = sum_d W1[r][d] * x[b][d], r < H.  W1 is 4 MB and x is
// bf16 already (one term, N = 16), so the kernel is all latency: the grid is (row tiles of 128) x (K ranges), every
// block loads its few K blocks (a 16 KB tile of W1 and a 2 KB tile of x each) at once, multiplies, and stores its
// partial sums [K range][sequence][row]; k_split_hidden adds the ranges in a fixed order (no atomics: the result
// does not depend on the order in which blocks finish) and applies the ReLU.
constexpr int kL1N = 16;
constexpr int kL1MaxKb = 8;  // K blocks per block, all in flight at once
constexpr uint32_t kL1XBytes = kL1N * kTcKBlock * 2;
constexpr uint32_t kL1StageBytes = kTcStageBytes + kL1XBytes;  // a multiple of 1024: both tiles stay swizzle-aligned

__global__ void __launch_bounds__(kTcThreads, 1)
k_pred_l1_tc(const __grid_constant__ CUtensorMap map_w1, const __grid_constant__ CUtensorMap map_x, float* __restrict__ part,
             int H, int n_kb, int kb_per_block, int32_t* status) {
  extern __shared__ __align__(1024) unsigned char tsm[];
  __shared__ __align__(8) uint64_t full_bar[kL1MaxKb];
  __shared__ __align__(8) uint64_t acc_full;
  __shared__ uint32_t s_tmem_base;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tsm) + 1023) & ~(uintptr_t)1023);
  const int mt = blockIdx.x, kr = blockIdx.y;
  const int kb0 = kr * kb_per_block, nkb = min(kb_per_block, n_kb - kb0);
  if (tid == 0) {
    for (int i = 0; i < kL1MaxKb; ++i) npp::mbar_init(&full_bar[i], 1);
    npp::mbar_init(&acc_full, 1);
    npp::fence_barrier_init();
  }
  if (wid == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(npp::smem_addr(&s_tmem_base)), "r"(32) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  npp::pdl_launch_dependents();
  const uint32_t tmem_base = s_tmem_base;
  if (wid == 0) {
    if (lane == 0) {
      // W1 does not depend on anything before this kernel; x may be the previous operation's
      for (int i = 0; i < nkb; ++i) {
        npp::mbar_expect_tx(&full_bar[i], kL1StageBytes);
        tma_load_2d(base + (size_t)i * kL1StageBytes, &map_w1, (kb0 + i) * kTcKBlock, mt * kTcTileRows, &full_bar[i]);
      }
      npp::pdl_wait_prior();
      for (int i = 0; i < nkb; ++i)
        tma_load_2d(base + (size_t)i * kL1StageBytes + kTcStageBytes, &map_x, (kb0 + i) * kTcKBlock, 0, &full_bar[i]);
    }
  } else if (wid == 1) {
    if (lane == 0) {
      // instruction descriptor: D fp32, A and B bf16, both K-major, N = 16, M = 128
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kL1N >> 3) << 17) | ((uint32_t)(kTcTileRows >> 4) << 24);
      bool ok = true;
      for (int i = 0; i < nkb && ok; ++i) {
        if (!npp::mbar_wait(&full_bar[i], 0)) {
          atomicOr(status, npp::kStatTimeout);
          ok = false;
          break;
        }
        tc_fence_after();
        const uint64_t a0 = tc_smem_desc(base + (size_t)i * kL1StageBytes);
        const uint64_t b0 = tc_smem_desc(base + (size_t)i * kL1StageBytes + kTcStageBytes);
#pragma unroll
        for (int k = 0; k < kTcKBlock / 16; ++k) tc_mma(tmem_base, a0 + (uint64_t)(2 * k), b0 + (uint64_t)(2 * k), idesc, (i | k) != 0 ? 1u : 0u);
      }
      tc_commit(&acc_full);  // also on a timeout: the epilogue must not wait in vain
    }
  } else {
    const int q = wid & 3;  // the TMEM lane quarter this warp may read
    if (npp::mbar_wait(&acc_full, 0)) {
      tc_fence_after();
      uint32_t t0[16];
      tc_ld16(tmem_base + ((uint32_t)(q * 32) << 16), t0);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      const int r = mt * kTcTileRows + q * 32 + lane;
      if (r < H && nkb > 0) {
#pragma unroll
        for (int b = 0; b < kL1N; ++b) part[((size_t)kr * kL1N + b) * H + r] = __uint_as_float(t0[b]);
      }
    } else if (lane == 0) {
      atomicOr(status, npp::kStatTimeout);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (wid == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(32) : "memory");
  }
}

// ---------------------------------------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

bool make_map(CUtensorMap* map, const void* gptr, uint64_t inner, uint64_t outer, uint32_t box_inner,
              uint32_t box_outer) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {inner, outer};
  const cuuint64_t strides[1] = {inner * 2};  // bytes between rows
  const cuuint32_t box[2] = {box_inner, box_outer};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(gptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool pred_tc_supported(const Dims& d) { return d.H % kTcKBlock == 0 && d.H >= kTcKBlock; }

bool pred_tc_prepare(const Dims& d, const void* w1, const void* w2, void* hsplit, float* l1_part, int sm_count, PredTcState* st) {
  static_assert(sizeof(CUtensorMap) <= sizeof(st->map_w2), "tensor map blob too small");
  st->ready = 0;
  st->l1_ready = 0;
  if (!pred_tc_supported(d)) return false;
  // layer 1 on the tensor cores: whole row tiles of W1 and whole K blocks, and room for the partial sums
  if (l1_part && d.H % kTcTileRows == 0 && d.D % kTcKBlock == 0) {
    CUtensorMap w;
    if (make_map(&w, w1, (uint64_t)d.D, (uint64_t)d.H, kTcKBlock, kTcTileRows)) {
      memcpy(st->map_w1, &w, sizeof w);
      const int n_kb = d.D / kTcKBlock, n_mt = d.H / kTcTileRows;
      // K ranges: enough blocks to fill the machine, at most kPredL1Parts partial sums, at most kL1MaxKb K blocks each
      int parts = std::min(std::min(n_kb, kPredL1Parts), std::max(1, sm_count / n_mt));
      int per = (n_kb + parts - 1) / parts;
      if (per <= kL1MaxKb) {
        st->l1_kb_per_block = per;
        st->l1_parts = (n_kb + per - 1) / per;
        st->l1_part = l1_part;
        st->l1_ready = 1;
      }
    }
  }
  CUtensorMap a, b;
  const uint64_t rows = (uint64_t)d.L * d.M;
  if (!make_map(&a, w2, (uint64_t)d.H, rows, kTcKBlock, kTcTileRows)) return false;
  if (!make_map(&b, hsplit, (uint64_t)d.H, kTcN, kTcKBlock, kTcN)) return false;
  memcpy(st->map_w2, &a, sizeof a);
  memcpy(st->map_h, &b, sizeof b);
  const size_t h_bytes = (size_t)(d.H / kTcKBlock) * kTcN * kTcKBlock * 2;
  const size_t budget = 220 * 1024 - 1024;  // alignment slack
  if (h_bytes + 2 * kTcStageBytes > budget) return false;
  st->n_stages = (int)std::min<size_t>(kTcMaxStages, (budget - h_bytes) / kTcStageBytes);
  st->smem = (size_t)st->n_stages * kTcStageBytes + h_bytes + 1024;
  st->hsplit = hsplit;
  st->ready = 1;
  return true;
}

cudaError_t launch_pred_l1_tc(const Dims& d, const PredTcState& st, const void* x_bf16, int B, int32_t* status, cudaStream_t s) {
  if (!st.ready || !st.l1_ready) return cudaErrorInvalidValue;
  CUtensorMap w, x;
  memcpy(&w, st.map_w1, sizeof w);
  // x is the caller's buffer: its map is made per call.  The box has 16 rows, the tensor B: rows past the end read zero.
  if (!make_map(&x, x_bf16, (uint64_t)d.D, (uint64_t)B, kTcKBlock, kL1N)) return cudaErrorInvalidValue;
  const size_t smem = (size_t)st.l1_kb_per_block * kL1StageBytes + 1024;
  cudaError_t e = cudaFuncSetAttribute(k_pred_l1_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  k_pred_l1_tc<<<dim3(d.H / kTcTileRows, st.l1_parts), kTcThreads, smem, s>>>(w, x, st.l1_part, d.H, d.D / kTcKBlock, st.l1_kb_per_block,
                                                                              status);
  return cudaGetLastError();
}

// l1_parts > 0: layer 1 ran on the tensor cores and left that many partial sums; the split kernel adds them up,
// applies the ReLU and stores the hidden vectors to `hidden` as the other layer-1 kernels do.
cudaError_t launch_pred_l2_tc(const Dims& d, const PredTcState& st, float* hidden, int B, float* logits,
                              int32_t* status, cudaStream_t s, int sm_count, int l1_parts) {
  if (!st.ready) return cudaErrorInvalidValue;
  CUtensorMap a, b;
  memcpy(&a, st.map_w2, sizeof a);
  memcpy(&b, st.map_h, sizeof b);
  const int n = 16 * d.H;
  k_split_hidden<<<(n + 255) / 256, 256, 0, s>>>(l1_parts > 0 ? st.l1_part : hidden, static_cast<__nv_bfloat16*>(st.hsplit), d.H, B,
                                                 l1_parts, hidden);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(k_pred_l2_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)st.smem);
  if (e != cudaSuccess) return e;
  const long long rows = (long long)d.L * d.M;
  const long long n_tiles = (rows + kTcTileRows - 1) / kTcTileRows;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)std::min<long long>(sm_count, n_tiles));
  cfg.blockDim = dim3(kTcThreads);
  cfg.dynamicSmemBytes = st.smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k_pred_l2_tc, a, b, logits, rows, d.H, B, st.n_stages, status);
}

}  // namespace npi
