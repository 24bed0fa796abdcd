// Stage 1: predictor forward, logits = W2 * relu(W1 * x)  (one pass after
// layer 0 scores every FFN neuron of every downstream layer; Section 3.1 step 2).
//
// Both layers are matrix-vector products at small batch: every weight byte is
// read once, so the kernels are organised around 16-byte coalesced streaming
// loads with many loads in flight per thread, fp32 accumulation and
// warp-shuffle reductions.
#include <algorithm>

#include "np_device.cuh"
#include "np_internal.h"
#include "np_pipe.cuh"

namespace npi {
using namespace npd;

// ---------------------------------------------------------------------------
// Layer 1: hidden[b][m] = max(0, sum_j W1[m][j] * x[b][j]).   W1 is small
// (H*D*2 bytes): one warp per output row, all sequences per pass.
// ---------------------------------------------------------------------------
template <int NB>
__global__ void __launch_bounds__(128) k_pred_l1(const uint4* __restrict__ w1,
                                                  const uint4* __restrict__ x,  // bf16 [B][D]
                                                  float* __restrict__ hidden, int H, int D, int B) {
  npp::pdl_launch_dependents();  // layer 2 may start prefetching its weights now
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp >= H) return;
  const int chunks = D >> 3;  // 16-byte chunks per row
  const uint4* row = w1 + (size_t)warp * chunks;
  float acc[NB];
#pragma unroll
  for (int b = 0; b < NB; ++b) acc[b] = 0.f;
  for (int c0 = 0; c0 < chunks; c0 += 32 * 4) {
    uint4 w[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int c = c0 + u * 32 + lane;
      w[u] = c < chunks ? ldg_stream(row + c) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int c = c0 + u * 32 + lane;
      if (c < chunks) {
#pragma unroll
        for (int b = 0; b < NB; ++b) {
          if (b < B) {
            const uint4 xv = __ldg(x + (size_t)b * chunks + c);
            const float4 xa = make_float4(bf16_lo(xv.x), bf16_hi(xv.x), bf16_lo(xv.y), bf16_hi(xv.y));
            const float4 xb = make_float4(bf16_lo(xv.z), bf16_hi(xv.z), bf16_lo(xv.w), bf16_hi(xv.w));
            acc[b] = dot8(w[u], xa, xb, acc[b]);
          }
        }
      }
    }
  }
#pragma unroll
  for (int b = 0; b < NB; ++b) {
    const float v = warp_sum(acc[b]);
    if (lane == 0 && b < B) hidden[(size_t)b * H + warp] = fmaxf(v, 0.f);
  }
}

// One sequence: a row per block, a quarter of the row per warp, so that (for rows of up to
// 4096 values) every weight load of the kernel is issued at once and the kernel lasts one
// trip to memory, not four; the layer behind it waits for exactly this kernel.
__global__ void __launch_bounds__(128) k_pred_l1_row(const uint4* __restrict__ w1, const uint4* __restrict__ x,
                                                      float* __restrict__ hidden, int H, int D) {
  __shared__ float part[4];
  npp::pdl_launch_dependents();  // layer 2 may start prefetching its weights now
  const int row = blockIdx.x, lane = threadIdx.x & 31, wq = threadIdx.x >> 5;
  const int chunks = D >> 3;  // 16-byte chunks per row
  const uint4* wr = w1 + (size_t)row * chunks;
  float acc = 0.f;
  for (int c0 = wq * 128; c0 < chunks; c0 += 512) {
    uint4 w[4], xv[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int c = c0 + u * 32 + lane;
      w[u] = c < chunks ? ldg_stream(wr + c) : make_uint4(0, 0, 0, 0);
      xv[u] = c < chunks ? __ldg(x + c) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const float4 xa = make_float4(bf16_lo(xv[u].x), bf16_hi(xv[u].x), bf16_lo(xv[u].y), bf16_hi(xv[u].y));
      const float4 xb = make_float4(bf16_lo(xv[u].z), bf16_hi(xv[u].z), bf16_lo(xv[u].w), bf16_hi(xv[u].w));
      acc = dot8(w[u], xa, xb, acc);
    }
  }
  acc = warp_sum(acc);
  if (lane == 0) part[wq] = acc;
  __syncthreads();
  if (threadIdx.x == 0) hidden[row] = fmaxf((part[0] + part[1]) + (part[2] + part[3]), 0.f);
}

// Batched form (B > 4): the B input vectors are staged once per block in shared memory (as
// bf16), so that a weight chunk is multiplied with all sequences without going back to L1/L2
// for x; one warp per output row.
__global__ void __launch_bounds__(128) k_pred_l1_batch(const uint4* __restrict__ w1, const uint4* __restrict__ x,
                                                        float* __restrict__ hidden, int H, int D, int B) {
  extern __shared__ __align__(16) uint4 xsm[];  // [B][D/8]
  npp::pdl_launch_dependents();
  const int chunks = D >> 3;
  for (int i = threadIdx.x; i < B * chunks; i += blockDim.x) xsm[i] = __ldg(x + i);
  __syncthreads();
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp >= H) return;
  const uint4* row = w1 + (size_t)warp * chunks;
  float acc[kMaxBatch];
#pragma unroll
  for (int b = 0; b < kMaxBatch; ++b) acc[b] = 0.f;
  for (int c0 = lane; c0 < chunks; c0 += 64) {
    const int c1 = c0 + 32;
    const uint4 wa = ldg_stream(row + c0);
    const uint4 wb = c1 < chunks ? ldg_stream(row + c1) : make_uint4(0, 0, 0, 0);
    const float4 wa0 = make_float4(bf16_lo(wa.x), bf16_hi(wa.x), bf16_lo(wa.y), bf16_hi(wa.y));
    const float4 wa1 = make_float4(bf16_lo(wa.z), bf16_hi(wa.z), bf16_lo(wa.w), bf16_hi(wa.w));
    const float4 wb0 = make_float4(bf16_lo(wb.x), bf16_hi(wb.x), bf16_lo(wb.y), bf16_hi(wb.y));
    const float4 wb1 = make_float4(bf16_lo(wb.z), bf16_hi(wb.z), bf16_lo(wb.w), bf16_hi(wb.w));
#pragma unroll
    for (int b = 0; b < kMaxBatch; ++b) {
      if (b < B) {
        acc[b] = dot8(xsm[(size_t)b * chunks + c0], wa0, wa1, acc[b]);
        if (c1 < chunks) acc[b] = dot8(xsm[(size_t)b * chunks + c1], wb0, wb1, acc[b]);
      }
    }
  }
#pragma unroll
  for (int b = 0; b < kMaxBatch; ++b) {
    const float v = warp_sum(acc[b]);
    if (lane == 0 && b < B) hidden[(size_t)b * H + warp] = fmaxf(v, 0.f);
  }
}

cudaError_t launch_pred_l1(const Dims& d, const void* w1, const void* x_bf16, int B, float* hidden,
                           cudaStream_t s) {
  const int threads = 128;
  const int blocks = (d.H * 32 + threads - 1) / threads;
  const uint4* w = static_cast<const uint4*>(w1);
  const uint4* x = static_cast<const uint4*>(x_bf16);
  if (B == 1)
    k_pred_l1_row<<<d.H, threads, 0, s>>>(w, x, hidden, d.H, d.D);
  else if (B <= 4)
    k_pred_l1<4><<<blocks, threads, 0, s>>>(w, x, hidden, d.H, d.D, B);
  else {
    const size_t sm = (size_t)B * d.D * 2;
    if (sm <= 200 * 1024) {
      cudaError_t e = cudaFuncSetAttribute(k_pred_l1_batch, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
      if (e != cudaSuccess) return e;
      k_pred_l1_batch<<<blocks, threads, sm, s>>>(w, x, hidden, d.H, d.D, B);
    } else {
      k_pred_l1<16><<<blocks, threads, 0, s>>>(w, x, hidden, d.H, d.D, B);
    }
  }
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Layer 2: logits[b][r] = sum_m W2[r][m] * hidden[b][m] for all L*M rows.
//
// W2 is one contiguous array that is read exactly once, so each block streams
// its contiguous share of rows through a ring of shared-memory stages filled by
// 1-D bulk copies (one producer warp, mbarrier full/empty pairs).  Nothing but
// the ring's size limits the bytes in flight per SM, and no register is spent
// on loads.  Consumer warps read rows from shared memory: LPR lanes share a row
// (a quarter-warp reads 128 contiguous bytes: conflict-free), each lane owns CPL
// 16-byte chunks; for one sequence the lane's slice of `hidden` stays in
// registers, for several it is read from shared memory.
// ---------------------------------------------------------------------------
constexpr int kL2ConsumerWarps = 8;
constexpr int kL2Threads = (kL2ConsumerWarps + 1) * 32;
constexpr int kL2MaxStages = 8;

template <int LPR, int CPL, int NB>
__global__ void __launch_bounds__(kL2Threads, 1) k_pred_l2(const uint4* __restrict__ w2,
                                                            const float* hidden,  // [B][H]; written by the previous kernel
                                                            float* __restrict__ logits,        // [B][rows]
                                                            long long rows, int H, int B, int stage_rows,
                                                            int n_stages, int32_t* status) {
  extern __shared__ __align__(128) unsigned char l2sm[];
  __shared__ __align__(8) uint64_t full_bar[kL2MaxStages];
  __shared__ __align__(8) uint64_t empty_bar[kL2MaxStages];
  constexpr int RPW = 32 / LPR;  // rows per warp pass
  const int chunks = H >> 3;
  const uint32_t row_bytes = (uint32_t)H * 2u;
  const uint32_t stage_bytes = (uint32_t)stage_rows * row_bytes;
  unsigned char* ring = l2sm;
  float* hs = reinterpret_cast<float*>(l2sm + (size_t)n_stages * stage_bytes);  // [NB][H] when NB > 1

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  // this block's contiguous share of rows
  const long long r_begin = rows * blockIdx.x / gridDim.x;
  const long long r_end = rows * (blockIdx.x + 1) / gridDim.x;
  const int n_iter = (int)((r_end - r_begin + stage_rows - 1) / stage_rows);

  if (tid == 0) {
    for (int s = 0; s < n_stages; ++s) {
      npp::mbar_init(&full_bar[s], 1);
      npp::mbar_init(&empty_bar[s], kL2ConsumerWarps);
    }
    npp::fence_barrier_init();
  }
  __syncthreads();

  if (wid == kL2ConsumerWarps) {
    // ---------------- producer warp: one lane issues the bulk copies ----------------
    if (lane == 0) {
      const uint64_t pol = npp::policy_evict_first();
      for (int it = 0; it < n_iter; ++it) {
        const int s = it % n_stages;
        const uint32_t ph = (uint32_t)(it / n_stages) & 1u;
        if (!npp::mbar_wait(&empty_bar[s], ph ^ 1u)) {
          atomicOr(status, npp::kStatTimeout);
          break;
        }
        const long long r0 = r_begin + (long long)it * stage_rows;
        const uint32_t nrows = (uint32_t)min((long long)stage_rows, r_end - r0);
        const uint32_t bytes = nrows * row_bytes;
        npp::mbar_expect_tx(&full_bar[s], bytes);
        npp::bulk_g2s_stream(ring + (size_t)s * stage_bytes, reinterpret_cast<const unsigned char*>(w2) + (size_t)r0 * row_bytes,
                             bytes, &full_bar[s], pol);
      }
    }
    return;
  }

  // ---------------- consumer warps ----------------
  // the weights above do not depend on the previous kernel; `hidden` does
  npp::pdl_wait_prior();
  const int sub = lane % LPR, rsel = lane / LPR;
  float hreg[NB == 1 ? CPL * 8 : 1];
  if (NB == 1) {
#pragma unroll
    for (int i = 0; i < CPL; ++i) {
      const int c = sub + i * LPR;
#pragma unroll
      for (int e = 0; e < 8; ++e) hreg[NB == 1 ? i * 8 + e : 0] = c < chunks ? hidden[c * 8 + e] : 0.f;
    }
  } else {
    for (int i = tid; i < B * H; i += kL2ConsumerWarps * 32) hs[i] = hidden[i];
    asm volatile("bar.sync 1, %0;" ::"n"(kL2ConsumerWarps * 32) : "memory");  // consumers only
  }

  for (int it = 0; it < n_iter; ++it) {
    const int s = it % n_stages;
    const uint32_t ph = (uint32_t)(it / n_stages) & 1u;
    if (!npp::mbar_wait(&full_bar[s], ph)) {
      if (lane == 0) atomicOr(status, npp::kStatTimeout);
      break;
    }
    const long long r0 = r_begin + (long long)it * stage_rows;
    const int nrows = (int)min((long long)stage_rows, r_end - r0);
    const unsigned char* st = ring + (size_t)s * stage_bytes;
    for (int g = wid * RPW; g < nrows; g += kL2ConsumerWarps * RPW) {
      const int rl = g + rsel;
      const bool live = rl < nrows;
      const uint4* row = reinterpret_cast<const uint4*>(st + (size_t)(live ? rl : 0) * row_bytes);
      float acc[NB];
#pragma unroll
      for (int b = 0; b < NB; ++b) acc[b] = 0.f;
#pragma unroll
      for (int i = 0; i < CPL; ++i) {
        const int c = sub + i * LPR;
        if (c < chunks) {
          const uint4 w = row[c];
          if (NB == 1) {
            const float4 ha = make_float4(hreg[NB == 1 ? i * 8 + 0 : 0], hreg[NB == 1 ? i * 8 + 1 : 0],
                                          hreg[NB == 1 ? i * 8 + 2 : 0], hreg[NB == 1 ? i * 8 + 3 : 0]);
            const float4 hb = make_float4(hreg[NB == 1 ? i * 8 + 4 : 0], hreg[NB == 1 ? i * 8 + 5 : 0],
                                          hreg[NB == 1 ? i * 8 + 6 : 0], hreg[NB == 1 ? i * 8 + 7 : 0]);
            acc[0] = dot8(w, ha, hb, acc[0]);
          } else {
#pragma unroll
            for (int b = 0; b < NB; ++b) {
              if (b < B) {
                const float4* hp = reinterpret_cast<const float4*>(hs + (size_t)b * H + c * 8);
                acc[b] = dot8(w, hp[0], hp[1], acc[b]);
              }
            }
          }
        }
      }
#pragma unroll
      for (int b = 0; b < NB; ++b) {
        float v = acc[b];
#pragma unroll
        for (int o = LPR / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (sub == 0 && live && b < B) logits[(size_t)b * rows + r0 + rl] = v;
      }
    }
    __syncwarp();
    if (lane == 0) npp::mbar_arrive(&empty_bar[s]);  // this warp is done reading the stage
  }
}

// Ring geometry of k_pred_l2 for rows of H values, B sequences and LPR lanes per row: a stage is
// about 32 KB of whole rows (a multiple of the rows one pass of all consumer warps covers); the
// hidden vectors of a batch sit beside the ring.  False when they and two stages do not fit.
static bool l2_ring_plan(int H, int B, int lpr, int* stage_rows_out, int* n_stages_out) {
  const long long row_bytes = (long long)H * 2;
  const int pass_rows = kL2ConsumerWarps * (32 / lpr);
  int stage_rows = (int)std::max<long long>(1, 32768 / row_bytes);
  stage_rows = std::max(pass_rows, stage_rows / pass_rows * pass_rows);
  const long long stage_bytes = stage_rows * row_bytes;
  const long long hs_bytes = B > 1 ? (long long)B * H * 4 : 0;
  const long long n = std::min<long long>(kL2MaxStages, (200 * 1024 - hs_bytes) / stage_bytes);  // signed: may be <= 0
  if (n < 2) return false;
  *stage_rows_out = stage_rows;
  *n_stages_out = (int)n;
  return true;
}
static int l2_ring_lpr(int chunks) { return chunks <= 1 ? 1 : chunks <= 2 ? 2 : chunks <= 4 ? 4 : chunks <= 96 ? 8 : chunks <= 128 ? 16 : 32; }

bool pred_l2_ring_fits(int H, int B) {
  int a, b;
  return l2_ring_plan(H, B, l2_ring_lpr(H >> 3), &a, &b);
}

template <int LPR, int CPL>
static cudaError_t l2_dispatch_nb(const uint4* w2, const float* hidden, float* logits, long long rows,
                                  int H, int B, int blocks, int32_t* status, cudaStream_t s) {
  int stage_rows = 0, n_stages = 0;
  if (!l2_ring_plan(H, B, LPR, &stage_rows, &n_stages)) return cudaErrorInvalidValue;
  const size_t stage_bytes = (size_t)stage_rows * H * 2;
  const size_t hs_bytes = B > 1 ? (size_t)B * H * 4 : 0;
  const size_t sm = (size_t)n_stages * stage_bytes + hs_bytes;

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(blocks);
  cfg.blockDim = dim3(kL2Threads);
  cfg.dynamicSmemBytes = sm;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
#define NP_L2_LAUNCH(NBV)                                                                             \
  do {                                                                                                \
    auto kfn = k_pred_l2<LPR, CPL, NBV>;                                                              \
    cudaError_t e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);  \
    if (e != cudaSuccess) return e;                                                                   \
    return cudaLaunchKernelEx(&cfg, kfn, w2, hidden, logits, rows, H, B, stage_rows, n_stages, status); \
  } while (0)
  if (B == 1) NP_L2_LAUNCH(1);
  if (B <= 4) NP_L2_LAUNCH(4);
  NP_L2_LAUNCH(16);
#undef NP_L2_LAUNCH
}

// ---------------------------------------------------------------------------
// Layer 2 for one sequence, without the ring: LPR lanes share a row, each lane
// keeps its CPL 16-byte chunks of `hidden` in registers for the whole kernel
// and loads its chunks of RIF rows straight from global memory into registers
// before it uses any (16 loads in flight per lane at H = 512); a shuffle
// reduction per row, no shared memory, no barrier.  The hand-over per ring
// stage (mbarrier polls, one stage at a time per warp) held the ring kernel at
// 0.65 of the copy bandwidth; this one streams like a copy.
// The first loads go out before the wait for layer 1: the weights do not depend
// on it, `hidden` does.
// ---------------------------------------------------------------------------
constexpr int kL2dWarps = 16;
constexpr int kL2dThreads = kL2dWarps * 32;

template <int LPR, int CPL>
__global__ void __launch_bounds__(kL2dThreads, 1) k_pred_l2_direct(const uint4* __restrict__ w2,
                                                                   const float* hidden,  // [H]; written by the previous kernel
                                                                   float* __restrict__ logits, long long rows, int H) {
  constexpr int RPW = 32 / LPR;                           // rows a warp works on side by side
  constexpr int RIF = CPL >= 16 ? 1 : (CPL >= 8 ? 2 : (CPL >= 4 ? 4 : 8));  // rows in flight per lane
  constexpr int kGroup = RPW * RIF;                       // rows per warp and iteration
  const int chunks = H >> 3;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int sub = lane % LPR, rsel = lane / LPR;
  const long long r_begin = rows * blockIdx.x / gridDim.x;
  const long long r_end = rows * (blockIdx.x + 1) / gridDim.x;
  uint4 w[RIF][CPL];
  // every load is issued, unconditionally: indices past the end are clamped, their results dropped
  auto load = [&](long long base) {
#pragma unroll
    for (int u = 0; u < RIF; ++u) {
      const long long r = min(base + u * RPW + rsel, r_end - 1);
      const uint4* row = w2 + (size_t)r * chunks;
#pragma unroll
      for (int i = 0; i < CPL; ++i) w[u][i] = ldg_stream(row + min(sub + i * LPR, chunks - 1));
    }
  };
  long long base = r_begin + (long long)wid * kGroup;
  if (base < r_end) load(base);
  npp::pdl_wait_prior();
  npp::pdl_launch_dependents();  // the selection's blocks take the SMs as this grid's blocks leave them
  float hreg[CPL * 8];
#pragma unroll
  for (int i = 0; i < CPL; ++i) {
    const int c = sub + i * LPR;
#pragma unroll
    for (int e = 0; e < 8; ++e) hreg[i * 8 + e] = c < chunks ? hidden[c * 8 + e] : 0.f;
  }
  while (base < r_end) {
    float acc[RIF];
#pragma unroll
    for (int u = 0; u < RIF; ++u) {
      acc[u] = 0.f;
#pragma unroll
      for (int i = 0; i < CPL; ++i) {
        const float4 ha = make_float4(hreg[i * 8 + 0], hreg[i * 8 + 1], hreg[i * 8 + 2], hreg[i * 8 + 3]);
        const float4 hb = make_float4(hreg[i * 8 + 4], hreg[i * 8 + 5], hreg[i * 8 + 6], hreg[i * 8 + 7]);
        acc[u] = dot8(w[u][i], ha, hb, acc[u]);  // chunks past the row's end meet zeros of `hidden`
      }
    }
    // the sums are complete before the registers of w are loaded again (the compiler would
    // otherwise keep both generations of w alive, and spill)
#pragma unroll
    for (int u = 0; u < RIF; ++u) asm volatile("" : "+f"(acc[u]));
    const long long cur = base;
    base += (long long)kL2dWarps * kGroup;
    if (base < r_end) load(base);  // the next rows are on their way while these are reduced and stored
#pragma unroll
    for (int u = 0; u < RIF; ++u) {
      float v = acc[u];
#pragma unroll
      for (int o = LPR / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      const long long r = cur + u * RPW + rsel;
      if (sub == 0 && r < r_end) logits[r] = v;
    }
  }
}

template <int LPR, int CPL>
static cudaError_t l2_direct_launch(const uint4* w2, const float* hidden, float* logits, long long rows, int H,
                                    int blocks, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(blocks);
  cfg.blockDim = dim3(kL2dThreads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k_pred_l2_direct<LPR, CPL>, w2, hidden, logits, rows, H);
}

cudaError_t launch_pred_l2(const Dims& d, const void* w2v, const float* hidden, int B, float* logits,
                           int32_t* status, cudaStream_t s, int sm_count) {
  const uint4* w2 = static_cast<const uint4*>(w2v);
  const long long rows = (long long)d.L * d.M;
  const int chunks = d.H >> 3;
  const int blocks = sm_count;
  if (B == 1 && rows > 0) {
#define NP_L2D(LPR, CPL) return l2_direct_launch<LPR, CPL>(w2, hidden, logits, rows, d.H, blocks, s)
    if (chunks <= 1) NP_L2D(1, 1);
    if (chunks <= 2) NP_L2D(2, 1);
    if (chunks <= 4) NP_L2D(4, 1);
    if (chunks <= 8) NP_L2D(8, 1);
    if (chunks <= 16) NP_L2D(16, 1);
    if (chunks <= 32) NP_L2D(16, 2);
    if (chunks <= 64) NP_L2D(16, 4);
    if (chunks <= 128) NP_L2D(32, 4);
    // wider hidden vectors do not fit a lane's registers beside its loads: the ring kernel below
#undef NP_L2D
  }
#define NP_L2(LPR, CPL) return l2_dispatch_nb<LPR, CPL>(w2, hidden, logits, rows, d.H, B, blocks, status, s)
  if (chunks <= 1) NP_L2(1, 1);
  if (chunks <= 2) NP_L2(2, 1);
  if (chunks <= 4) NP_L2(4, 1);
  if (chunks <= 8) NP_L2(8, 1);
  if (chunks <= 16) NP_L2(8, 2);
  if (chunks <= 32) NP_L2(8, 4);
  if (chunks <= 64) NP_L2(8, 8);
  if (chunks <= 96) NP_L2(8, 12);
  if (chunks <= 128) NP_L2(16, 8);
  if (chunks <= 256) NP_L2(32, 8);
  if (chunks <= 512) NP_L2(32, 16);
#undef NP_L2
  return cudaErrorInvalidValue;  // H > 4096 is rejected by np_init
}

// ---------------------------------------------------------------------------
// Self-test of the bounded waits: one thread waits on an mbarrier that nothing
// ever arrives at.  The wait gives up after kSpinLimit polls and records
// kStatTimeout; the kernel returns normally.
// ---------------------------------------------------------------------------
__global__ void k_selftest_wait(int32_t* status) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    npp::mbar_init(&bar, 1);
    npp::fence_barrier_init();
    if (!npp::mbar_wait(&bar, 0)) atomicOr(status, npp::kStatTimeout);
  }
}

cudaError_t launch_selftest_wait(int32_t* status, cudaStream_t s) {
  k_selftest_wait<<<1, 32, 0, s>>>(status);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// small elementwise helpers of the residual chain
// ---------------------------------------------------------------------------
__global__ void k_widen_bf16(const uint16_t* __restrict__ x, float* __restrict__ out, size_t n) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = __uint_as_float((uint32_t)x[i] << 16);
}

__global__ void k_add_vec(const float* __restrict__ a, const float* __restrict__ b, int reps,
                          float* __restrict__ out, size_t n) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) {
    float v = a[i];
    for (int r = 0; r < reps; ++r) v += b[(size_t)r * n + i];
    out[i] = v;
  }
}

cudaError_t launch_widen_bf16(const void* x_bf16, float* out, size_t n, cudaStream_t s) {
  k_widen_bf16<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(static_cast<const uint16_t*>(x_bf16), out, n);
  return cudaGetLastError();
}

cudaError_t launch_add_vec(const float* a, const float* b, int reps, float* out, size_t n, cudaStream_t s) {
  k_add_vec<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(a, b, reps, out, n);
  return cudaGetLastError();
}

}  // namespace npi
