// Stage 1: predictor forward, logits = W2 * relu(W1 * x)  (one pass after
// layer 0 scores every FFN neuron of every downstream layer; Section 3.1 step 2).
//
// Both layers are matrix-vector products at small batch: every weight byte is
// read once, so the kernels are organised around 16-byte coalesced streaming
// loads with many loads in flight per thread, fp32 accumulation and
// warp-shuffle reductions.
#include "np_device.cuh"
#include "np_internal.h"

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

cudaError_t launch_pred_l1(const Dims& d, const void* w1, const void* x_bf16, int B, float* hidden,
                           cudaStream_t s) {
  const int threads = 128;
  const int blocks = (d.H * 32 + threads - 1) / threads;
  const uint4* w = static_cast<const uint4*>(w1);
  const uint4* x = static_cast<const uint4*>(x_bf16);
  if (B == 1)
    k_pred_l1<1><<<blocks, threads, 0, s>>>(w, x, hidden, d.H, d.D, B);
  else if (B <= 4)
    k_pred_l1<4><<<blocks, threads, 0, s>>>(w, x, hidden, d.H, d.D, B);
  else
    k_pred_l1<16><<<blocks, threads, 0, s>>>(w, x, hidden, d.H, d.D, B);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Layer 2: logits[b][r] = sum_m W2[r][m] * hidden[b][m] for all L*M rows.
// A row is short (H bf16), so LPR lanes share a row and a warp covers 32/LPR
// consecutive rows per pass; each lane keeps CPL 16-byte loads in flight.  For
// one sequence the lane's slice of `hidden` lives in registers.
// ---------------------------------------------------------------------------
template <int LPR, int CPL, int NB>
__global__ void __launch_bounds__(256) k_pred_l2(const uint4* __restrict__ w2,
                                                  const float* __restrict__ hidden,  // [B][H]
                                                  float* __restrict__ logits,        // [B][rows]
                                                  long long rows, int H, int B) {
  extern __shared__ __align__(16) float sh[];  // [NB][H] when NB > 1
  constexpr int RPW = 32 / LPR;                // rows per warp pass
  const int chunks = H >> 3;
  const int lane = threadIdx.x & 31;
  const int sub = lane % LPR;  // position inside the row
  const int rsel = lane / LPR;

  float hreg[NB == 1 ? CPL * 8 : 1];
  if (NB == 1) {
#pragma unroll
    for (int i = 0; i < CPL; ++i) {
      const int c = sub + i * LPR;
#pragma unroll
      for (int e = 0; e < 8; ++e) hreg[(NB == 1 ? i * 8 + e : 0)] = c < chunks ? hidden[c * 8 + e] : 0.f;
    }
  } else {
    for (int i = threadIdx.x; i < B * H; i += blockDim.x) sh[i] = hidden[i];
    __syncthreads();
  }

  const long long warps_total = (long long)gridDim.x * (blockDim.x >> 5);
  const long long wglobal = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long passes = (rows + RPW - 1) / RPW;
  // contiguous range of passes per warp keeps each warp streaming through one region
  const long long per = (passes + warps_total - 1) / warps_total;
  const long long p0 = wglobal * per, p1 = min(passes, p0 + per);

  for (long long p = p0; p < p1; ++p) {
    const long long r = p * RPW + rsel;
    const bool live = r < rows;
    const uint4* row = w2 + (size_t)(live ? r : 0) * chunks;
    uint4 w[CPL];
#pragma unroll
    for (int i = 0; i < CPL; ++i) {
      const int c = sub + i * LPR;
      w[i] = (live && c < chunks) ? ldg_stream(row + c) : make_uint4(0, 0, 0, 0);
    }
    float acc[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) acc[b] = 0.f;
    if (NB == 1) {
#pragma unroll
      for (int i = 0; i < CPL; ++i) {
        const float4 ha = make_float4(hreg[i * 8 + 0], hreg[i * 8 + 1], hreg[i * 8 + 2], hreg[i * 8 + 3]);
        const float4 hb = make_float4(hreg[i * 8 + 4], hreg[i * 8 + 5], hreg[i * 8 + 6], hreg[i * 8 + 7]);
        acc[0] = dot8(w[i], ha, hb, acc[0]);
      }
    } else {
#pragma unroll
      for (int i = 0; i < CPL; ++i) {
        const int c = sub + i * LPR;
        if (c < chunks) {
#pragma unroll
          for (int b = 0; b < NB; ++b) {
            if (b < B) {
              const float4* hp = reinterpret_cast<const float4*>(sh + (size_t)b * H + c * 8);
              acc[b] = dot8(w[i], hp[0], hp[1], acc[b]);
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
      if (sub == 0 && live && b < B) logits[(size_t)b * rows + r] = v;
    }
  }
}

template <int LPR, int CPL>
static cudaError_t l2_dispatch_nb(const uint4* w2, const float* hidden, float* logits, long long rows,
                                  int H, int B, int blocks, cudaStream_t s) {
  const int threads = 256;
  if (B == 1) {
    k_pred_l2<LPR, CPL, 1><<<blocks, threads, 0, s>>>(w2, hidden, logits, rows, H, B);
  } else if (B <= 4) {
    k_pred_l2<LPR, CPL, 4><<<blocks, threads, (size_t)B * H * 4, s>>>(w2, hidden, logits, rows, H, B);
  } else {
    const size_t sm = (size_t)B * H * 4;
    auto kfn = k_pred_l2<LPR, CPL, 16>;
    if (sm > 48 * 1024) {
      cudaError_t e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
      if (e != cudaSuccess) return e;
    }
    kfn<<<blocks, threads, sm, s>>>(w2, hidden, logits, rows, H, B);
  }
  return cudaGetLastError();
}

cudaError_t launch_pred_l2(const Dims& d, const void* w2v, const float* hidden, int B, float* logits,
                           cudaStream_t s, int sm_count) {
  const uint4* w2 = static_cast<const uint4*>(w2v);
  const long long rows = (long long)d.L * d.M;
  const int chunks = d.H >> 3;
  const int blocks = sm_count * 4;
#define NP_L2(LPR, CPL) return l2_dispatch_nb<LPR, CPL>(w2, hidden, logits, rows, d.H, B, blocks, s)
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
// small elementwise helpers of the residual chain
// ---------------------------------------------------------------------------
__global__ void k_widen_bf16(const uint16_t* __restrict__ x, float* __restrict__ out, size_t n) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = __uint_as_float((uint32_t)x[i] << 16);
}

__global__ void k_add_vec(const float* __restrict__ a, const float* __restrict__ b,
                          float* __restrict__ out, size_t n) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = a[i] + b[i];
}

cudaError_t launch_widen_bf16(const void* x_bf16, float* out, size_t n, cudaStream_t s) {
  k_widen_bf16<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(static_cast<const uint16_t*>(x_bf16), out, n);
  return cudaGetLastError();
}

cudaError_t launch_add_vec(const float* a, const float* b, float* out, size_t n, cudaStream_t s) {
  k_add_vec<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(a, b, out, n);
  return cudaGetLastError();
}

}  // namespace npi
