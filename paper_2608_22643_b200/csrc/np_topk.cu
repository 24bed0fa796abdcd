// Stage 2: per-layer top-k of the predictor's logits -> active-neuron bitmap.
// (The paper turns predictor outputs into one active set per layer, Section 3.4;
// here the set is the k highest-scoring neurons, the K_max budget of Section 4.1.)
//
// One block of 1024 threads per (layer, sequence).  A layer is only 44 KB of logits: the
// kernel is a chain of block-wide steps on one SM, and what it costs is the instructions of
// those steps.  Every thread keeps its logits in registers, index tid + 1024 j, so that the 32
// lanes of a warp hold the 32 neurons of one bitmap word and a ballot is a word.
//
// Fast path (finite logits that are not all equal): ONE histogram pass over 2048 bins that
// are linear in the logit's value, bin = floor((z - min) * 2047 / (max - min)).  Every step of
// that formula is monotone in z, so the bins are ordered like the keys and every key above
// the bin of the k-th largest belongs to the set; values spread over the bins like their
// density, so the adds to shared memory rarely meet (a radix digit of the float's bits puts
// most of a layer into a handful of bins: sign and exponent are shared).  The few keys inside
// that one bin are listed and ranked against each other exactly, by (key, then lower index).
//
// General path (an infinity or NaN among the logits, a degenerate range, or more than 1024
// keys in the deciding bin, i.e. heavy ties): a radix select on the order-preserving uint32
// image of the fp32 bits, 8 + 12 + 12 bits; the first digit counts into one histogram per warp.
// Both paths select the same set: the k largest keys, ties broken towards the lower index.
#include "np_device.cuh"
#include "np_internal.h"
#include "np_pipe.cuh"

namespace npi {
using namespace npd;

constexpr int kTopkThreads = 1024;
constexpr int kTopkHist = 8192;   // ints: 32 warps x 256 bins in the first radix pass, 4096 bins after; 2048 linear bins + candidate list
constexpr int kLinBins = 2048;
constexpr int kMaxCand = 1024;    // keys of the deciding bin that are ranked directly

#ifdef NP_TRACE  // development builds only: clock stamps of one block
__device__ long long np_tk_clk[32];
extern "C" int np_debug_tk(void* out) { return (int)cudaMemcpyFromSymbol(out, np_tk_clk, sizeof(np_tk_clk)); }
#define TK(ev) do { if (blockIdx.x == 5 && blockIdx.y == 0 && threadIdx.x == 0) np_tk_clk[ev] = clock64(); } while (0)
#else
#define TK(ev) do { } while (0)
#endif

// bit pattern of an fp32 value -> order-preserving uint32 (larger float, larger key; +0 above -0)
__device__ __forceinline__ uint32_t order_key(uint32_t b) { return (b & 0x80000000u) ? ~b : (b | 0x80000000u); }

// KPT: keys per thread, ceil(M / 1024)
template <int KPT>
__global__ void __launch_bounds__(kTopkThreads) k_topk(const float* __restrict__ logits,  // [B][L][M]
                                                       uint32_t* __restrict__ bitmap,     // [L][W]
                                                       int L, int M, int k, int use_atomic) {
  extern __shared__ __align__(16) int wsm[];  // [W] per word: selected keys of the deciding bin / count of threshold-equal keys
  __shared__ __align__(16) int hist[kTopkHist];
  __shared__ int wsum[33];
  __shared__ float wlo[32], whi[32];
  __shared__ uint32_t s_prefix;
  __shared__ int s_remaining, s_bin_count, s_bin, s_ncand;

  const int W = M >> 5;
  const int layer = blockIdx.x, b = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const float* z = logits + ((size_t)b * L + layer) * M;
  uint32_t* out = bitmap + (size_t)layer * W;

  TK(0);
  npp::pdl_launch_dependents();
  npp::pdl_wait_prior();  // the logits are the previous kernel's
  TK(1);

  if (k <= 0) {  // nothing selected
    if (!use_atomic)
      for (int w = tid; w < W; w += kTopkThreads) out[w] = 0u;
    return;
  }
  if (k >= M) {
    for (int w = tid; w < W; w += kTopkThreads) {
      if (use_atomic) atomicOr(out + w, 0xffffffffu);
      else out[w] = 0xffffffffu;
    }
    return;
  }

  // The logits are kept as bit patterns: the keys must be exact, and floating-point moves under flush-to-zero
  // arithmetic need not preserve a denormal.  Only the fast path's bin arithmetic looks at them as numbers.
  uint32_t zb[KPT];
  float lo = __int_as_float(0x7f800000), hi = __int_as_float(0xff800000);
  int bad = 0;
  const uint32_t* zbits = reinterpret_cast<const uint32_t*>(z);
#pragma unroll
  for (int j = 0; j < KPT; ++j) {
    const int i = tid + kTopkThreads * j;
    zb[j] = i < M ? zbits[i] : 0u;  // entries past the layer's end are never counted (every use tests the index)
  }
#pragma unroll
  for (int j = 0; j < KPT; ++j) {
    if (tid + kTopkThreads * j < M) {
      bad |= (zb[j] & 0x7f800000u) == 0x7f800000u;  // infinity or NaN
      lo = fminf(lo, __uint_as_float(zb[j]));
      hi = fmaxf(hi, __uint_as_float(zb[j]));
    }
  }
  hist[tid] = 0;
  hist[tid + kTopkThreads] = 0;
  for (int w = tid; w < W; w += kTopkThreads) wsm[w] = 0;
  if (tid == 0) s_ncand = 0;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
    hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
  }
  if (lane == 0) {
    wlo[wid] = lo;
    whi[wid] = hi;
  }
  TK(2);
  const int any_bad = __syncthreads_or(bad);
  lo = wlo[lane];
  hi = whi[lane];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
    hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
  }
  const float range = hi - lo;
  const float scale = (float)(kLinBins - 1) / range;
  // block-uniform: every thread holds the same lo, hi and flags
  const bool linear = !any_bad && range > 0.f && (__float_as_uint(range) & 0x7f800000u) != 0x7f800000u &&
                      (__float_as_uint(scale) & 0x7f800000u) != 0x7f800000u;
  TK(3);
  if (linear) {
    auto bin_of = [&](float v) { return min(kLinBins - 1, (int)((v - lo) * scale)); };
#pragma unroll
    for (int j = 0; j < KPT; ++j)
      if (tid + kTopkThreads * j < M) atomicAdd(&hist[bin_of(__uint_as_float(zb[j]))], 1);
    __syncthreads();
    TK(4);
    // the bin of the k-th largest key: thread t takes the two highest bins not taken by the threads below it
    const int top = kLinBins - 1 - 2 * tid;
    const int c_hi = hist[top], c_lo = hist[top - 1];
    const int mine = c_hi + c_lo;
    const int above = block_inclusive_scan_1024(mine, wsum, lane, wid) - mine;  // keys in higher bins
    if (above < k && k <= above + mine) {  // exactly one thread
      const bool first = k <= above + c_hi;
      s_bin = first ? top : top - 1;
      s_remaining = k - (first ? above : above + c_hi);
      s_bin_count = first ? c_hi : c_lo;
    }
    __syncthreads();
    TK(5);
    const int bstar = s_bin, need = s_remaining, ncand = s_bin_count;
    if (ncand <= kMaxCand) {  // block-uniform
      uint32_t* ckey = reinterpret_cast<uint32_t*>(hist + kLinBins);
      int* cidx = hist + kLinBins + kMaxCand;
      // one pass: the words of the keys above the bin go out, the keys inside it are listed
#pragma unroll
      for (int j = 0; j < KPT; ++j) {
        const int i = tid + kTopkThreads * j;
        const int w = wid + 32 * j;  // the word of neurons 32 w .. 32 w + 31: this warp's logits of round j
        const int bn = i < M ? bin_of(__uint_as_float(zb[j])) : -1;
        const uint32_t gt = __ballot_sync(0xffffffffu, bn > bstar);
        if (lane == 0 && w < W) {
          if (use_atomic) {
            if (gt) atomicOr(out + w, gt);
          } else {
            out[w] = gt;
          }
        }
        if (bn == bstar) {
          const int q = atomicAdd(&s_ncand, 1);
          ckey[q] = order_key(zb[j]);
          cidx[q] = i;
        }
      }
      __syncthreads();  // the list is complete; the words stored above are ordered before the bits added below
      TK(6);
      if (tid < ncand) {  // rank among the keys of the bin: larger key first, then lower index
        const uint32_t mk = ckey[tid];
        const int mi = cidx[tid];
        int rank = 0;
        for (int q = 0; q < ncand; ++q) {
          const uint32_t qk = ckey[q];
          rank += (qk > mk || (qk == mk && cidx[q] < mi)) ? 1 : 0;
        }
        if (rank < need) atomicOr(out + (mi >> 5), 1u << (mi & 31));
      }
      TK(16);
      return;
    }
    __syncthreads();  // heavy ties: the general path reuses the histogram and the per-word array
    for (int w = tid; w < W; w += kTopkThreads) wsm[w] = 0;
  }

  // ---- general path: radix select on the keys --------------------------------------------
  if (tid == 0) {
    s_prefix = 0u;
    s_remaining = k;
  }
  uint32_t mask = 0u;
#pragma unroll 1
  for (int pass = 0; pass < 3; ++pass) {
    const int shift = pass == 0 ? 24 : (pass == 1 ? 12 : 0);
    const uint32_t dmask = pass == 0 ? 0xffu : 0xfffu;
    // pass 0: one histogram of 256 bins per warp (8192 ints); passes 1 and 2: one of 4096 bins
    int4* h4 = reinterpret_cast<int4*>(hist);
    __syncthreads();
    h4[tid] = make_int4(0, 0, 0, 0);
    if (pass == 0) h4[tid + kTopkThreads] = make_int4(0, 0, 0, 0);
    __syncthreads();
    const uint32_t prefix = s_prefix;
    const int remaining = s_remaining;
    int* my_hist = pass == 0 ? hist + wid * 256 : hist;
#pragma unroll
    for (int j = 0; j < KPT; ++j) {
      const uint32_t key = order_key(zb[j]);
      const bool in = tid + kTopkThreads * j < M && (key & mask) == prefix;
      // lanes with the same digit add once
      const uint32_t d = in ? (key >> shift) & dmask : 0xffffffffu;
      const uint32_t peers = __match_any_sync(0xffffffffu, d);
      if (in && lane == __ffs(peers) - 1) atomicAdd(&my_hist[d], __popc(peers));
    }
    __syncthreads();
    // the bin of the remaining-th largest key: thread t takes the highest bins not taken by the threads below it
    int c[4] = {0, 0, 0, 0};
    int top;
    if (pass == 0) {
      top = 255 - tid;
      if (tid < 256) {
#pragma unroll 8
        for (int w = 0; w < 32; ++w) c[0] += hist[w * 256 + top];
      }
    } else {
      top = 4095 - 4 * tid;
      const int4 v = h4[1023 - tid];  // bins top - 3 .. top
      c[0] = v.w;
      c[1] = v.z;
      c[2] = v.y;
      c[3] = v.x;
    }
    const int mine = c[0] + c[1] + c[2] + c[3];
    const int above = block_inclusive_scan_1024(mine, wsum, lane, wid) - mine;  // keys with a higher digit
    if (above < remaining && remaining <= above + mine) {  // exactly one thread
      int acc = above, bin = top, cnt = c[0];
#pragma unroll
      for (int i = 0; i < 3; ++i) {
        if (remaining > acc + c[i] && bin == top - i) {
          acc += c[i];
          bin = top - i - 1;
          cnt = c[i + 1];
        }
      }
      s_prefix = prefix | ((uint32_t)bin << shift);
      s_remaining = remaining - acc;
      s_bin_count = cnt;
    }
    mask |= dmask << shift;
    __syncthreads();
  }

  const uint32_t thr = s_prefix;   // key of the k-th largest element
  const int admit = s_remaining;   // how many keys equal to thr are taken, lowest index first
  const bool surplus = s_bin_count > admit;  // more keys equal to thr than fit: rank them by index

  if (surplus) {  // block-uniform: ranks of the equal keys in index order
#pragma unroll
    for (int j = 0; j < KPT; ++j) {
      const int w = wid + 32 * j;
      const uint32_t eq = __ballot_sync(0xffffffffu, tid + kTopkThreads * j < M && order_key(zb[j]) == thr);
      if (lane == 0 && w < W) wsm[w] = __popc(eq);
    }
    block_exclusive_scan(wsm, W, hist);
  }
#pragma unroll
  for (int j = 0; j < KPT; ++j) {
    const int w = wid + 32 * j;
    const bool valid = tid + kTopkThreads * j < M;
    const uint32_t key = order_key(zb[j]);
    const uint32_t gt = __ballot_sync(0xffffffffu, valid && key > thr);
    const uint32_t eq = __ballot_sync(0xffffffffu, valid && key == thr);
    if (lane == 0 && w < W) {
      const uint32_t word = gt | (surplus ? lowest_bits(eq, admit - wsm[w]) : eq);
      if (use_atomic) {
        if (word) atomicOr(out + w, word);
      } else {
        out[w] = word;
      }
    }
  }
}

template <int KPT>
static cudaError_t topk_launch(const Dims& d, const float* logits, int B, uint32_t* bitmap, int use_atomic, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(d.L, B);
  cfg.blockDim = dim3(kTopkThreads);
  cfg.dynamicSmemBytes = (size_t)d.W * 4;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // its prologue overlaps the predictor's tail
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k_topk<KPT>, logits, bitmap, d.L, d.M, d.k, use_atomic);
}

cudaError_t launch_topk(const Dims& d, const float* logits, int B, uint32_t* bitmap, cudaStream_t s) {
  const int use_atomic = B > 1 ? 1 : 0;
  if (use_atomic) {
    cudaError_t e = cudaMemsetAsync(bitmap, 0, (size_t)d.L * d.W * 4, s);
    if (e != cudaSuccess) return e;
  }
  const int kpt = (d.M + kTopkThreads - 1) / kTopkThreads;
  if (kpt <= 12) return topk_launch<12>(d, logits, B, bitmap, use_atomic, s);
  if (kpt <= 16) return topk_launch<16>(d, logits, B, bitmap, use_atomic, s);
  if (kpt <= 28) return topk_launch<28>(d, logits, B, bitmap, use_atomic, s);
  if (kpt <= 40) return topk_launch<40>(d, logits, B, bitmap, use_atomic, s);
  return cudaErrorInvalidValue;  // d_ffn > 40960 is rejected by np_init
}

}  // namespace npi
