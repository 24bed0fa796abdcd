// The shared predictor of Section 3.3 for one token: per-feature projection blocks
// (Linear -> LayerNorm -> SiLU), the centroid-ID branch (embedding row -> one such block), the
// residual trunk (z <- z + W2 SiLU(LayerNorm(W1 z + b1)) + b2) and the centroid heads (2 per
// sparse layer, K logits each).  Inference only: dropout is the identity.
//
// Every stage is a matrix-vector product over bf16 weights that are read once (414 MB in all at
// the paper's sizes, 260 MB of it the heads), so one kernel serves them all: k_gemv streams rows
// the way the dense-layer kernel does (a warp per row, 16-byte pieces loaded straight into
// registers, 16 in flight per lane, every load unconditional), with the input vector in shared
// memory.  The LayerNorm + SiLU between two linear layers is applied by the consumer as it loads
// its input (each block computes the two moments of the short vector itself), so a trunk block
// is two launches and nothing is synchronised across blocks inside a kernel.  The launches are
// chained by programmatic dependent launch: a kernel requests its first weights before it waits
// for the kernel that produces its input.
#include <algorithm>

#include "np_device.cuh"
#include "np_internal.h"
#include "np_pipe.cuh"

namespace npi {
using namespace npd;
namespace trunk {

constexpr int kWarps = 16;
constexpr int kThreads = kWarps * 32;
// a warp works on kRows rows side by side with kPieces 16-byte pieces of each in flight per lane:
// (2, 8) where there are rows enough for every warp of the device, (1, 16) for the short matrices
// of the trunk, so that they spread over all SMs and a row of 8 KB is one round of loads
constexpr int kMaxSegs = 8;
constexpr float kLnEps = 1e-5f;   // the LayerNorm epsilon (the paper does not state one)

struct Seg {
  const uint4* w;            // bf16 [rows][in_dim], in_dim a multiple of 8
  const float* b;            // [rows] or NULL
  const float* x;            // fp32 [in_dim]; NULL: the input is row *x_row of x_rows
  const uint16_t* x_rows;    // bf16 [n][in_dim]
  const int32_t* x_row;      // device scalar
  const float* ln_gain;      // non-NULL: the input is SiLU(LayerNorm(x; gain, bias))
  const float* ln_bias;
  const float* res;          // [rows] or NULL: y = res + W x + b
  float* y;                  // [rows]
  int rows, in_dim;
};
struct GemvArgs {
  Seg seg[kMaxSegs];  // blockIdx.y picks the segment
};

__device__ __forceinline__ float block_sum(float v, float* red) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) red[wid] = v;
  __syncthreads();
  float t = 0.f;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) t += red[w];
  return t;
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

template <int kRows, int kPieces>
__global__ void __launch_bounds__(kThreads, 1) k_gemv(GemvArgs a) {
  extern __shared__ __align__(16) float xs[];  // the input: even 4-float granules first, then the odd ones
  __shared__ float red[kWarps];
  const Seg& s = a.seg[blockIdx.y];
  const int in_dim = s.in_dim, chunks = in_dim >> 3, rows = s.rows;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  npp::pdl_launch_dependents();
  // rows are dealt to the warps of all blocks in groups of kRows
  const int warps_total = gridDim.x * kWarps;
  int r0 = (blockIdx.x * kWarps + wid) * kRows;
  uint4 w[kRows][kPieces];
  // every load is issued, unconditionally, before any is used; indices past the end are clamped
  auto load = [&](int row0, int p0) {
#pragma unroll
    for (int u = 0; u < kRows; ++u) {
      const uint4* row = s.w + (size_t)min(row0 + u, rows - 1) * chunks;
#pragma unroll
      for (int i = 0; i < kPieces; ++i) w[u][i] = ldg_stream(row + min(p0 + 32 * i, chunks - 1));
    }
  };
  if (r0 < rows) load(r0, lane);  // the weights do not depend on the previous kernel; the input does
  npp::pdl_wait_prior();

  // ---- the input vector, normalised and activated if asked for ----
  float mean = 0.f, rstd = 1.f;
  const bool ln = s.ln_gain != nullptr;
  const uint16_t* xr = s.x ? nullptr : s.x_rows + (size_t)(*s.x_row) * in_dim;
  auto xin = [&](int i) { return s.x ? __ldcg(s.x + i) : __uint_as_float((uint32_t)xr[i] << 16); };
  if (ln) {
    float t = 0.f;
    for (int i = tid; i < in_dim; i += kThreads) t += xin(i);
    mean = block_sum(t, red) / (float)in_dim;
    t = 0.f;
    for (int i = tid; i < in_dim; i += kThreads) {
      const float dv = xin(i) - mean;
      t += dv * dv;
    }
    rstd = rsqrtf(block_sum(t, red) / (float)in_dim + kLnEps);
  }
  for (int i = tid; i < in_dim; i += kThreads) {
    float v = xin(i);
    if (ln) {
      v = (v - mean) * rstd * s.ln_gain[i] + s.ln_bias[i];
      v = v / (1.f + __expf(-v));
    }
    const int g = i >> 2;  // granule
    xs[((g & 1) * chunks + (g >> 1)) * 4 + (i & 3)] = v;
  }
  __syncthreads();

  // ---- rows ----
  while (r0 < rows) {
    float acc[kRows];
#pragma unroll
    for (int u = 0; u < kRows; ++u) acc[u] = 0.f;
    const int cur = r0;
    // the trip count is the same for every lane (the loop advances r0 and is followed by
    // warp-wide shuffles): a lane whose pieces lie past the row's end works on clamped loads
    for (int pb = 0; pb < chunks; pb += 32 * kPieces) {
      const int p0 = pb + lane;
#pragma unroll
      for (int i = 0; i < kPieces; ++i) {
        const int p = p0 + 32 * i;
        if (p < chunks) {
          const float4 x0 = reinterpret_cast<const float4*>(xs)[p];
          const float4 x1 = reinterpret_cast<const float4*>(xs)[chunks + p];
#pragma unroll
          for (int u = 0; u < kRows; ++u) acc[u] = dot8(w[u][i], x0, x1, acc[u]);
        }
      }
      // the sums are complete before the registers of w are loaded again (the compiler would
      // otherwise keep both generations of w alive, and spill)
#pragma unroll
      for (int u = 0; u < kRows; ++u) asm volatile("" : "+f"(acc[u]));
      if (pb + 32 * kPieces < chunks) {
        load(cur, p0 + 32 * kPieces);  // the rest of these rows
      } else {
        r0 += warps_total * kRows;
        if (r0 < rows) load(r0, lane);  // the next rows are on their way while these are reduced and stored
      }
    }
#pragma unroll
    for (int u = 0; u < kRows; ++u) {
      const float v = warp_sum(acc[u]);
      const int r = cur + u;
      if (lane == 0 && r < rows) s.y[r] = v + (s.b ? s.b[r] : 0.f) + (s.res ? s.res[r] : 0.f);
    }
  }
}

// out[i] = SiLU(LayerNorm(in[i])) per segment (one block each): the concatenation that enters the trunk
struct NormSegs {
  int off[kMaxSegs + 1];        // segment s covers [off[s], off[s+1])
  const float* gain[kMaxSegs];  // [len]
  const float* bias[kMaxSegs];
  const float* in;
  float* out;
};
__global__ void __launch_bounds__(kThreads) k_norm_segments(NormSegs a) {
  __shared__ float red[kWarps];
  npp::pdl_launch_dependents();
  npp::pdl_wait_prior();
  const int sgm = blockIdx.x, lo = a.off[sgm], n = a.off[sgm + 1] - lo;
  const float* in = a.in + lo;
  float t = 0.f;
  for (int i = threadIdx.x; i < n; i += kThreads) t += __ldcg(in + i);
  const float mean = block_sum(t, red) / (float)n;
  t = 0.f;
  for (int i = threadIdx.x; i < n; i += kThreads) {
    const float dv = __ldcg(in + i) - mean;
    t += dv * dv;
  }
  const float rstd = rsqrtf(block_sum(t, red) / (float)n + kLnEps);
  for (int i = threadIdx.x; i < n; i += kThreads) {
    const float v = (__ldcg(in + i) - mean) * rstd * a.gain[sgm][i] + a.bias[sgm][i];
    a.out[lo + i] = v / (1.f + __expf(-v));
  }
}

template <typename K, typename A>
static cudaError_t launch_pdl(K kfn, dim3 grid, size_t smem, cudaStream_t s, const A& args) {
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
  return cudaLaunchKernelEx(&cfg, kfn, args);
}

static cudaError_t gemv(const GemvArgs& a, int n_seg, cudaStream_t s, int sm_count) {
  int max_in = 8, max_rows = 1;
  for (int i = 0; i < n_seg; ++i) {
    max_in = std::max(max_in, a.seg[i].in_dim);
    max_rows = std::max(max_rows, a.seg[i].rows);
  }
  const size_t smem = (size_t)max_in * 4;
  // two rows per warp where every warp of the device gets two, and where a row is so short that
  // one row's pieces would leave half of a lane's loads unused
  const bool wide = max_rows >= 2 * kWarps * sm_count || max_in <= 2048;
  auto kfn = wide ? k_gemv<2, 8> : k_gemv<1, 16>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  const int per_block = kWarps * (wide ? 2 : 1);
  const int want = (max_rows + per_block - 1) / per_block;
  return launch_pdl(kfn, dim3(std::max(1, std::min(want, sm_count)), n_seg), smem, s, a);
}

}  // namespace trunk
}  // namespace npi

extern "C" {

namespace {
thread_local char g_trunk_err[256] = "";
int trunk_fail(int code, const char* msg) {
  snprintf(g_trunk_err, sizeof g_trunk_err, "%s", msg);
  return code;
}
}  // namespace

const char* np_trunk_last_error(void) { return g_trunk_err; }

int np_trunk_workspace_floats(const np_trunk_desc* d, uint64_t* out) {
  if (!d || !out) return trunk_fail(NP_E_INVAL, "NULL argument");
  if (d->T < 8 || d->T % 8 || d->T > 1024) return trunk_fail(NP_E_INVAL, "T must be a multiple of 8 in [8, 1024]");
  *out = 28ull * d->T;  // raw stage-1 outputs (8T), z twice (8T each), the block's hidden vector (4T)
  return NP_OK;
}

int np_trunk_forward(const np_trunk_desc* d, const np_trunk_weights* w, const float* const* features,
                     const int32_t* centroid_id, float* workspace, float* head_logits, void* stream) {
  using namespace npi::trunk;
  if (!d || !w || !features || !centroid_id || !workspace || !head_logits) return trunk_fail(NP_E_INVAL, "NULL argument");
  const int T = d->T;
  if (T < 8 || T % 8 || T > 1024) return trunk_fail(NP_E_INVAL, "T must be a multiple of 8 in [8, 1024]");
  if (d->n_features != 4) return trunk_fail(NP_E_INVAL, "the predictor takes four continuous features");
  if (d->n_blocks < 0 || d->n_blocks > NP_TRUNK_MAX_BLOCKS) return trunk_fail(NP_E_INVAL, "n_blocks outside [0, 16]");
  if (d->n_heads < 1 || d->K < 1 || d->K0 < 1 || d->E < 8 || d->E % 8 || d->E > 8192)
    return trunk_fail(NP_E_INVAL, "n_heads, K, K0 must be positive, E a multiple of 8 in [8, 8192]");
  for (int i = 0; i < 4; ++i) {
    if (d->feature_dim[i] < 8 || d->feature_dim[i] % 8 || d->feature_dim[i] > 16384)
      return trunk_fail(NP_E_INVAL, "feature dimensions must be multiples of 8 in [8, 16384] (pad with zeros)");
    if (!features[i] || !w->proj_w[i] || !w->proj_b[i] || !w->proj_gain[i] || !w->proj_bias[i])
      return trunk_fail(NP_E_INVAL, "a feature or projection pointer is NULL");
  }
  if (!w->emb || !w->cproj_w || !w->cproj_b || !w->cproj_gain || !w->cproj_bias || !w->heads)
    return trunk_fail(NP_E_INVAL, "a weight pointer is NULL");
  for (int j = 0; j < d->n_blocks; ++j)
    if (!w->blk_w1[j] || !w->blk_b1[j] || !w->blk_gain[j] || !w->blk_bias[j] || !w->blk_w2[j] || !w->blk_b2[j])
      return trunk_fail(NP_E_INVAL, "a trunk block pointer is NULL");
  if ((uintptr_t)workspace % 16 || (uintptr_t)head_logits % 4) return trunk_fail(NP_E_INVAL, "workspace must be 16-byte aligned");
  int dev = 0, sm_count = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return trunk_fail(NP_E_CUDA, "no CUDA device");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  float* raw = workspace;          // [8T] stage-1 linear outputs
  float* z[2] = {raw + 8 * T, raw + 16 * T};
  float* hid = raw + 24 * T;       // [4T]
  cudaError_t e;
  {  // stage 1: the four feature projections and the centroid branch, one launch
    GemvArgs a = {};
    for (int i = 0; i < 4; ++i) {
      Seg& sg = a.seg[i];
      sg.w = static_cast<const uint4*>(w->proj_w[i]);
      sg.b = w->proj_b[i];
      sg.x = features[i];
      sg.y = raw + i * T;
      sg.rows = T;
      sg.in_dim = d->feature_dim[i];
    }
    Seg& c = a.seg[4];
    c.w = static_cast<const uint4*>(w->cproj_w);
    c.b = w->cproj_b;
    c.x_rows = static_cast<const uint16_t*>(w->emb);
    c.x_row = centroid_id;
    c.y = raw + 4 * T;
    c.rows = 4 * T;
    c.in_dim = d->E;
    e = gemv(a, 5, s, sm_count);
    if (e != cudaSuccess) return trunk_fail(NP_E_CUDA, cudaGetErrorString(e));
    NormSegs n = {};
    for (int i = 0; i < 4; ++i) {
      n.off[i] = i * T;
      n.gain[i] = w->proj_gain[i];
      n.bias[i] = w->proj_bias[i];
    }
    n.off[4] = 4 * T;
    n.off[5] = 8 * T;
    n.gain[4] = w->cproj_gain;
    n.bias[4] = w->cproj_bias;
    n.in = raw;
    n.out = z[0];
    e = launch_pdl(k_norm_segments, dim3(5), 0, s, n);
    if (e != cudaSuccess) return trunk_fail(NP_E_CUDA, cudaGetErrorString(e));
  }
  int cur = 0;
  for (int j = 0; j < d->n_blocks; ++j) {  // stage 2: the residual trunk, two launches per block
    GemvArgs a = {};
    Seg& dn = a.seg[0];
    dn.w = static_cast<const uint4*>(w->blk_w1[j]);
    dn.b = w->blk_b1[j];
    dn.x = z[cur];
    dn.y = hid;
    dn.rows = 4 * T;
    dn.in_dim = 8 * T;
    e = gemv(a, 1, s, sm_count);
    if (e != cudaSuccess) return trunk_fail(NP_E_CUDA, cudaGetErrorString(e));
    GemvArgs b = {};
    Seg& up = b.seg[0];
    up.w = static_cast<const uint4*>(w->blk_w2[j]);
    up.b = w->blk_b2[j];
    up.x = hid;
    up.ln_gain = w->blk_gain[j];
    up.ln_bias = w->blk_bias[j];
    up.res = z[cur];
    up.y = z[cur ^ 1];
    up.rows = 8 * T;
    up.in_dim = 4 * T;
    e = gemv(b, 1, s, sm_count);
    if (e != cudaSuccess) return trunk_fail(NP_E_CUDA, cudaGetErrorString(e));
    cur ^= 1;
  }
  {  // stage 3: the heads
    GemvArgs a = {};
    Seg& h = a.seg[0];
    h.w = static_cast<const uint4*>(w->heads);
    h.x = z[cur];
    h.y = head_logits;
    h.rows = d->n_heads * 2 * d->K;
    h.in_dim = 8 * T;
    e = gemv(a, 1, s, sm_count);
    if (e != cudaSuccess) return trunk_fail(NP_E_CUDA, cudaGetErrorString(e));
  }
  return NP_OK;
}

}  // extern "C"
