// Stage 4 over a run of consecutive layers in ONE resident kernel, partitioned in two
// directions (B = 1):
//
//   x_{l+1} = x_l + sum_{i in act_l} silu(gate_l[s_i].n_l) * (up_l[s_i].n_l) * downT_l[s_i],
//   n_l = x_l / sqrt(mean(x_l^2) + 1e-6)   (pre-MLP RMS normalisation, unit gain)
//
// (Section 3.4: the sparse MLP reads each active row through the slot map.)
//
// A layer moves ~27 MB at the 7B shape, 4 us of HBM time, so what a layer costs is decided by
// what crosses between the blocks and by how many instructions a warp walks through between
// two layers (with a handful of warps per scheduler every instruction of the per-layer path
// costs several cycles).  Two things follow.
//
// 1. The grid is Q x R blocks (Q = 4 column slices, R = SMs / 4 row groups).  Block (r, q) owns
//    the rows of row group r and the q-th quarter of the columns: it reads the q-th quarter of
//    those rows' gate, up and down vectors (2 KB pieces at D = 4096, each byte still read
//    exactly once).  Phase 1 gives partial dot products over its quarter of K; the four blocks
//    of a row group exchange them ONCE per layer (2 floats per row) through 64-bit
//    (value, stamp) words that are written with one store and polled by the readers: no fence,
//    no counter.  Phase 2 gives a partial sum of its quarter of the outputs only: a quarter of
//    the reduction volume and of the accumulator re-read of a kernel that deals whole rows to
//    the blocks (np_mlp_chain.cu), and the hand-over of x_{l+1} spans only the R blocks of the
//    same quarter (x's quarter q is all block (r, q) ever needs: its K range in phase 1 is its
//    column range in phase 2).  The sum of squares of x for the normalisation travels with the
//    exchange.
//
//    Between two layers of a launch the R partial sums of a column meet in 64-bit words that
//    carry their own arrival count: a block adds, with one 64-bit reduction per column,
//    2^56 + round(y * 2^30), so the word's top byte counts the blocks that have added and the
//    rest is their sum in fixed point (resolution 2^-30, |y| < 2^19 per block, checked).  A
//    reader polls the words of its own columns until the count is R: no fence, no arrival
//    counter and no second trip to read the sums, the adds commute exactly (the result does not
//    depend on their order), and nothing is cleared while it is in use: the words only grow, two
//    sets of them alternate by layer, and a reader subtracts what it saw at the set's previous
//    completion (all arithmetic modulo 2^64).  What the sets held when the launch began is read at
//    its start (which also brings the words into the L2: a launch that found them zeroed by its
//    predecessor instead measured 340-400 us per 32 layers against 261); a block's first adds wait
//    until every block of its slice has done that reading (one arrival counter per slice, counted
//    once per launch and long complete by the time the first layer ends).  The launch's last layer
//    leaves its sums as fp32 in the stack's rotating accumulators, the form every other kernel of
//    the chain reads -- unless the launch ends the stack: then the last layer's sums go through the
//    counted words too, and the blocks of row group 0 wait for them and write the stack's result.
//
//    This form is used where a thread owns one or two 4-column granules of the slice (row widths
//    up to 8192).  Wider slices keep the fp32 form between all layers: 16-byte fp32 reductions into
//    the rotating accumulators (kZRep copies), a fence, one arrival counter per slice that the next
//    layer's first thread polls, then every thread reads the copies of its columns (the counted
//    form would hold the previous sums of four granules in registers there).
//
// 2. Both phases run on the tensor cores (mma.sync m16n8k16, bf16 x bf16 -> fp32), not for
//    their arithmetic rate but because one ldmatrix + one mma replace a hundred unpack and FMA
//    instructions.  Phase 1: A = the 16 gate / up vectors of a group (rows) over a 16-wide K
//    block, B = x as three truncated bf16 terms (exact to 2^-24) in columns 0-2; the K blocks
//    are dealt to the warps.  Phase 2: A = 16 output columns x 16 down rows (ldmatrix.trans of
//    the row-major pieces), B = the activations as three bf16 terms; a warp keeps the
//    accumulators of its column tiles in registers over the whole layer.
//
// Shared memory is one ring of load groups in the order they are consumed: the gate|up pieces
// of a layer's rows (groups of VG vectors), then its down pieces (groups of VG rows), then the
// next layer's.  A producer warp fills it with 1-D bulk copies (one mbarrier per group) and
// runs as far ahead as the ring allows, across layers.  Pieces are 16 bytes further apart
// than they are long, so that the eight row addresses of an ldmatrix fall into different
// banks.  An exchange warp does the trip through L2 and leaves the activations.  Inside a
// layer the consumer warps meet at no block-wide barrier until their sums are reduced.
//
// Every wait (mbarrier, exchange words, counted sums) is bounded; once one has run out
// the block records kStatTimeout and skips all later waits, so every thread still passes the
// same barriers and the kernel drains; the blocks that depend on it follow at their next wait.
#include <algorithm>
#include <cstdlib>

#include "np_device.cuh"
#include "np_internal.h"
#include "np_pipe.cuh"

namespace npi {
namespace chain_slices {
using namespace npd;

constexpr int kQ = 4;                  // column slices
constexpr int kWarps = 8;              // consumer warps
constexpr int kThreads = kWarps * 32;  // consumer threads
constexpr int kBlock = kThreads + 64;  // plus one producer warp and one exchange warp
constexpr int kMaxGroups = 16;         // ring slots
constexpr int kMaxLayers = 64;         // layers per launch (longer runs are split by the host)
constexpr int kBarStride = 32;         // one 128-byte line per counter
constexpr int kFixShift = 30;          // fixed-point position of the counted sums
constexpr float kFixLimit = 524288.f;  // |partial sum| a block may add (2^19: 63 of them stay below 2^25 = 2^(55 - kFixShift))
constexpr int kMaxR = 63;              // row groups whose counts and sums fit a word
constexpr int kFixMaxKS = 16;          // widest slices (in 16-column tiles per warp) that use the counted words: one or two
                                       // 4-column granules per thread, row widths up to 8192
#ifndef NP_SL_FIXREP
#define NP_SL_FIXREP 1
#endif
constexpr int kFixRep = NP_SL_FIXREP;  // copies of the counted words (row group r adds to copy r % kFixRep).  One: the 37
                                       // adds to a word cost less than reading more copies (7B shape, 32 layers: 250 us
                                       // with one copy, 252 with two, 262 with four)
constexpr int kHist = 8;               // pacing history of the producer (> window)
constexpr int kGroupTarget = 68 * 1024;  // largest load group: up to 16 vectors, three groups to a ring at least (70B shape:
                                         // 66 KB groups of 16 vectors, 1.39 ms per 80 layers; 33 KB groups of 8: 1.51 ms)
constexpr int kPad = 16;               // bytes between pieces in shared memory

struct KArgs {
  const unsigned char* gate;   // layer 0 of each buffer; layer stride = C * D * 2 bytes
  const unsigned char* up;
  const unsigned char* downT;
  const int32_t* slots;        // active_slots [L][C]
  const int32_t* counters;     // [L][NP_N_COUNTERS]
  const uint16_t* x_bf16;      // not NULL: the run starts the stack (layer 0) and reads its input from here (bf16 [D])
  float* xbuf[2];              // x_l of the run's last layer is stored to xbuf[l & 1]
  float* x_out;                // counted form only, may be NULL: the launch ends the stack and leaves x_L = x_{L-1} + MLP_{L-1} here
  float* zbuf[3];              // MLP_l(x_l) accumulates into zbuf[l % 3]: kZRep copies of [D]
  unsigned long long* zfix;    // [2][kFixRep][D] counted fixed-point sums of MLP_l(x_l), sets alternate by layer, never cleared
  unsigned int* bars;          // [kQ][kBarStride] arrival counters, never reset (the host tracks their value).  Counted
                               // sums: blocks of a slice that have read the sets at the launch's start.  fp32 form:
                               // blocks that have added their part of a layer (R per layer but the launch's last).
  unsigned int bar_base;       // value of every counter when the launch starts
  unsigned long long* xch;     // [2][grid][xch_stride] (value, stamp) words
  int32_t* status;
  unsigned int seq_base;       // stamp of the launch's first exchange minus one
  unsigned int ng_magic;       // ceil(2^32 / ng): group sequence number -> ring slot without a division
  int l_begin, l_end, D, C, check;
  int vg_shift, ng, window;    // log2 of the vectors per gate|up group (= rows per down group), ring slots, groups in flight
  int gw_shift;                // log2 of the consumer warps that share one gate|up group in phase 1
  int max_rows;                // most rows a block can have in a layer
  int xch_stride;              // words per block in the exchange area (2 * max_rows + 1, rounded up)
  uint32_t group_bytes;
};

#ifdef NP_TRACE  // development builds only: time stamps of four blocks, read back by np_debug_trace
__device__ unsigned long long np_trace_buf[4][64][32];
__device__ unsigned long long np_trace_all[160][8][8];
extern "C" int np_debug_trace_all(void* out) { return (int)cudaMemcpyFromSymbol(out, np_trace_all, sizeof(np_trace_all)); }
__device__ __forceinline__ unsigned long long gtime() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ long long np_trace_clk[4][64];
#define NP_CK(ev) do { if (blockIdx.x == 0 && li == 3 && lane == 0 && (wid & 1) == 0 && (ev) < 64) np_trace_clk[wid >> 1][ev] = clock64(); } while (0)
extern "C" int np_debug_clk(void* out) { return (int)cudaMemcpyFromSymbol(out, np_trace_clk, sizeof(np_trace_clk)); }
#define NP_TR(slot)                                                                                       \
  do {                                                                                                    \
    const int tb__ = blockIdx.x < 4 ? (int)blockIdx.x : -1;                                               \
    if (threadIdx.x == 0 && tb__ >= 0 && li < 64 && (slot) < 32) np_trace_buf[tb__][li][slot] = gtime();  \
    if (threadIdx.x == 0 && blockIdx.x < 160 && li < 8 && (slot) < 8) np_trace_all[blockIdx.x][li][slot] = gtime(); \
  } while (0)
extern "C" int np_debug_trace(void* out) { return (int)cudaMemcpyFromSymbol(out, np_trace_buf, sizeof(np_trace_buf)); }
#else
#define NP_CK(ev) do { } while (0)
#define NP_TR(slot) do { } while (0)
#endif

__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory"); }

// 16-byte floating-point reduction to global memory, no return value
__device__ __forceinline__ void red_add_v4(float* p, float4 v) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
// mma.sync m16n8k16, bf16 x bf16 -> fp32
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t smem_row) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(smem_row));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t smem_row) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(smem_row));
}
// fp32 -> three bf16 terms by truncation: v = t0 + t1 + t2 up to 2^-24 |v|; the terms come back
// as fp32 bit patterns whose low 16 bits are zero
__device__ __forceinline__ void split3(float v, uint32_t& t0, uint32_t& t1, uint32_t& t2) {
  t0 = __float_as_uint(v) & 0xffff0000u;
  const float r1 = v - __uint_as_float(t0);
  t1 = __float_as_uint(r1) & 0xffff0000u;
  const float r2 = r1 - __uint_as_float(t1);
  t2 = __float_as_uint(r2) & 0xffff0000u;
}
// two truncated terms -> one packed bf16x2 word (first element in the low half)
__device__ __forceinline__ uint32_t pack_hi16(uint32_t first, uint32_t second) { return __byte_perm(first, second, 0x7632); }
__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ void ld_relaxed_v2u64(const unsigned long long* p, unsigned long long& a, unsigned long long& b) {
  asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(a), "=l"(b) : "l"(p));
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void red_add_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long stamped(float v, unsigned int stamp) {
  return ((unsigned long long)stamp << 32) | (unsigned long long)__float_as_uint(v);
}

// A bounded wait on an mbarrier by one lane.  Once any wait of the block has run out
// (*ok == 0) every later wait is skipped, so no barrier is ever left short of threads.
__device__ __forceinline__ void wait_or_flag(uint64_t* bar, uint32_t parity, volatile int* ok, int32_t* status) {
  if (npp::mbar_try_wait(bar, parity)) return;  // the usual case: already complete
  if (!*ok) return;
  if (!npp::mbar_wait(bar, parity)) {
    *ok = 0;
    atomicOr(status, npp::kStatTimeout);
  }
}

__device__ __forceinline__ void mbar_arrive_n(uint64_t* bar, uint32_t n) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(npp::smem_addr(bar)), "r"(n) : "memory");
}

// A consumer's wait for group number gq of the launch.  The parity test of an mbarrier only tells
// the current phase from the one before it, and a warp does not visit every use of a ring slot
// (phase 1 deals the gate|up groups to sets of warps), so it first makes sure that the producer
// has armed this very use (the groups are armed in order; `armed` counts them): then the slot's
// barrier is in the phase of group gq or one past it, and the parity test is exact.
__device__ __forceinline__ void wait_group(unsigned int gq, uint64_t* bar, uint32_t parity, const volatile unsigned int* armed,
                                           volatile int* ok, int32_t* status) {
  if (*armed <= gq) {
    if (!*ok) return;
    bool there = false;
    for (uint32_t spin = 0; spin < npp::kSpinLimit * 16u && !there; ++spin) there = *armed > gq;
    if (!there) {
      *ok = 0;
      atomicOr(status, npp::kStatTimeout);
      return;
    }
  }
  wait_or_flag(bar, parity, ok, status);
}

// ring slot and use parity of the group with sequence number g (exact for g < 2^32 / ng)
__device__ __forceinline__ void slot_of(unsigned int g, unsigned int magic, int ng, int& slot, uint32_t& par) {
  const unsigned int qd = __umulhi(g, magic);
  slot = (int)(g - qd * (unsigned int)ng);
  par = qd & 1u;
}

// KS: 16-column tiles (phase 2) per warp: ceil(D / kQ / 16 / kWarps).  XB: a warp has at most 32 K blocks
// in phase 1 and keeps their B operands (x) in registers for the whole layer.
template <int KS, bool XB>
__global__ void __launch_bounds__(kBlock, 1) k_mlp_slices(KArgs a) {
  extern __shared__ __align__(128) unsigned char csm[];
  __shared__ __align__(8) uint64_t full_bar[kMaxGroups];   // the group's copies have landed
  __shared__ __align__(8) uint64_t empty_bar[kMaxGroups];  // every consumer warp is done with the group
  __shared__ __align__(8) uint64_t p1_bar;                 // every consumer warp has left its partial sums of the layer
  __shared__ __align__(8) uint64_t act_bar;                // the exchange warp has left the layer's activations
  __shared__ float ssq_part[kWarps];                       // per-warp sums of this slice's x_l^2
  __shared__ int s_ok;
  __shared__ unsigned int s_armed;                         // groups the producer has armed so far
  __shared__ int lay_rb[kMaxLayers];       // first active-list index of this block's row group, per layer
  __shared__ int lay_pre[kMaxLayers + 1];  // rows of this row group before each layer (virtual row index)

  constexpr bool kFix = KS <= kFixMaxKS;  // counted fixed-point sums between the layers of a launch
  const bool fin = kFix && a.x_out != nullptr;  // ... and behind its last layer: the launch leaves the stack's result itself
  const int D = a.D, Ds = D / kQ;
  const int nk = Ds >> 4;     // 16-wide K blocks = 16-column tiles of the slice
  const uint32_t piece_bytes = (uint32_t)Ds * 2u;
  const uint32_t pstride = piece_bytes + kPad;  // distance between pieces in shared memory
  const size_t row_bytes = (size_t)D * 2;
  const size_t layer_bytes = (size_t)a.C * row_bytes;
  const int gs = a.vg_shift, VG = 1 << gs;  // vectors per gate|up group, rows per down group
  const int ng = a.ng;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int G = gridDim.x, R = G / kQ;
  const int q = blockIdx.x % kQ, r = blockIdx.x / kQ;
  const int qoff = q * Ds;  // first column (= first K index) of this slice
  const int nl = a.l_end - a.l_begin;
  const int apad = ((a.max_rows + 15) & ~15) + 16;  // activations per term, padded so that a 16-row block never runs out
  const int n_gu_max = (2 * a.max_rows + VG - 1) >> gs;
  // dynamic shared memory: ring | x as 3 bf16 terms | staging of the block's output sums | partial sums | activations | slots
  unsigned char* xterm = csm + (size_t)ng * a.group_bytes;           // [3][pstride]
  float* ybuf = reinterpret_cast<float*>(xterm + 3 * pstride);       // [Ds]
  const int GW = 1 << a.gw_shift;  // consumer warps per gate|up group: each takes every GW-th K block
  float* part = ybuf + Ds;                                           // [groups][GW][VG] partial gate / up sums
  uint16_t* aterm = reinterpret_cast<uint16_t*>(part + (size_t)n_gu_max * GW * VG);  // [3][apad] bf16 terms of a_i
  int* slot_cache = reinterpret_cast<int*>(aterm + 3 * apad + (apad & 1));
  volatile int* ok = &s_ok;
  volatile unsigned int* armed = &s_armed;

  // ---- this row group's share of every layer of the run ----
  if (tid < nl) {
    int n = a.counters[(size_t)(a.l_begin + tid) * NP_N_COUNTERS + NP_CNT_ACTIVE];
    if (a.check && (n < 0 || n > a.C)) {
      atomicOr(a.status, kStatBadCount);
      n = 0;
    }
    const int rb = (int)(((long long)n * r) / R);
    const int re = (int)(((long long)n * (r + 1)) / R);
    lay_rb[tid] = rb;
    lay_pre[tid + 1] = min(re - rb, a.max_rows);  // turned into a prefix sum below
  }
  if (tid == 0) {
    for (int s = 0; s < ng; ++s) {
      npp::mbar_init(&full_bar[s], 1);
      npp::mbar_init(&empty_bar[s], kWarps);
    }
    npp::mbar_init(&p1_bar, kWarps);
    npp::mbar_init(&act_bar, 1);
    npp::fence_barrier_init();
    s_ok = 1;
    s_armed = 0;
  }
  // The tensor-core tiles read whole 16 x 16 blocks: rows of a ragged group that no copy fills are
  // multiplied by zero activations, so what they hold must at least be finite.
  for (uint32_t i = tid; i < (uint32_t)ng * a.group_bytes / 16; i += blockDim.x)
    reinterpret_cast<uint4*>(csm)[i] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  if (tid == 0) {
    lay_pre[0] = 0;
    for (int i = 0; i < nl; ++i) lay_pre[i + 1] += lay_pre[i];
  }
  npp::fence_proxy_async();  // the zeros precede the bulk copies into the same bytes
  __syncthreads();
  for (int li = 0; li < nl; ++li) {
    const int nr = lay_pre[li + 1] - lay_pre[li];
    for (int i = tid; i < nr; i += blockDim.x) {
      int slot = a.slots[(size_t)(a.l_begin + li) * a.C + lay_rb[li] + i];
      if (a.check && (slot < 0 || slot >= a.C)) {
        atomicOr(a.status, kStatBadSlot);
        slot = 0;
      }
      slot_cache[lay_pre[li] + i] = slot;
    }
  }
  __syncthreads();

  if (wid == kWarps) {
    // =========================== producer warp ===========================
    // The groups are requested in the order they are consumed.  The waits are lane 0's (several
    // lanes waiting on different barriers must not be used: the compiler may reconverge the warp
    // after a wait); the copies of a group are then issued by as many lanes as it has pieces,
    // since one lane issuing ninety 2 KB copies per layer sets the pace otherwise.
    int hist_slot[kHist];
    uint32_t hist_par[kHist];
    int issued = 0, slot = 0;
    uint32_t par = 0;
    // A row is read once per token: the copies mark their lines evict-first, so that the 27 MB a layer streams
    // through the L2 do not push out the few hundred KB every layer meets in (exchange words, counted sums,
    // slot lists): 7B shape 236 us per 32 layers against 249, 13B shape 341 us per 40 layers against 358.
    const uint64_t l2_policy = npp::policy_evict_first();
    const size_t qbytes = (size_t)q * piece_bytes;
    for (int li = 0; li < nl; ++li) {
      const int vbase = lay_pre[li], nrows = lay_pre[li + 1] - vbase;
      const size_t lbase = (size_t)(a.l_begin + li) * layer_bytes + qbytes;
      // pass 0: gate|up groups (VG / 2 rows, two pieces each); pass 1: down groups (VG rows)
      for (int pass = 0; pass < 2; ++pass) {
        const int grows_max = pass == 0 ? (VG >> 1) : VG;
        for (int r0 = 0; r0 < nrows; r0 += grows_max) {
          const int grows = min(grows_max, nrows - r0);
          const int npieces = pass == 0 ? 2 * grows : grows;
          if (lane == 0) {
            wait_or_flag(&empty_bar[slot], par ^ 1u, ok, a.status);
            // pacing: at most `window` groups in flight per block.  A deeper burst moves no more
            // bytes (HBM is shared by all blocks) but queues in front of the short loads on the
            // layer's critical path (exchange words, barrier counter, accumulators).
            if (a.window > 0 && issued >= a.window) {
              const int h = (issued - a.window) % kHist;
              wait_or_flag(&full_bar[hist_slot[h]], hist_par[h], ok, a.status);
            }
            npp::mbar_expect_tx(&full_bar[slot], (uint32_t)npieces * piece_bytes);
            __threadfence_block();
            *armed = (unsigned int)issued + 1u;  // consumers of this group may now test the barrier's parity
          }
          __syncwarp();  // the expect_tx precedes the copies
          hist_slot[issued % kHist] = slot;
          hist_par[issued % kHist] = par;
          ++issued;
          unsigned char* dst = csm + (size_t)slot * a.group_bytes;
#ifdef NP_TUNE
          if (a.window < 0) {  // development: no copies at all
            if (lane == 0) asm volatile("mbarrier.complete_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(npp::smem_addr(&full_bar[slot])), "r"((uint32_t)npieces * piece_bytes) : "memory");
          } else
#endif
          for (int idx = lane; idx < npieces; idx += 32) {
            const int i = pass == 0 ? idx >> 1 : idx;
            const size_t off = lbase + (size_t)slot_cache[vbase + r0 + i] * row_bytes;
            const unsigned char* src = (pass == 0 ? ((idx & 1) ? a.up : a.gate) : a.downT) + off;
            npp::bulk_g2s_stream(dst + (size_t)idx * pstride, src, piece_bytes, &full_bar[slot], l2_policy);
          }
          __syncwarp();
          if (++slot == ng) {
            slot = 0;
            par ^= 1u;
          }
        }
      }
    }
    return;
  }

  if (wid == kWarps + 1) {
    // =========================== exchange warp ===========================
    // Per layer: publish this block's partial dot products, collect the other three slices',
    // turn the sums into activations (three bf16 terms each, the B operand of phase 2).
    unsigned int nx = 0;  // exchanges so far (layers in which this row group has rows)
    for (int li = 0; li < nl; ++li) {
      const int nrows = lay_pre[li + 1] - lay_pre[li];
      if (nrows == 0) continue;
      if (lane == 0) wait_or_flag(&p1_bar, nx & 1u, ok, a.status);
      __syncwarp();
      const unsigned int stamp = a.seq_base + 1u + nx;
      unsigned long long* mine = a.xch + ((size_t)(nx & 1u) * G + blockIdx.x) * a.xch_stride;
      const unsigned long long* base = a.xch + ((size_t)(nx & 1u) * G + (size_t)r * kQ) * a.xch_stride;
      float own_ss = 0.f;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) own_ss += ssq_part[w];
      if (lane == 0) st_relaxed_u64(mine + 2 * a.max_rows, stamped(own_ss, stamp));
      float inv_rms = 0.f;
      const int nrows16 = (nrows + 15) & ~15;
      for (int r0 = 0; r0 < nrows16; r0 += 32) {
        const int row = r0 + lane;
        const bool has_row = row < nrows, want_ss = r0 == 0 && lane == 0;
        // this block's own sums of the row: the partial sums of the consumer warps (their K blocks)
        float own_g = 0.f, own_u = 0.f;
        if (has_row) {
          const int v = 2 * row;
          const float* pp = part + ((size_t)(v >> gs) * GW) * VG + (v & (VG - 1));
          for (int w = 0; w < GW; ++w) {
            own_g += pp[w * VG];
            own_u += pp[w * VG + 1];
          }
          st_relaxed_u64(mine + v, stamped(own_g, stamp));
          st_relaxed_u64(mine + v + 1, stamped(own_u, stamp));
        }
        // One 16-byte load per row and peer (its gate and up words), issued only by the lanes that
        // have a row; lane 0 also fetches the peers' sums of squares.  Strong loads are not merged
        // across lanes, so every load that is not needed costs a request of its own at the L2 (all
        // blocks poll at about the same moment).
        float gsum[kQ], usum[kQ], ssv[kQ];  // indexed by unrolled constants only (registers)
        bool done = !*ok;
        for (uint32_t spin = 0; spin < npp::kSpinLimit && !done; ++spin) {
          unsigned long long wg[kQ], wu[kQ], ws[kQ];  // every load of the round is issued before any is looked at
#pragma unroll
          for (int qq = 0; qq < kQ; ++qq) {
            const unsigned long long* w = base + (size_t)qq * a.xch_stride;
            wg[qq] = wu[qq] = ws[qq] = (unsigned long long)stamp << 32;
            if (has_row && qq != q) ld_relaxed_v2u64(w + 2 * row, wg[qq], wu[qq]);
            if (want_ss && qq != q) ws[qq] = ld_relaxed_u64(w + 2 * a.max_rows);
          }
          unsigned int bad = 0;
#pragma unroll
          for (int qq = 0; qq < kQ; ++qq) {
            bad |= ((unsigned int)(wg[qq] >> 32) ^ stamp) | ((unsigned int)(wu[qq] >> 32) ^ stamp) |
                   ((unsigned int)(ws[qq] >> 32) ^ stamp);
            gsum[qq] = __uint_as_float((unsigned int)wg[qq]);
            usum[qq] = __uint_as_float((unsigned int)wu[qq]);
            ssv[qq] = __uint_as_float((unsigned int)ws[qq]);
          }
          done = bad == 0;
        }
        if (!done) {
          *ok = 0;
          atomicOr(a.status, npp::kStatTimeout);
        }
        if (r0 == 0) {
          float ss = 0.f;
#pragma unroll
          for (int qq = 0; qq < kQ; ++qq) ss += qq == q ? own_ss : ssv[qq];  // the same order in every block
          inv_rms = __shfl_sync(0xffffffffu, rsqrtf(ss / (float)D + kRmsEps), 0);  // lane 0 holds the peers' sums
        }
        if (row < nrows16) {
          float av = 0.f;  // rows that pad the last 16-row block: zero
          if (has_row) {
            float gsv = 0.f, usv = 0.f;
#pragma unroll
            for (int qq = 0; qq < kQ; ++qq) {
              gsv += qq == q ? own_g : gsum[qq];
              usv += qq == q ? own_u : usum[qq];
            }
            // the MLP's input is x_l scaled to unit RMS; the dot products are linear in it
            gsv *= inv_rms;
            usv *= inv_rms;
            av = gsv / (1.f + __expf(-gsv)) * usv;
          }
          uint32_t t0, t1, t2;
          split3(av, t0, t1, t2);
          aterm[row] = (uint16_t)(t0 >> 16);
          aterm[apad + row] = (uint16_t)(t1 >> 16);
          aterm[2 * apad + row] = (uint16_t)(t2 >> 16);
        }
      }
      __syncwarp();
      if (lane == 0) npp::mbar_arrive(&act_bar);
      ++nx;
    }
    return;
  }

  // =========================== consumer warps ===========================
  const int l_last = a.l_end - 1;
  const int g8 = lane >> 2, t4 = lane & 3;  // mma fragment coordinates of this lane
  const int m4 = lane >> 3, rr = lane & 7;  // ldmatrix: lanes 8 m4 .. 8 m4 + 7 give the row addresses of 8x8 matrix m4
  const uint32_t ring = npp::smem_addr(csm);
  constexpr int J4 = (KS * kWarps * 16 / 4 + kThreads - 1) / kThreads;  // float4 granules of the slice per thread
  const int nf4 = Ds >> 2;
  float4 xown[J4];        // x_l of the columns this thread owns, for the whole run
  unsigned int gseq = 0;  // sequence number of the layer's first group
  unsigned int nx = 0;    // exchanges so far
  // counted sums: what the words of this thread's columns added up to (over the copies) when their set was last complete
  // (zprev: the set read next, zprev2: the other one; they trade places after every read)
  unsigned long long zprev[J4][4] = {}, zprev2[J4][4] = {};
  if (kFix && (nl > 1 || fin)) {
    unsigned long long seen = 0ull;
#pragma unroll
    for (int j = 0; j < J4; ++j) {
      const int c = tid + j * kThreads;
#pragma unroll
      for (int e = 0; e < 4; ++e) zprev[j][e] = zprev2[j][e] = 0ull;
      if (c < nf4) {
#pragma unroll
        for (int rep = 0; rep < kFixRep; ++rep) {
          const ulonglong2* w = reinterpret_cast<const ulonglong2*>(a.zfix + (size_t)rep * D + qoff) + 2 * c;
          const ulonglong2* w2 = reinterpret_cast<const ulonglong2*>(a.zfix + (size_t)(kFixRep + rep) * D + qoff) + 2 * c;
          const ulonglong2 p0 = __ldcg(w), p1 = __ldcg(w + 1), q0 = __ldcg(w2), q1 = __ldcg(w2 + 1);
          zprev[j][0] += p0.x, zprev[j][1] += p0.y, zprev[j][2] += p1.x, zprev[j][3] += p1.y;
          zprev2[j][0] += q0.x, zprev2[j][1] += q0.y, zprev2[j][2] += q1.x, zprev2[j][3] += q1.y;
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) seen ^= zprev[j][e] ^ zprev2[j][e];
      }
    }
    // Every value has arrived (it is looked at) before the block counts itself in: only then may any block of
    // the slice add to these words.  (The words' top bytes hold small counts, so the pattern below cannot occur.)
    if (seen == 0xffffffffffffffffull) atomicOr(a.status, kStatBadCount);
    consumer_sync();
    if (tid == 0) atomicAdd(a.bars + q * kBarStride, 1u);
  }
  // phase 1, A operand: row = vector rr + 8 (m4 & 1) of the group (clamped into the group), K offset 8 (m4 >> 1)
  const uint32_t a1_off = (uint32_t)((rr + 8 * (m4 & 1)) & (VG - 1)) * pstride + (uint32_t)(m4 >> 1) * 16u;
  // phase 2, A operand (transposed load): stored row = down row rr + 8 (m4 >> 1) of the group, column offset 8 (m4 & 1)
  const uint32_t a2_off = (uint32_t)((rr + 8 * (m4 >> 1)) & (VG - 1)) * pstride + (uint32_t)(m4 & 1) * 16u;

  for (int li = 0; li < nl; ++li) {
    const int l = a.l_begin + li;
    NP_TR(0);
    // ---- the sums of layer l-1 over this thread's columns, once every row group has added its part ----
    float4 zsum[J4];
#pragma unroll
    for (int j = 0; j < J4; ++j) zsum[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (!kFix && li > 0) {
      // fp32 form: wait until every block of this column slice has added its part of layer l-1
      if (tid == 0 && *ok) {
        const unsigned int target = a.bar_base + (unsigned int)li * (unsigned int)R;
        bool arrived = false;
        for (uint32_t spin = 0; spin < npp::kSpinLimit; ++spin) {
          unsigned int v;
          asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(a.bars + q * kBarStride) : "memory");
          if ((int)(v - target) >= 0) {
            arrived = true;
            break;
          }
        }
        if (!arrived) {
          *ok = 0;
          atomicOr(a.status, npp::kStatTimeout);
        }
      }
      consumer_sync();
    }
    if (kFix && li > 0) {
      const int pb = (li - 1) & 1;
      const unsigned long long* zw = a.zfix + (size_t)pb * kFixRep * D + qoff;
      // Every thread polls the words of its own columns (two 16-byte loads per round with one copy of the
      // words).  With four copies, 148 x 256 threads polling eight loads each kept the L2 busy enough to slow
      // every other trip through it, and a lane per warp watched one column first; with one copy that watch
      // only costs a round trip (7B shape, 32 layers: 250 us without it, 253 with it).
#pragma unroll
      for (int j = 0; j < J4; ++j) {  // one or two granules per thread, one after the other
        const int c = tid + j * kThreads;
        if (c >= nf4) continue;
        unsigned long long sum[4] = {0ull, 0ull, 0ull, 0ull};
        bool done = !*ok;
        for (uint32_t spin = 0; spin < npp::kSpinLimit && !done; ++spin) {
          unsigned long long w[kFixRep][4];  // every load of the round is issued before any is looked at
#pragma unroll
          for (int rep = 0; rep < kFixRep; ++rep) {
            const unsigned long long* wp = zw + (size_t)rep * D + 4 * c;
            ld_relaxed_v2u64(wp, w[rep][0], w[rep][1]);
            ld_relaxed_v2u64(wp + 2, w[rep][2], w[rep][3]);
          }
          done = true;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            sum[e] = 0ull;
#pragma unroll
            for (int rep = 0; rep < kFixRep; ++rep) sum[e] += w[rep][e];
            const long long delta = (long long)(sum[e] - zprev[j][e]);
            done = done && ((delta + (1ll << 55)) >> 56) == (long long)R;
          }
        }
        if (!done && *ok) {
          *ok = 0;
          atomicOr(a.status, npp::kStatTimeout);
        }
        float zv[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const long long value = (long long)(sum[e] - zprev[j][e]) - ((long long)R << 56);
          zv[e] = done ? __ll2float_rn(value) * (1.f / (float)(1u << kFixShift)) : 0.f;
          zprev[j][e] = zprev2[j][e];  // the other set is read next; this one, as it stands now, after that
          zprev2[j][e] = sum[e];
        }
        zsum[j] = make_float4(zv[0], zv[1], zv[2], zv[3]);
      }
      // the launch's last layer adds into an accumulator that another block cleared one layer earlier (and
      // fenced before it added the sums read above): the fence that completes that order on this side
      if (li == nl - 1 && !fin) __threadfence();
    }
    NP_TR(1);
    // ---- x_l (this slice): first layer of the run from global, afterwards x_l = x_{l-1} + MLP_{l-1};
    //      each thread updates its own columns and publishes them as three bf16 terms ----
    {
      const float* xa = a.xbuf[(l + 1) & 1] + qoff;
      // fp32 sums of the layer before: the previous kernel's; in the fp32 form also those of this launch's layers
      const float* zb = ((!kFix || li == 0) && l > 0) ? a.zbuf[(l - 1) % 3] + qoff : nullptr;
      float* xst = a.xbuf[l & 1] + qoff;
      float ssq = 0.f;
      float4 w[J4][kZRep];
#pragma unroll
      for (int j = 0; j < J4; ++j) {  // every load of the pass is issued before any is used
        const int c = tid + j * kThreads;
        if (c < nf4) {
          if (li == 0) {
            if (a.x_bf16) {  // the stack's input: bf16 values widened here (no kernel in front for that)
              const uint2 h = __ldg(reinterpret_cast<const uint2*>(a.x_bf16 + qoff) + c);
              xown[j] = make_float4(bf16_lo(h.x), bf16_hi(h.x), bf16_lo(h.y), bf16_hi(h.y));
            } else {
              xown[j] = __ldcg(reinterpret_cast<const float4*>(xa) + c);
            }
          }
          if (zb) {
#pragma unroll
            for (int rep = 0; rep < kZRep; ++rep) w[j][rep] = __ldcg(reinterpret_cast<const float4*>(zb + (size_t)rep * D) + c);
          }
        } else {
          xown[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
#pragma unroll
      for (int j = 0; j < J4; ++j) {
        const int c = tid + j * kThreads;
        if (c < nf4) {
          float4 v = xown[j];
          v.x += zsum[j].x, v.y += zsum[j].y, v.z += zsum[j].z, v.w += zsum[j].w;
          if (zb) {
#pragma unroll
            for (int rep = 0; rep < kZRep; ++rep) {
              v.x += w[j][rep].x;
              v.y += w[j][rep].y;
              v.z += w[j][rep].z;
              v.w += w[j][rep].w;
            }
          }
          xown[j] = v;
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
            *reinterpret_cast<uint2*>(xterm + (size_t)term * pstride + (size_t)c * 8) = packed;
          }
          if (r == 0 && l == l_last) reinterpret_cast<float4*>(xst)[c] = v;  // x for the next launch
        }
      }
      ssq = warp_sum(ssq);
      if (lane == 0) ssq_part[wid] = ssq;
      // The launch's last layer adds fp32 sums into the stack's rotating accumulators: its own is cleared one
      // layer ahead (by the layer before it; a launch of one layer finds it cleared by the kernel in front),
      // and it clears the one the next kernel's first layer adds into.  Every row group takes a share.
      if (!kFix || (!fin && li >= nl - 2)) {
        float* znext = a.zbuf[(l + 1) % 3] + qoff;
        const int zper = (nf4 * kZRep + R - 1) / R;
        bool cleared = false;
        for (int i = r * zper + tid; i < min((r + 1) * zper, nf4 * kZRep); i += kThreads) {
          int rep = 0, c = i;
          while (c >= nf4) {
            c -= nf4;
            ++rep;
          }
          reinterpret_cast<float4*>(znext + (size_t)rep * D)[c] = make_float4(0.f, 0.f, 0.f, 0.f);
          cleared = true;
        }
        // the zeros are ahead of this block's counted sums of this layer (added after the barriers below),
        // which every block reads before it adds to the cleared accumulator
        if (kFix && cleared && li == nl - 2) __threadfence();
      }
    }
    consumer_sync();  // the terms of x and ssq_part are in place
    NP_TR(2);
    const int nrows = lay_pre[li + 1] - lay_pre[li];
    const int n_gu = (2 * nrows + VG - 1) >> gs, n_dn = (nrows + VG - 1) >> gs;
    // ---- phase 1: [VG vectors of a group] x [x as 3 terms].  The layer's gate|up groups are dealt to sets of GW
    //      warps, so that several groups are worked on at once; within a set a warp takes every GW-th K block.
    //      B: column n = term n of x (columns 3-7 zero): b0 = k 2 t4, 2 t4 + 1 of the block, b1 = the same + 8. ----
    {
      const int set = wid >> a.gw_shift, ki = wid & (GW - 1), nset = kWarps >> a.gw_shift;
      const unsigned char* bp0 = xterm + (size_t)(g8 < 3 ? g8 : 0) * pstride + (size_t)t4 * 4 + (size_t)ki * 32;
      const int trip = (nk - ki + GW - 1) >> a.gw_shift;  // K blocks of this warp
      const uint32_t kstep = (uint32_t)GW * 32u;
      uint32_t xb0[XB ? 32 : 1], xb1[XB ? 32 : 1];
      if (XB) {
#pragma unroll
        for (int u = 0; u < 32; ++u) {
          xb0[u] = xb1[u] = 0u;
          if (u < trip && g8 < 3) {
            xb0[u] = *reinterpret_cast<const uint32_t*>(bp0 + (size_t)u * kstep);
            xb1[u] = *reinterpret_cast<const uint32_t*>(bp0 + (size_t)u * kstep + 16);
          }
        }
      }
      for (int g = set; g < n_gu; g += nset) {
        int slot;
        uint32_t par;
        NP_CK(g * 5);
        slot_of(gseq + g, a.ng_magic, ng, slot, par);
        if (lane == 0) wait_group(gseq + g, &full_bar[slot], par, armed, ok, a.status);
        __syncwarp();
        NP_CK(g * 5 + 1);
        uint32_t ap = ring + (uint32_t)slot * a.group_bytes + a1_off + (uint32_t)ki * 32u;
        float c[4][4];
#pragma unroll
        for (int u = 0; u < 4; ++u) c[u][0] = c[u][1] = c[u][2] = c[u][3] = 0.f;
        if (XB) {
          // K blocks past this warp's last one multiply by zero operands: a fixed trip count keeps the loop
          // free of branches (their A tiles are read from the group's first K block)
#pragma unroll
          for (int it = 0; it < 32; it += 4) {
            if (it < trip) {  // warp-uniform; four independent chains, the four loads before the four mma (eight
                              // chains cost registers and measured 271 us per 32 layers against 250)
              uint32_t af[4][4];
#pragma unroll
              for (int u = 0; u < 4; ++u) ldmatrix_x4(af[u], ap + (it + u < trip ? (uint32_t)(it + u) * kstep : 0u));
#pragma unroll
              for (int u = 0; u < 4; ++u) mma_bf16_16816(c[u], af[u], xb0[it + u], xb1[it + u]);
            }
          }
        } else {
          const unsigned char* bp = bp0;
          int it = 0;
          for (; it + 4 <= trip; it += 4) {  // four independent chains; every load of the round before any mma
            uint32_t af[4][4], b0[4], b1[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              ldmatrix_x4(af[u], ap + (uint32_t)u * kstep);
              b0[u] = *reinterpret_cast<const uint32_t*>(bp + (size_t)u * kstep);
              b1[u] = *reinterpret_cast<const uint32_t*>(bp + (size_t)u * kstep + 16);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) mma_bf16_16816(c[u], af[u], g8 < 3 ? b0[u] : 0u, g8 < 3 ? b1[u] : 0u);
            ap += 4 * kstep;
            bp += 4 * (size_t)kstep;
          }
          for (; it < trip; ++it) {
            uint32_t af[4];
            ldmatrix_x4(af, ap);
            const uint32_t b0 = *reinterpret_cast<const uint32_t*>(bp), b1 = *reinterpret_cast<const uint32_t*>(bp + 16);
            mma_bf16_16816(c[0], af, g8 < 3 ? b0 : 0u, g8 < 3 ? b1 : 0u);
            ap += kstep;
            bp += kstep;
          }
        }
        NP_CK(g * 5 + 2);
        // C: [0], [1] = (vector g8, terms 2 t4, 2 t4 + 1); [2], [3] = (vector g8 + 8, same terms).  Columns 3-7 of B
        // are zero, so a lane's two columns add up to its share of the three terms: terms 0 + 1 in lane t4 = 0,
        // term 2 in lane t4 = 1, nothing in the others.
        float lo = ((c[0][0] + c[1][0]) + (c[2][0] + c[3][0])) + ((c[0][1] + c[1][1]) + (c[2][1] + c[3][1]));
        float hi = ((c[0][2] + c[1][2]) + (c[2][2] + c[3][2])) + ((c[0][3] + c[1][3]) + (c[2][3] + c[3][3]));
        lo += __shfl_xor_sync(0xffffffffu, lo, 1);
        hi += __shfl_xor_sync(0xffffffffu, hi, 1);
        if (t4 == 0) {
          float* pp = part + ((size_t)g * GW + ki) * VG;
          if (g8 < VG) pp[g8] = lo;
          if (g8 + 8 < VG) pp[g8 + 8] = hi;
        }
        NP_CK(g * 5 + 3);
        __syncwarp();
        if (lane == 0) mbar_arrive_n(&empty_bar[slot], (uint32_t)nset);  // the set's GW warps stand for all kWarps
        NP_CK(g * 5 + 4);
      }
    }
    NP_TR(3);
    NP_CK(30);
    if (nrows > 0) {
      if (lane == 0) {
        npp::mbar_arrive(&p1_bar);
        wait_or_flag(&act_bar, nx & 1u, ok, a.status);
      }
      __syncwarp();
      ++nx;
    }
    NP_TR(4);
    NP_CK(31);
    // ---- phase 2: y[cols] += a_i * downT[s_i][cols]: [16 columns x VG rows] x [a as 3 terms], this warp's
    //      column tiles mt = wid + kWarps j, accumulated over the layer's down groups ----
    float acc[KS][4];
#pragma unroll
    for (int j = 0; j < KS; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;
    for (int g = 0; g < n_dn; ++g) {
      int slot;
      uint32_t par;
      NP_CK(32 + g * 3);
      slot_of(gseq + n_gu + g, a.ng_magic, ng, slot, par);
      if (lane == 0) wait_group(gseq + n_gu + g, &full_bar[slot], par, armed, ok, a.status);
      __syncwarp();
      NP_CK(33 + g * 3);
      // B: column n = term n of the activations of rows (g << gs) + k; rows past the group are not its own: zero
      uint32_t b0 = 0u, b1 = 0u;
      if (g8 < 3) {
        const uint16_t* ap = aterm + (size_t)g8 * apad + (g << gs) + 2 * t4;
        if (2 * t4 < VG) b0 = *reinterpret_cast<const uint32_t*>(ap);
        if (VG == 16) b1 = *reinterpret_cast<const uint32_t*>(ap + 8);
      }
      const uint32_t dbase = ring + (uint32_t)slot * a.group_bytes + a2_off + (uint32_t)wid * 32u;
      // no guard on the tile index: a tile past the slice's end is computed from the last valid
      // tile's bytes and never looked at, which keeps the loop free of branches
#pragma unroll
      for (int j0 = 0; j0 < KS; j0 += 8) {  // eight loads, then their eight mma
        uint32_t af[8][4];
#pragma unroll
        for (int u = 0; u < 8; ++u) ldmatrix_x4_trans(af[u], dbase + (uint32_t)min((j0 + u) * kWarps, nk - 1 - wid) * 32u);
#pragma unroll
        for (int u = 0; u < 8; ++u) mma_bf16_16816(acc[j0 + u], af[u], b0, b1);
      }
      __syncwarp();
      if (lane == 0) npp::mbar_arrive(&empty_bar[slot]);
      NP_CK(34 + g * 3);
    }
    gseq += (unsigned int)(n_gu + n_dn);
    NP_TR(5);

    // ---- this block's partial MLP_l(x_l) over its column slice ----
    if (kFix && (li + 1 < nl || fin)) {
      // Between layers of the launch (and behind the last one where the launch ends the stack): counted fixed-point sums, straight from the accumulators.  One 64-bit
      // reduction per column carries the value and this block's arrival (a row group without rows still
      // counts); a warp's adds leave as soon as its own tiles are done.
      unsigned long long* zacc = a.zfix + ((size_t)((li & 1) * kFixRep + r % kFixRep)) * D + qoff;
      if (li == 0) {  // the launch's first adds: every block of the slice has read what the sets held before
        if (lane == 0 && *ok) {
          const unsigned int target = a.bar_base + (unsigned int)R;
          bool arrived = false;
          for (uint32_t spin = 0; spin < npp::kSpinLimit && !arrived; ++spin) {
            unsigned int v;
            asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(a.bars + q * kBarStride) : "memory");
            arrived = (int)(v - target) >= 0;
          }
          if (!arrived) {
            *ok = 0;
            atomicOr(a.status, npp::kStatTimeout);
          }
        }
        __syncwarp();
      }
#pragma unroll
      for (int j = 0; j < KS; ++j) {
        // acc[j]: [0], [1] = (column g8 of tile mt, terms 2 t4, 2 t4 + 1); [2], [3] = (column g8 + 8, same terms)
        // (columns 3-7 of B are zero: lanes t4 = 0 and 1 hold the three terms between them)
        float lo = acc[j][0] + acc[j][1];
        float hi = acc[j][2] + acc[j][3];
        lo += __shfl_xor_sync(0xffffffffu, lo, 1);
        hi += __shfl_xor_sync(0xffffffffu, hi, 1);
        const int mt = wid + kWarps * j;
        if (t4 < 2 && mt < nk) {  // lane t4 = 0 adds column g8, lane t4 = 1 column g8 + 8
          const float y = t4 == 0 ? lo : hi;
          long long fx = 0;
          if (fabsf(y) < kFixLimit) fx = __float2ll_rn(y * (float)(1u << kFixShift));
          else atomicOr(a.status, kStatRange);  // also a NaN: the sum would not mean anything
          red_add_u64(zacc + mt * 16 + g8 + 8 * t4, (unsigned long long)fx + (1ull << 56));
        }
      }
      NP_TR(6);
      NP_TR(7);
      continue;
    }
    // The launch's last layer: the three terms are added up and staged in shared memory, so that the
    // reductions to the stack's fp32 accumulator are 16 bytes wide.
#pragma unroll
    for (int j = 0; j < KS; ++j) {
      float lo = acc[j][0] + acc[j][1];
      float hi = acc[j][2] + acc[j][3];
      lo += __shfl_xor_sync(0xffffffffu, lo, 1);
      hi += __shfl_xor_sync(0xffffffffu, hi, 1);
      const int mt = wid + kWarps * j;
      if (t4 == 0 && mt < nk) {
        ybuf[mt * 16 + g8] = lo;
        ybuf[mt * 16 + g8 + 8] = hi;
      }
    }
    consumer_sync();
    if (nrows > 0) {
      float* yacc = a.zbuf[l % 3] + (size_t)(r % kZRep) * D + qoff;
#pragma unroll
      for (int j = 0; j < J4; ++j) {
        const int c = tid + j * kThreads;
        if (c < nf4) red_add_v4(yacc + 4 * c, reinterpret_cast<const float4*>(ybuf)[c]);
      }
    }
    if (!kFix && li + 1 < nl) {
      // fp32 form, publish: every warp waits for its own adds (the lanes' adds precede lane 0's fence), then
      // one thread counts the block in
      __syncwarp();
      if (lane == 0) __threadfence();
      NP_TR(6);
      consumer_sync();  // every warp's fence is behind it: the count is ordered after all of the block's adds
      if (tid == 0) atomicAdd(a.bars + q * kBarStride, 1u);
      NP_TR(7);
    }
  }
  // ---- the launch ends the stack: the blocks of row group 0 wait for the last layer's sums like a next layer
  //      would and leave x_L (no kernel behind this one has to add the accumulator copies up) ----
  if (fin && r == 0) {
    const unsigned long long* zw = a.zfix + (size_t)((nl - 1) & 1) * kFixRep * D + qoff;
#pragma unroll
    for (int j = 0; j < J4; ++j) {
      const int c = tid + j * kThreads;
      if (c >= nf4) continue;
      unsigned long long sum[4] = {0ull, 0ull, 0ull, 0ull};
      bool done = !*ok;
      for (uint32_t spin = 0; spin < npp::kSpinLimit && !done; ++spin) {
        unsigned long long w[kFixRep][4];
#pragma unroll
        for (int rep = 0; rep < kFixRep; ++rep) {
          const unsigned long long* wp = zw + (size_t)rep * D + 4 * c;
          ld_relaxed_v2u64(wp, w[rep][0], w[rep][1]);
          ld_relaxed_v2u64(wp + 2, w[rep][2], w[rep][3]);
        }
        done = true;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          sum[e] = 0ull;
#pragma unroll
          for (int rep = 0; rep < kFixRep; ++rep) sum[e] += w[rep][e];
          done = done && ((((long long)(sum[e] - zprev[j][e])) + (1ll << 55)) >> 56) == (long long)R;
        }
      }
      if (!done && *ok) {
        *ok = 0;
        atomicOr(a.status, npp::kStatTimeout);
      }
      float zv[4];
#pragma unroll
      for (int e = 0; e < 4; ++e)
        zv[e] = done ? __ll2float_rn((long long)(sum[e] - zprev[j][e]) - ((long long)R << 56)) * (1.f / (float)(1u << kFixShift)) : 0.f;
      reinterpret_cast<float4*>(a.x_out + qoff)[c] =
          make_float4(xown[j].x + zv[0], xown[j].y + zv[1], xown[j].z + zv[2], xown[j].w + zv[3]);
    }
  }
}

bool plan(const Dims& d, int sm_count, Plan* p) {
  if (d.D % (16 * kQ) || sm_count < kQ) return false;
  const int Ds = d.D / kQ;
  const int nk = Ds / 16;
  const int ks = (nk + kWarps - 1) / kWarps;
  if (ks > 32) return false;
  const int R = sm_count / kQ;
  if (R > kMaxR) return false;
  const size_t pstride = (size_t)Ds * 2 + kPad;
  const int max_rows = (d.C + R - 1) / R;  // whatever the active count turns out to be
  // a group: VG vectors (a power of two, at most the 16 rows of an MMA tile), up to kGroupTarget bytes
  size_t group_target = kGroupTarget;
#ifdef NP_TUNE
  if (const char* e = getenv("NP_SL_GT")) group_target = (size_t)atoi(e) * 1024;
#endif
  int vg_shift = 1;
  while (vg_shift < 4 && ((size_t)2 << vg_shift) * pstride <= group_target) ++vg_shift;
  const int VG = 1 << vg_shift;
  const size_t group_bytes = (size_t)VG * pstride;
  const size_t budget = 227 * 1024 - 2048;  // static shared memory of the kernel
  const int apad = ((max_rows + 15) & ~15) + 16;
  const int n_gu_max = (2 * max_rows + VG - 1) / VG;
  // phase 1 deals a layer's gate|up groups to sets of GW warps: as many sets as the expected share has groups
  const long long expect = std::min<long long>(d.C, std::max(1, d.k));
  const int n_gu_typ = (int)((2 * ((expect + R - 1) / R) + VG - 1) / VG);
  // ... but never a warp alone on a long K range: with more groups than warps (70B shape: ten groups of eight
  // 4 KB vectors) one warp per group walks through all 128 K blocks twice per layer; pairs walk through 64 three
  // times (1.51 ms per 80 layers against 1.58).  Four warps per group
  // measured worse at every shape (70B 1.82 ms, 13B 449 us against 357, 7B 261 us against 248): the layer's groups
  // are then worked on one or two at a time, and each has to have landed whole.
  int gw_shift = 3;
  while (gw_shift > 0 && (kWarps >> gw_shift) < n_gu_typ) --gw_shift;
  if (gw_shift == 0 && nk >= 64) gw_shift = 1;
#ifdef NP_TUNE
  if (const char* e = getenv("NP_SL_GW")) gw_shift = std::max(0, std::min(3, atoi(e)));
#endif
  const int GW = 1 << gw_shift;
  // everything but the ring and the slot cache; the cache (the slots of a launch's rows) takes a minimum first
  // and, once the ring's slots are counted, whatever is left, so that a launch can span more layers
  const size_t fixed0 = 3 * pstride + (size_t)Ds * 4 + (size_t)n_gu_max * GW * VG * 4 + (size_t)(3 * apad + (apad & 1)) * 2 + 64;
  const size_t cache_min = std::max<size_t>(4 * (size_t)max_rows, std::min<size_t>(8192, 4 * (size_t)max_rows * 8));
  if (fixed0 + cache_min + 3 * group_bytes > budget) return false;
  int ng = (int)std::min<size_t>(kMaxGroups, (budget - fixed0 - cache_min) / group_bytes);
  if (d.ring_stages >= 2) ng = std::max(3, std::min(ng, d.ring_stages));
  const size_t cache_bytes = std::min<size_t>(budget - fixed0 - (size_t)ng * group_bytes, 4 * (size_t)max_rows * kMaxLayers);
  p->run_layers = (int)std::max<size_t>(1, std::min<size_t>(kMaxLayers, cache_bytes / (4 * (size_t)max_rows)));
  p->slot_cache_rows = p->run_layers * max_rows;
  const size_t fixed = fixed0 + (size_t)p->slot_cache_rows * 4;
  // Groups in flight per block.  Where the hand-over between layers has no fence (counted sums) the producer runs
  // as far ahead as the ring and its pacing history allow (7B shape: 284 us per 32 layers with one group in
  // flight, 274 with five; 13B shape: 390 us per 40 layers against 357).  The fp32 form keeps about 40 KB in
  // flight: a deeper burst queues in front of its fence and of the short loads behind it (13B shape, when it
  // still used this form: 385 us with one 41 KB group in flight, 411 with two or more).
  int window = ks <= kFixMaxKS ? std::max(1, std::min(ng - 1, kHist - 1)) : std::max(1, std::min(ng - 1, (int)(40 * 1024 / group_bytes)));
  if (ng <= 3) window = 1;  // a ring of three large groups (70B shape, 66 KB each): 1.36 ms per 80 layers with one in flight, 1.39 with two
#ifdef NP_TUNE  // development builds only: geometry from the environment
  if (const char* e = getenv("NP_SL_NG")) ng = std::max(2, std::min(ng, atoi(e)));
  if (const char* e = getenv("NP_SL_WIN")) window = std::min(atoi(e), std::min(kHist - 1, ng - 1));
  if (getenv("NP_SL_NOFILL")) window = -1;
#endif
  p->R = R;
  p->ks = ks <= 8 ? 8 : (ks <= 16 ? 16 : 32);
  p->vg_shift = vg_shift;
  p->gw_shift = gw_shift;
  p->ng = ng;
  p->window = window;
  p->max_rows = max_rows;
  p->xch_stride = (2 * max_rows + 1 + 15) / 16 * 16;
  p->group_bytes = group_bytes;
  p->smem = (size_t)ng * group_bytes + fixed;
  return true;
}

bool supported(const Dims& d, int sm_count) {
  Plan p;
  return plan(d, sm_count, &p);
}

bool counted_handover(const Dims& d, int sm_count) {
  Plan p;
  return plan(d, sm_count, &p) && p.ks <= kFixMaxKS;
}

size_t xch_words(const Dims& d, int sm_count) {
  Plan p;
  if (!plan(d, sm_count, &p)) return 16;
  return (size_t)2 * (p.R * kQ) * p.xch_stride;
}
size_t zfix_words(const Dims& d) { return (size_t)2 * kFixRep * d.D; }
size_t bar_words() { return (size_t)kQ * kBarStride; }

template <int KS, bool XB>
static cudaError_t launch_one(const KArgs& ka, size_t sm, int grid_x, cudaStream_t s) {
  auto kfn = k_mlp_slices<KS, XB>;
  cudaError_t e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
  if (e != cudaSuccess) return e;
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kfn, kBlock, sm);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorCooperativeLaunchTooLarge;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid_x);
  cfg.blockDim = dim3(kBlock);
  cfg.dynamicSmemBytes = sm;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;  // all blocks co-resident: no wait can starve
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kfn, ka);
}

cudaError_t launch(const Dims& d, const ChainArgs& a, State* st, cudaStream_t s, int sm_count) {
  Plan p;
  if (!plan(d, sm_count, &p) || !st || !st->zfix || !st->bars || !st->xch) return cudaErrorInvalidValue;
  cudaError_t e = cudaSuccess;
  for (int l0 = a.l_begin; l0 < a.l_end; l0 += p.run_layers) {
    KArgs ka;
    ka.gate = static_cast<const unsigned char*>(a.gate);
    ka.up = static_cast<const unsigned char*>(a.up);
    ka.downT = static_cast<const unsigned char*>(a.downT);
    ka.slots = a.active_slots;
    ka.counters = a.counters;
    ka.x_bf16 = l0 == 0 ? static_cast<const uint16_t*>(a.x_bf16) : nullptr;
    for (int i = 0; i < 2; ++i) ka.xbuf[i] = a.xbuf[i];
    // the launch that ends the stack leaves the result itself where the hand-over is counted
    ka.x_out = (p.ks <= kFixMaxKS && std::min(a.l_end, l0 + p.run_layers) == a.l_end) ? a.x_out : nullptr;
    st->wrote_out = ka.x_out != nullptr;
    for (int i = 0; i < 3; ++i) ka.zbuf[i] = a.zbuf[i];
    ka.zfix = st->zfix;
    ka.bars = st->bars;
    ka.bar_base = st->bar_base;
    ka.xch = st->xch;
    ka.status = a.status;
    ka.seq_base = st->seq_base;
    ka.ng_magic = (unsigned int)((0x100000000ull + p.ng - 1) / p.ng);
    ka.l_begin = l0;
    ka.l_end = std::min(a.l_end, l0 + p.run_layers);
    ka.D = d.D;
    ka.C = d.C;
    ka.check = a.check;
    ka.vg_shift = p.vg_shift;
    ka.gw_shift = p.gw_shift;
    ka.ng = p.ng;
    ka.window = p.window;
    ka.max_rows = p.max_rows;
    ka.xch_stride = p.xch_stride;
    ka.group_bytes = (uint32_t)p.group_bytes;
    const int nl = ka.l_end - ka.l_begin;
    // the counters and stamps only ever grow; the next launch starts where this one ends
    if (p.ks <= kFixMaxKS) st->bar_base += (nl > 1 || ka.x_out) ? (unsigned int)p.R : 0u;
    else if (nl > 1) st->bar_base += (unsigned int)(nl - 1) * (unsigned int)p.R;
    st->seq_base += (unsigned int)nl + 1u;
    const bool xb = ((d.D / kQ / 16) >> p.gw_shift) <= 32 && p.ks <= 16;  // phase 1's B operands fit a warp's registers
    if (p.ks == 8) e = xb ? launch_one<8, true>(ka, p.smem, p.R * kQ, s) : launch_one<8, false>(ka, p.smem, p.R * kQ, s);
    else if (p.ks == 16) e = xb ? launch_one<16, true>(ka, p.smem, p.R * kQ, s) : launch_one<16, false>(ka, p.smem, p.R * kQ, s);
    else e = launch_one<32, false>(ka, p.smem, p.R * kQ, s);
    if (e != cudaSuccess) return e;
  }
  return e;
}

}  // namespace chain_slices
}  // namespace npi
