// Stage 4 over a run of layers in one resident kernel, whole rows per block, blocks in
// clusters of four (one sequence).
//
//   x_{l+1} = x_l + sum_{i in act_l} silu(gate_l[s_i].n_l) * (up_l[s_i].n_l) * downT_l[s_i],
//   n_l = x_l / sqrt(mean(x_l^2) + 1e-6)
//
// (Section 3.4: the sparse MLP reads each active row through the slot map.)
//
// A layer is one trip through HBM (its active rows, 4 us at the 7B shape) and one all-reduce
// of a D-vector over all blocks; what a resident kernel over many layers can lose is the
// latency of that all-reduce.  Here it is cut in three:
//   * a block owns whole rows (about 8 of a layer's 1101), so the dot products of phase 1 and
//     the activations need nothing from other blocks;
//   * the blocks of a cluster first reduce their partial output vectors among themselves
//     through distributed shared memory (rank o collects columns [o D/4, (o+1) D/4) of all
//     four), so only a quarter of a vector per block goes to the global accumulator, and
//     every accumulator word is added to by one block per cluster;
//   * after the grid-wide counter of its column range has filled, rank o reads that range of
//     the sum, forms x_{l+1} there (it keeps its range of x_l in registers), splits it into
//     the three bf16 terms phase 1 multiplies with and writes them, with its share of
//     sum(x^2), into the shared memory of all four blocks.
// Phase 1 runs on mma.sync m16n8k16 (rows = 8 gate + 8 up rows, K = 16 columns per step and
// warp, columns = the three terms of x); phase 2 on the ALUs (a thread per 8 output columns).
// The rows come through a ring of row-sized pieces in shared memory, filled by 1-D bulk
// copies from a producer lane: gate and up rows of a tile of 8 rows, then the layer's down
// rows.  Cooperative launch with clusters: every block is resident.  Every wait is bounded
// (kStatTimeout on expiry); after one has run out the later ones are skipped, and every
// block still meets its cluster at the end, so no block leaves while a peer may write to it.
#include <algorithm>

#include "np_device.cuh"
#include "np_internal.h"
#include "np_pipe.cuh"

namespace npi {
namespace chain_rows {
using namespace npd;

#ifndef NP_ROWS_CS
#define NP_ROWS_CS 2
#endif
constexpr int kCS = NP_ROWS_CS;              // blocks per cluster
constexpr int kWarps = 16;                   // consumer warps
constexpr int kThreads = kWarps * 32;        // consumer threads
constexpr int kBlock = kThreads + 64;        // plus the producer warp (gate and up rows) and the mover warp (down rows)
constexpr int kDS = 2;                       // staging pieces of the down rows on their way into tensor memory
constexpr int kTmemCols = 512;               // tensor memory columns: two buffers (layer parity) of 16 rows x 16 columns
constexpr int kTmemRows = 16;                // down rows of a block and layer that a buffer holds
constexpr int kZR = kCS >= 4 ? 4 : 8;        // copies of an accumulator: adds to one address queue up in L2 (about 30 ns
                                             // each), so the clusters spread over the copies and the readers add them up
constexpr int kMaxRows = 16;                 // rows of a block and layer, at most (one MMA row block of gate rows, one of up rows)
constexpr int kMaxSlots = 32;                // ring pieces
constexpr int kMaxLayers = 64;               // layers per launch
constexpr int kPad = 16;                     // bytes between pieces: rows of a tile fall into different banks

struct KArgs {
  const unsigned char* gate;  // layer 0 of each row buffer; layer stride = C * D * 2 bytes
  const unsigned char* up;
  const unsigned char* downT;
  const int32_t* slots;       // active_slots [L][C]
  const int32_t* counters;    // [L][NP_N_COUNTERS]
  const uint16_t* x_bf16;     // the stack's input (run that starts at layer 0), or NULL
  const float* x_in;          // else x_{l_begin} = x_in + sum of the kZRep copies of z_in (z_in may be NULL)
  const float* z_in;
  float* x_out;               // x_{l_end} at the end of the run
  float* zclr_a;              // accumulators (kZRep copies of [D]) the next kernel expects cleared
  float* zclr_b;
  float* z4;                  // [4][kZR][D] accumulators of this kernel (kZR copies each), used in rotation, cleared two layers ahead
  unsigned int* cnt;          // [kCS] arrival counters, one per column range; they only grow
  int32_t* status;
  unsigned int cnt_base;      // value of the counters before this launch
  unsigned int seq;           // layers run by earlier launches (position in the rotation of z4)
  unsigned int ns_magic;      // ceil(2^32 / ns)
  int l_begin, l_end, D, C, check, ns, max_rows, slot_cache_rows;
};

#ifdef NP_TRACE  // development builds only: clock stamps of thread 0 of two blocks
#ifndef NP_RK_B
#define NP_RK_B 1
#endif
__device__ long long np_rows_clk[2][8][24];
extern "C" int np_debug_rows(void* out) { return (int)cudaMemcpyFromSymbol(out, np_rows_clk, sizeof(np_rows_clk)); }
#define RK(ev) do { if (threadIdx.x == 0 && (blockIdx.x == 0 || blockIdx.x == NP_RK_B) && li >= 8 && li < 16) np_rows_clk[blockIdx.x ? 1 : 0][li - 8][ev] = clock64(); } while (0)
__device__ long long np_rows_pc[2][8][24];  // [0]: producer lane 0 (batch issued), [1]: consumer thread 0 (down row r waited)
extern "C" int np_debug_rows_pc(void* out) { return (int)cudaMemcpyFromSymbol(out, np_rows_pc, sizeof(np_rows_pc)); }
#define PK(who, ev) do { if ((threadIdx.x & 31) == 0 && blockIdx.x == 0 && li >= 8 && li < 16 && (ev) < 24) np_rows_pc[who][li - 8][ev] = clock64(); } while (0)
__device__ unsigned long long np_rows_all[160][4][8];  // per block, layers 8-11: globaltimer stamps of thread 0
extern "C" int np_debug_rows_all(void* out) { return (int)cudaMemcpyFromSymbol(out, np_rows_all, sizeof(np_rows_all)); }
__device__ __forceinline__ unsigned long long gtime() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
#define AK(ev) do { if (threadIdx.x == 0 && blockIdx.x < 160 && li >= 8 && li < 12) np_rows_all[blockIdx.x][li - 8][ev] = gtime(); } while (0)
#define AKV(ev, val) do { if (threadIdx.x == 0 && blockIdx.x < 160 && li >= 8 && li < 12) np_rows_all[blockIdx.x][li - 8][ev] = (unsigned long long)(val); } while (0)
#else
#define RK(ev) do { } while (0)
#define PK(who, ev) do { } while (0)
#define AK(ev) do { } while (0)
#define AKV(ev, val) do { } while (0)
#endif

__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory"); }
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// the address of the same shared-memory location in block `rank` of this cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_cluster_f4(uint32_t addr, float4 v) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ void st_cluster_u4(uint32_t addr, uint4 v) {
  asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
// arrival on a peer's mbarrier; orders this thread's earlier writes (and, behind a __syncwarp,
// its warp's) to the peer before the arrival
__device__ __forceinline__ void mbar_arrive_peer(uint32_t addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(addr) : "memory");
}
// 1-D bulk copy from this block's shared memory into a peer's; the bytes are reported to the peer's mbarrier
__device__ __forceinline__ void bulk_s2peer(uint32_t dst_cluster_addr, const void* src_smem, uint32_t bytes, uint32_t bar_cluster_addr) {
  asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_cluster_addr),
               "r"(npp::smem_addr(src_smem)), "r"(bytes), "r"(bar_cluster_addr)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(npp::smem_addr(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void red_add_v4(float* p, float4 v) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
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

// ---- tensor memory as a parking place: 128 lanes x 512 columns of 32 bits per SM, otherwise unused here ----
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
// the mbarrier gets one arrival when all tcgen05 operations issued so far by this thread are done
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(npp::smem_addr(bar)) : "memory");
}
// 2 KB of shared memory (128 rows of 16 bytes, contiguous: 8-row core matrices 128 bytes apart, no swizzle)
__device__ __forceinline__ uint64_t tc_rows16_desc(const void* p) {
  const uint64_t addr = (uint64_t)(npp::smem_addr(p) & 0x3ffffu) >> 4;
  return addr | ((uint64_t)(2048 >> 4) << 16)  // leading byte offset: not used by a 16-byte wide matrix
         | ((uint64_t)(128 >> 4) << 32)        // stride byte offset: from one group of 8 rows to the next
         | (1ull << 46);                       // descriptor version of this architecture; layout type 0 = no swizzle
}
// shared memory -> tensor memory: row i of the matrix goes to lane i, columns [col, col + 4)
__device__ __forceinline__ void tc_cp_128x16B(uint32_t taddr, uint64_t desc) {
  asm volatile("tcgen05.cp.cta_group::1.128x128b [%0], %1;" ::"r"(taddr), "l"(desc) : "memory");
}
// tensor memory -> registers: lane i of the warp reads columns [col, col + 4) of lane (taddr.lane + i)
__device__ __forceinline__ uint4 tc_ld4(uint32_t taddr) {
  uint4 v;
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(taddr));
  return v;
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Bounded waits.  Once any wait of the block has run out (*ok == 0) every later wait is
// skipped, so no barrier is ever left short of threads.
__device__ __forceinline__ void wait_or_flag(uint64_t* bar, uint32_t parity, volatile int* ok, int32_t* status) {
  if (npp::mbar_try_wait(bar, parity)) return;  // the usual case: already complete
  if (!*ok) return;
  if (!npp::mbar_wait(bar, parity)) {
    *ok = 0;
    atomicOr(status, npp::kStatTimeout);
  }
}
__device__ __forceinline__ void wait_cluster_or_flag(uint64_t* bar, uint32_t parity, volatile int* ok, int32_t* status) {
  if (mbar_try_wait_cluster(bar, parity)) return;
  if (!*ok) return;
  for (uint32_t i = 0; i < npp::kSpinLimit; ++i)
    if (mbar_try_wait_cluster(bar, parity)) return;
  *ok = 0;
  atomicOr(status, npp::kStatTimeout);
}

// ring slot and use parity of piece number v of the launch (exact for v < 2^32 / ns)
__device__ __forceinline__ void slot_of(unsigned int v, unsigned int magic, int ns, int& slot, uint32_t& par) {
  const unsigned int qd = __umulhi(v, magic);
  slot = (int)(v - qd * (unsigned int)ns);
  par = qd & 1u;
}

// three packed terms of eight consecutive values
struct Terms8 {
  uint4 t[3];
};
__device__ __forceinline__ Terms8 split8(const float (&v)[8]) {
  uint32_t a[8][3];
#pragma unroll
  for (int e = 0; e < 8; ++e) split3(v[e], a[e][0], a[e][1], a[e][2]);
  Terms8 r;
#pragma unroll
  for (int k = 0; k < 3; ++k)
    r.t[k] = make_uint4(pack_hi16(a[0][k], a[1][k]), pack_hi16(a[2][k], a[3][k]), pack_hi16(a[4][k], a[5][k]),
                        pack_hi16(a[6][k], a[7][k]));
  return r;
}

// KB: 16-wide K blocks per warp in phase 1, D / 16 / kWarps
template <int KB>
__global__ void __launch_bounds__(kBlock, 1) k_mlp_rows(KArgs a) {
  extern __shared__ __align__(128) unsigned char csm[];
  __shared__ __align__(8) uint64_t full_bar[kMaxSlots];   // the piece has landed
  __shared__ __align__(8) uint64_t empty_bar[kMaxSlots];  // every consumer warp is done with it
  __shared__ __align__(8) uint64_t ds_full[kDS];          // a down row has landed in its staging piece
  __shared__ __align__(8) uint64_t ds_free[kDS];          // ... and has been copied on into tensor memory
  __shared__ __align__(8) uint64_t tm_full[2];            // a layer's down rows are all in their tensor-memory buffer
  __shared__ __align__(8) uint64_t tm_empty[2];           // every consumer warp has read them
  __shared__ uint32_t s_tmem_base;
  __shared__ __align__(8) uint64_t rs_bar;                // the peers' partial sums of this block's column range are here
  __shared__ __align__(8) uint64_t ag_bar;                // x of the next layer is here, all ranges
  __shared__ float part[2][kMaxRows][kWarps];             // partial dot products: gate | up, by row and warp
  __shared__ float act[kMaxRows];                         // a_i of the block's rows
  __shared__ __align__(16) float ssq_part[kCS][kWarps / kCS][4];  // sum(x^2) by column range and warp of its owner (16-byte granules: first float)
  __shared__ __align__(16) float ag_ssq[kWarps / kCS][4];         // this block's own, on their way to the cluster
  __shared__ int s_ok;
  __shared__ int lay_rb[kMaxLayers];       // first active-list index of this block, per layer
  __shared__ int lay_pre[kMaxLayers + 1];  // rows of this block before each layer (virtual row index)

  const int D = a.D, chunks = D >> 3;
  const uint32_t row_bytes = (uint32_t)D * 2u;
  const uint32_t pstride = row_bytes + kPad;    // ring piece
  const uint32_t xt_stride = row_bytes + kPad;  // one term of x
  const size_t layer_bytes = (size_t)a.C * row_bytes;
  const int seg = D / kCS, seg_chunks = chunks / kCS;  // a rank's column range, in values and in 8-value chunks
  const int wpo = seg_chunks >> 5;                     // warps that hold a column range (its owner's threads)
  const int ns = a.ns;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int G = gridDim.x, NCL = G / kCS;
  const uint32_t rank = cluster_ctarank();
  const int cluster = blockIdx.x / kCS;
  const int nl = a.l_end - a.l_begin;
  // dynamic shared memory: ring | x as 3 bf16 terms | peers' partial sums of this block's range | slots
  unsigned char* dstage = csm + (size_t)ns * pstride;                         // [kDS][pstride] down rows on their way into tensor memory
  unsigned char* xt = dstage + (size_t)kDS * pstride;                         // [3][xt_stride]
  float* rs_buf = reinterpret_cast<float*>(xt + 3 * (size_t)xt_stride);       // [kCS - 1][seg]: peer p's sums sit at p - (p > rank)
  float* y_stage = rs_buf + (size_t)(kCS - 1) * seg;                          // [kCS - 1][seg] this block's partial sums for its peers, on their way out
  // the terms of x_{l+1} of this block's range, on their way out.  With four blocks they go where the peers' sums
  // were (those have been added up by then, and the next ones only come from peers that have taken these terms);
  // with two blocks that space is too small
  unsigned char* ag_own = reinterpret_cast<unsigned char*>(y_stage + (size_t)(kCS - 1) * seg);
  unsigned char* ag_stage = kCS >= 4 ? reinterpret_cast<unsigned char*>(rs_buf) : ag_own;  // [3][seg * 2]
  int* slot_cache = reinterpret_cast<int*>(ag_own + (kCS >= 4 ? 0 : 3 * (size_t)seg * 2));  // this block's slots, virtual row order
  volatile int* ok = &s_ok;

  // ---- this block's share of every layer of the run ----
  if (tid < nl) {
    int n = a.counters[(size_t)(a.l_begin + tid) * NP_N_COUNTERS + NP_CNT_ACTIVE];
    if (a.check && (n < 0 || n > a.C)) {
      atomicOr(a.status, kStatBadCount);
      n = 0;
    }
    const int rb = (int)(((long long)n * blockIdx.x) / G);
    const int re = (int)(((long long)n * (blockIdx.x + 1)) / G);
    if (re - rb > a.max_rows) atomicOr(a.status, kStatBadCount);  // more active rows than one sequence selects
    lay_rb[tid] = rb;
    lay_pre[tid + 1] = min(re - rb, a.max_rows);  // turned into a prefix sum below
  }
  if (tid == 0) {
    for (int s = 0; s < ns; ++s) {
      npp::mbar_init(&full_bar[s], 1);
      npp::mbar_init(&empty_bar[s], kWarps);
    }
    for (int i = 0; i < kDS; ++i) {
      npp::mbar_init(&ds_full[i], 1);
      npp::mbar_init(&ds_free[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      npp::mbar_init(&tm_full[i], 1);
      npp::mbar_init(&tm_empty[i], kWarps);
    }
    npp::mbar_init(&rs_bar, 1);  // armed by this block once per layer with the bytes it expects
    npp::mbar_init(&ag_bar, 1);
    npp::fence_barrier_init();
    s_ok = 1;
  }
  if (wid == kWarps + 1) {  // tensor memory: all of it (this kernel has the SM to itself); the address lands in shared memory
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(npp::smem_addr(&s_tmem_base)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (tid == 0) {
    lay_pre[0] = 0;
    for (int i = 0; i < nl; ++i) lay_pre[i + 1] += lay_pre[i];
  }
  __syncthreads();
  const int total_rows = min(lay_pre[nl], a.slot_cache_rows);
  for (int li = 0; li < nl; ++li) {
    const int nr = lay_pre[li + 1] - lay_pre[li];
    for (int i = tid; i < nr; i += kBlock) {
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
  // the peers' barriers are initialised before anybody writes to a peer
  cluster_sync_all();

  const uint32_t tmem_base = s_tmem_base;
  if (wid == kWarps) {
    // =========================== producer warp ===========================
    // The gate and up rows are requested in the order in which they are consumed: per layer its gate rows, then
    // its up rows.  A layer goes out at once, a lane per piece (one lane alone spends over 0.1 us per request).  A lane waits for its own slot: the slots of a batch are released in order by consumers that need
    // nothing from this batch, so the lanes may wait for one another at the end of a batch.
    unsigned int v0 = 0;
    bool good = true;
    // lane i < cnt requests the piece v0 + i from src
    auto issue = [&](const unsigned char* src, int cnt) {
      if (lane < cnt) {
        int s;
        uint32_t par;
        const unsigned int v = v0 + (unsigned int)lane;
        slot_of(v, a.ns_magic, ns, s, par);
        if (v >= (unsigned int)ns && !npp::mbar_wait(&empty_bar[s], par ^ 1u)) {
          atomicOr(a.status, npp::kStatTimeout);
          good = false;
        } else {
          npp::mbar_expect_tx(&full_bar[s], row_bytes);
          npp::bulk_g2s_stream(csm + (size_t)s * pstride, src, row_bytes, &full_bar[s], npp::policy_evict_first());
        }
      }
      good = __all_sync(0xffffffffu, good);
      v0 += (unsigned int)cnt;
    };
    for (int li = 0; li < nl && good; ++li) {
      const int vrow0 = lay_pre[li], nrows = min(lay_pre[li + 1], total_rows) - vrow0;
      const size_t lbase = (size_t)(a.l_begin + li) * layer_bytes;
      // a layer's pieces: its gate rows, then its up rows, a lane each
      const int j = lane < nrows ? lane : lane - nrows;
      const unsigned char* src = (lane < nrows ? a.gate : a.up) + lbase + (size_t)slot_cache[vrow0 + min(max(j, 0), max(nrows - 1, 0))] * row_bytes;
      if (nrows > 0) issue(src, 2 * nrows);
      PK(0, 0);
    }
  } else if (wid == kWarps + 1) {
    // =========================== mover warp ===========================
    // The down rows do not fit into the ring beside the gate and up rows (a block's rows of a layer are about 216 KB),
    // and what is fetched after x has arrived is late.  They go through two staging pieces into tensor memory, which
    // this kernel does not otherwise use: row r of a layer's share fills 16 columns of all 128 lanes (chunk c of 16
    // bytes sits in lane c % 128, columns 4 (c / 128) .. + 3), two buffers by layer parity.  One lane does it all:
    // request row k + 1, wait for row k, copy it on (4 copies of 2 KB), commit: the commit frees the staging piece,
    // and after a layer's last row it tells the consumers.
    if (lane == 0) {
      bool good = true;
      int li_n = 0, r_n = 0;    // the next row to request
      unsigned int kn = 0;      // its number within the launch
      auto rows_of = [&](int li) { return min(min(lay_pre[li + 1], total_rows) - lay_pre[li], kTmemRows); };
      auto request = [&]() {
        while (li_n < nl && r_n >= rows_of(li_n)) {
          ++li_n;
          r_n = 0;
        }
        if (li_n >= nl) return;
        const int s = (int)(kn % kDS);
        if (kn >= (unsigned int)kDS && !npp::mbar_wait(&ds_free[s], ((kn / kDS) & 1u) ^ 1u)) {
          atomicOr(a.status, npp::kStatTimeout);
          good = false;
          return;
        }
        npp::mbar_expect_tx(&ds_full[s], row_bytes);
        npp::bulk_g2s_stream(dstage + (size_t)s * pstride,
                             a.downT + (size_t)(a.l_begin + li_n) * layer_bytes + (size_t)slot_cache[lay_pre[li_n] + r_n] * row_bytes,
                             row_bytes, &ds_full[s], npp::policy_evict_first());
        ++kn;
        ++r_n;
      };
      request();
      unsigned int k = 0;
      for (int li = 0; li < nl && good; ++li) {
        const int nrows = rows_of(li), buf = li & 1;
        for (int r = 0; r < nrows && good; ++r, ++k) {
          request();  // the row after this one
          if (!good) break;
          const int s = (int)(k % kDS);
          if (!npp::mbar_wait(&ds_full[s], (k / kDS) & 1u)) {
            atomicOr(a.status, npp::kStatTimeout);
            good = false;
            break;
          }
          if (r == 0 && li >= 2 && !npp::mbar_wait(&tm_empty[buf], (uint32_t)((li >> 1) - 1) & 1u)) {  // the buffer's readers of two layers ago
            atomicOr(a.status, npp::kStatTimeout);
            good = false;
            break;
          }
          tc_fence_after();
          const uint32_t col = (uint32_t)(buf * (kTmemCols / 2) + r * 16);
          for (uint32_t j = 0; j < row_bytes / 2048u; ++j)
            tc_cp_128x16B(tmem_base + col + 4u * j, tc_rows16_desc(dstage + (size_t)s * pstride + (size_t)j * 2048));
          tc_commit(&ds_free[s]);
          if (r == nrows - 1) tc_commit(&tm_full[buf]);
        }
        if (nrows == 0 && good) {  // nothing to copy: the consumers still wait for the buffer's turn
          if (li >= 2 && !npp::mbar_wait(&tm_empty[buf], (uint32_t)((li >> 1) - 1) & 1u)) {
            atomicOr(a.status, npp::kStatTimeout);
            good = false;
          } else {
            npp::mbar_arrive(&tm_full[buf]);
          }
        }
      }
    }
  } else {
    // =========================== consumer warps ===========================
    const int g = lane >> 2, q = lane & 3;
    const bool has_chunk = tid < chunks;                 // a thread per 8 output columns
    const int owner = has_chunk ? tid / seg_chunks : -1; // whose column range this thread's columns are in
    const int lc = has_chunk ? tid - owner * seg_chunks : 0;  // the chunk's index inside that range
    const bool own = owner == (int)rank;                 // this thread works for the range this block owns
    const int ow = has_chunk ? (wid - owner * wpo) : 0;  // the warp's index among its range's warps

    // ---- x of the first layer of the run: every block computes all of it ----
    float xo[8];  // this thread's 8 values of x_l, kept by the owner's threads across layers
#pragma unroll
    for (int e = 0; e < 8; ++e) xo[e] = 0.f;
    if (has_chunk) {
      if (a.x_bf16) {
        const uint4 w = __ldg(reinterpret_cast<const uint4*>(a.x_bf16) + tid);
        xo[0] = bf16_lo(w.x), xo[1] = bf16_hi(w.x), xo[2] = bf16_lo(w.y), xo[3] = bf16_hi(w.y);
        xo[4] = bf16_lo(w.z), xo[5] = bf16_hi(w.z), xo[6] = bf16_lo(w.w), xo[7] = bf16_hi(w.w);
      } else {
        const float4 v0 = __ldcg(reinterpret_cast<const float4*>(a.x_in) + 2 * tid);
        const float4 v1 = __ldcg(reinterpret_cast<const float4*>(a.x_in) + 2 * tid + 1);
        xo[0] = v0.x, xo[1] = v0.y, xo[2] = v0.z, xo[3] = v0.w, xo[4] = v1.x, xo[5] = v1.y, xo[6] = v1.z, xo[7] = v1.w;
        if (a.z_in) {
#pragma unroll
          for (int r = 0; r < kZRep; ++r) {
            const float4 z0 = __ldcg(reinterpret_cast<const float4*>(a.z_in + (size_t)r * D) + 2 * tid);
            const float4 z1 = __ldcg(reinterpret_cast<const float4*>(a.z_in + (size_t)r * D) + 2 * tid + 1);
            xo[0] += z0.x, xo[1] += z0.y, xo[2] += z0.z, xo[3] += z0.w, xo[4] += z1.x, xo[5] += z1.y, xo[6] += z1.z, xo[7] += z1.w;
          }
        }
      }
      const Terms8 t8 = split8(xo);
#pragma unroll
      for (int k = 0; k < 3; ++k) *reinterpret_cast<uint4*>(xt + (size_t)k * xt_stride + (size_t)tid * 16) = t8.t[k];
      float ss = 0.f;
#pragma unroll
      for (int e = 0; e < 8; ++e) ss += xo[e] * xo[e];
      ss = warp_sum(ss);
      if (lane == 0) ssq_part[owner][ow][0] = ss;
    }
    consumer_sync();
    const uint32_t rs_bytes = (uint32_t)((kCS - 1) * seg * 4);
    const uint32_t ag_bytes = (uint32_t)(kCS * (3 * seg * 2 + wpo * 16));

    for (int li = 0; li < nl; ++li) {
      RK(0);
      if (li > 0) wait_cluster_or_flag(&ag_bar, (uint32_t)(li - 1) & 1u, ok, a.status);  // x_l and its sums are here
      RK(1);
      AK(0);
      if (wid == 0) PK(1, 20);
      if (tid == 0) {  // this layer's deliveries: the peers' partial sums, then x of the next layer
        npp::mbar_expect_tx(&rs_bar, rs_bytes);
        if (li < nl - 1) npp::mbar_expect_tx(&ag_bar, ag_bytes);
      }
      // ---- phase 1: gate / up dot products of this block's rows ----
      const int vrow0 = lay_pre[li], nrows = min(lay_pre[li + 1], total_rows) - vrow0;
      const unsigned int pbase = 2u * (unsigned int)vrow0;  // the layer's first piece in the ring: two per row
      const uint32_t ring = npp::smem_addr(csm);
      RK(2);
      // (the legacy tensor pipe takes about 9 clocks per MMA and sub-partition: 16 MMAs per warp and row block)
      if (nrows > 0) {
        // the layer's 2 nrows pieces: lane i waits for piece i
        if (lane < 2 * nrows) {
          int s;
          uint32_t par;
          slot_of(pbase + (unsigned int)lane, a.ns_magic, ns, s, par);
          wait_or_flag(&full_bar[s], par, ok, a.status);
        }
        __syncwarp();
        RK(16);
        // B operand: column n of the MMA is term n of x; lanes g < 3 hold term g at k = 2q, 2q+1 (b0) and 2q+8, 2q+9 (b1)
        const unsigned char* bp = xt + (size_t)(g < 3 ? g : 0) * xt_stride + ((size_t)(wid * KB) * 16 + 2 * q) * 2;
        const int mi = lane >> 3;
        if (nrows <= 8) {
          // one row block: rows 0-7 the gate rows, rows 8-15 the up rows.  ldmatrix row addresses: matrix mi = lane / 8
          // holds rows 8 (mi & 1) .. +7 of the A tile and k = 8 (mi / 2) .. +7 of the K block; rows past the end read
          // row 0 (their sums are dropped)
          const int jr = (lane & 7) < nrows ? (lane & 7) : 0;
          int s_a;
          uint32_t par_a;
          slot_of(pbase + (unsigned int)((mi & 1) * nrows + jr), a.ns_magic, ns, s_a, par_a);  // rows in consecutive pieces: no bank conflicts
          const uint32_t a_addr = ring + (uint32_t)s_a * pstride + (uint32_t)((wid * KB * 16 + (mi >> 1) * 8) * 2);
          float c[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};  // two chains: the MMAs of a chain are dependent
#pragma unroll
          for (int kb = 0; kb < KB; ++kb) {
            uint32_t af[4];
            ldmatrix_x4(af, a_addr + (uint32_t)kb * 32u);
            uint32_t b0 = *reinterpret_cast<const uint32_t*>(bp + kb * 32);
            uint32_t b1 = *reinterpret_cast<const uint32_t*>(bp + kb * 32 + 16);
            if (g >= 3) b0 = b1 = 0u;
            mma_bf16_16816(c[kb & 1], af, b0, b1);
          }
          // gate of row g = columns 0-2 of accumulator row g, up = of row g + 8; the columns sit in lanes q = 0, 1
          float gs = (c[0][0] + c[1][0]) + (c[0][1] + c[1][1]), us = (c[0][2] + c[1][2]) + (c[0][3] + c[1][3]);
          gs += __shfl_xor_sync(0xffffffffu, gs, 1);
          us += __shfl_xor_sync(0xffffffffu, us, 1);
          gs += __shfl_xor_sync(0xffffffffu, gs, 2);
          us += __shfl_xor_sync(0xffffffffu, us, 2);
          if (q == 0) {
            part[0][g][wid] = gs;
            part[1][g][wid] = us;
          }
        } else {
          // two row blocks: the gate rows in one, the up rows in the other (rows past the end read the last row)
          const int jr = min(8 * (mi & 1) + (lane & 7), nrows - 1);
          int s_g, s_u;
          uint32_t par_a;
          slot_of(pbase + (unsigned int)jr, a.ns_magic, ns, s_g, par_a);
          slot_of(pbase + (unsigned int)(nrows + jr), a.ns_magic, ns, s_u, par_a);
          const uint32_t koff = (uint32_t)((wid * KB * 16 + (mi >> 1) * 8) * 2);
          const uint32_t g_addr = ring + (uint32_t)s_g * pstride + koff, u_addr = ring + (uint32_t)s_u * pstride + koff;
          float cg[4] = {0.f, 0.f, 0.f, 0.f}, cu[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int kb = 0; kb < KB; ++kb) {
            uint32_t ag[4], au[4];
            ldmatrix_x4(ag, g_addr + (uint32_t)kb * 32u);
            ldmatrix_x4(au, u_addr + (uint32_t)kb * 32u);
            uint32_t b0 = *reinterpret_cast<const uint32_t*>(bp + kb * 32);
            uint32_t b1 = *reinterpret_cast<const uint32_t*>(bp + kb * 32 + 16);
            if (g >= 3) b0 = b1 = 0u;
            mma_bf16_16816(cg, ag, b0, b1);
            mma_bf16_16816(cu, au, b0, b1);
          }
          // accumulator rows g and g + 8 are rows g and g + 8 of the block's share
          float g0 = cg[0] + cg[1], g1 = cg[2] + cg[3], u0 = cu[0] + cu[1], u1 = cu[2] + cu[3];
#pragma unroll
          for (int o = 1; o <= 2; o <<= 1) {
            g0 += __shfl_xor_sync(0xffffffffu, g0, o);
            g1 += __shfl_xor_sync(0xffffffffu, g1, o);
            u0 += __shfl_xor_sync(0xffffffffu, u0, o);
            u1 += __shfl_xor_sync(0xffffffffu, u1, o);
          }
          if (q == 0) {
            part[0][g][wid] = g0;
            part[0][8 + g][wid] = g1;
            part[1][g][wid] = u0;
            part[1][8 + g][wid] = u1;
          }
        }
        RK(17);
        __syncwarp();  // every lane's ldmatrix has returned
        if (lane < 2 * nrows) {
          int s;
          uint32_t par;
          slot_of(pbase + (unsigned int)lane, a.ns_magic, ns, s, par);
          npp::mbar_arrive(&empty_bar[s]);
        }
      }
      RK(3);
      AK(1);
      AKV(7, nrows);
      consumer_sync();
      RK(4);
      // a warp per row: lanes 0-15 add the 16 warps' gate sums, lanes 16-31 their up sums
      for (int r = wid; r < nrows; r += kWarps) {
        float v = part[lane >> 4][r][lane & 15];
        float ss = 0.f;
        if (lane < kCS * wpo) ss = ssq_part[lane / wpo][lane % wpo][0];
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) {
          v += __shfl_xor_sync(0xffffffffu, v, o);
          ss += __shfl_xor_sync(0xffffffffu, ss, o);
        }
        const float us2 = __shfl_sync(0xffffffffu, v, 16);
        if (lane == 0) {
          // the MLP's input is x_l scaled to unit RMS; the dot products are linear in it
          const float inv_rms = rsqrtf(ss / (float)D + kRmsEps);
          const float gsn = v * inv_rms;
          act[r] = gsn / (1.f + __expf(-gsn)) * (us2 * inv_rms);
        }
      }
      consumer_sync();
      RK(5);

      // ---- phase 2: y[cols] = sum_i a_i * downT[s_i][cols], 8 columns per thread; the rows wait in tensor memory ----
      float acc[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] = 0.f;
      auto axpy = [&](float av, const uint4 w) {
        acc[0] = fmaf(av, bf16_lo(w.x), acc[0]);
        acc[1] = fmaf(av, bf16_hi(w.x), acc[1]);
        acc[2] = fmaf(av, bf16_lo(w.y), acc[2]);
        acc[3] = fmaf(av, bf16_hi(w.y), acc[3]);
        acc[4] = fmaf(av, bf16_lo(w.z), acc[4]);
        acc[5] = fmaf(av, bf16_hi(w.z), acc[5]);
        acc[6] = fmaf(av, bf16_lo(w.w), acc[6]);
        acc[7] = fmaf(av, bf16_hi(w.w), acc[7]);
      };
      {
        const int buf = li & 1;
        if (lane == 0) wait_or_flag(&tm_full[buf], (uint32_t)(li >> 1) & 1u, ok, a.status);
        __syncwarp();
        tc_fence_after();
        RK(18);
        // this thread's chunk (32 wid + lane) of row r: lane 32 (wid % 4) + lane, columns 16 r + 4 (wid / 4) .. + 3
        const uint32_t taddr = tmem_base + ((uint32_t)((wid & 3) * 32) << 16) + (uint32_t)(buf * (kTmemCols / 2) + (wid >> 2) * 4);
#pragma unroll
        for (int r0 = 0; r0 < kTmemRows; r0 += 8) {
          if (r0 < nrows) {  // warp-uniform
            uint4 w[8];
#pragma unroll
            for (int i = 0; i < 8; ++i)
              if (r0 + i < nrows) w[i] = tc_ld4(taddr + (uint32_t)((r0 + i) * 16));
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 8; ++i)
              if (has_chunk && r0 + i < nrows) axpy(act[r0 + i], w[i]);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) npp::mbar_arrive(&tm_empty[buf]);
      }
      RK(19);
      AK(2);

      RK(6);
      // ---- reduce among the cluster: every range to its owner ----
      // (a warp's 32 chunks are 1 KB of the vector: staged in shared memory, then one bulk copy into the owner's)
      if (has_chunk && !own) {
        const int from = owner - (owner > (int)rank ? 1 : 0);  // the owner's place among this block's peers
        float4* ys = reinterpret_cast<float4*>(y_stage + (size_t)from * seg) + 2 * lc;
        ys[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
        ys[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
        npp::fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
          const int at = (int)rank - ((int)rank > owner ? 1 : 0);  // this block's place among the owner's peers
          bulk_s2peer(map_to_rank(npp::smem_addr(rs_buf + (size_t)at * seg + (size_t)(lc & ~31) * 8), (uint32_t)owner),
                      y_stage + (size_t)from * seg + (size_t)(lc & ~31) * 8, 1024u, map_to_rank(npp::smem_addr(&rs_bar), (uint32_t)owner));
        }
      }
      float* zl = a.z4 + (size_t)((a.seq + (unsigned int)li) & 3u) * kZR * D + (size_t)rank * seg;  // copy 0 of this layer's accumulator, this block's range
      RK(7);
      if (own) {
        wait_cluster_or_flag(&rs_bar, (uint32_t)li & 1u, ok, a.status);
        RK(8);
        AK(3);
#pragma unroll
        for (int o = 0; o < kCS - 1; ++o) {
          const float4 p0 = *reinterpret_cast<const float4*>(rs_buf + (size_t)o * seg + (size_t)lc * 8);
          const float4 p1 = *reinterpret_cast<const float4*>(rs_buf + (size_t)o * seg + (size_t)lc * 8 + 4);
          acc[0] += p0.x, acc[1] += p0.y, acc[2] += p0.z, acc[3] += p0.w;
          acc[4] += p1.x, acc[5] += p1.y, acc[6] += p1.z, acc[7] += p1.w;
        }
        float* zmine = zl + (size_t)(cluster % kZR) * D;
        red_add_v4(zmine + (size_t)lc * 8, make_float4(acc[0], acc[1], acc[2], acc[3]));
        red_add_v4(zmine + (size_t)lc * 8 + 4, make_float4(acc[4], acc[5], acc[6], acc[7]));
        // the accumulator two layers ahead is cleared now (this range of every copy, a share per cluster): its last
        // readers have all arrived at the previous layer's counter, and nobody adds to it before this layer's has filled
        float* zc = a.z4 + (size_t)((a.seq + (unsigned int)li + 2u) & 3u) * kZR * D + (size_t)rank * seg;
        for (int f = cluster + NCL * lc; f < kZR * (seg / 4); f += NCL * seg_chunks) {
          const int copy = f / (seg / 4), at = f - copy * (seg / 4);
          reinterpret_cast<float4*>(zc + (size_t)copy * D)[at] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
      RK(9);
      consumer_sync();
      RK(10);
      // ---- the range's counter: one arrival per cluster ----
      if (tid == 0) {
        __threadfence();  // the block's reductions and stores above, before the arrival
        atomicAdd(a.cnt + rank, 1u);
        RK(11);
        const unsigned int target = a.cnt_base + (unsigned int)(li + 1) * (unsigned int)NCL;
        bool there = false;
        if (*ok) {
          for (uint32_t spin = 0; spin < npp::kSpinLimit && !there; ++spin) {
            unsigned int v;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(a.cnt + rank) : "memory");
            there = (int)(v - target) >= 0;
          }
          if (!there) {
            atomicOr(a.status, npp::kStatTimeout);
            s_ok = 0;
          }
        }
      }
      RK(12);
      AK(4);
      consumer_sync();
      RK(13);
      // ---- x_{l+1} of this block's range ----
      if (own) {
        float4 z0[kZR], z1[kZR];
#pragma unroll
        for (int r = 0; r < kZR; ++r) {  // all loads first
          z0[r] = __ldcg(reinterpret_cast<const float4*>(zl + (size_t)r * D + (size_t)lc * 8));
          z1[r] = __ldcg(reinterpret_cast<const float4*>(zl + (size_t)r * D + (size_t)lc * 8 + 4));
        }
#pragma unroll
        for (int r = 0; r < kZR; ++r) {
          xo[0] += z0[r].x, xo[1] += z0[r].y, xo[2] += z0[r].z, xo[3] += z0[r].w;
          xo[4] += z1[r].x, xo[5] += z1[r].y, xo[6] += z1[r].z, xo[7] += z1[r].w;
        }
        RK(14);
        if (li == nl - 1) {
          if (cluster == 0) {  // the hand-over to whatever runs next: x_{l_end}, and cleared accumulators
            float4* xout = reinterpret_cast<float4*>(a.x_out) + 2 * tid;
            xout[0] = make_float4(xo[0], xo[1], xo[2], xo[3]);
            xout[1] = make_float4(xo[4], xo[5], xo[6], xo[7]);
#pragma unroll
            for (int r = 0; r < kZRep; ++r) {
              float4* za = reinterpret_cast<float4*>(a.zclr_a + (size_t)r * D) + 2 * tid;
              float4* zb = reinterpret_cast<float4*>(a.zclr_b + (size_t)r * D) + 2 * tid;
              za[0] = za[1] = zb[0] = zb[1] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
          }
        } else {
          // ---- ... as three bf16 terms to every block of the cluster: a warp's 32 chunks are 512 bytes per term ----
          const Terms8 t8 = split8(xo);
#pragma unroll
          for (int k = 0; k < 3; ++k) *reinterpret_cast<uint4*>(ag_stage + (size_t)k * seg * 2 + (size_t)lc * 16) = t8.t[k];
          float ss = 0.f;
#pragma unroll
          for (int e = 0; e < 8; ++e) ss += xo[e] * xo[e];
          ss = warp_sum(ss);
          if (lane == 0) ag_ssq[ow][0] = ss;
          npp::fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
#pragma unroll
            for (uint32_t dst = 0; dst < (uint32_t)kCS; ++dst) {
              const uint32_t bar = map_to_rank(npp::smem_addr(&ag_bar), dst);
#pragma unroll
              for (int k = 0; k < 3; ++k)
                bulk_s2peer(map_to_rank(npp::smem_addr(xt + (size_t)k * xt_stride + ((size_t)rank * seg_chunks + (lc & ~31)) * 16), dst),
                            ag_stage + (size_t)k * seg * 2 + (size_t)(lc & ~31) * 16, 512u, bar);
              bulk_s2peer(map_to_rank(npp::smem_addr(&ssq_part[rank][ow][0]), dst), &ag_ssq[ow][0], 16u, bar);
            }
          }
        }
      }
      RK(15);
      AK(5);
    }
  }
  // tensor memory goes back once every warp of the block is done with it
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (wid == kWarps + 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
  // nobody leaves while a peer may still write to its shared memory or arrive on its barriers
  cluster_sync_all();
}

// ---------------------------------------------------------------------------------------
namespace {

struct Geometry {
  int ns, max_rows, run_layers, slot_cache_rows;
  size_t smem;
};

bool geometry(const Dims& d, int G, Geometry* g) {
  if (d.D % 1024 != 0 || d.D > 4096 || d.D / 8 > kThreads) return false;  // a thread per 8 columns, whole warps per range
  if ((d.D / 8 / kCS) % 32 != 0) return false;
  if (G < kCS) return false;
  const int kb = d.D / 16 / kWarps;
  if (kb != 4 && kb != 8 && kb != 12 && kb != 16) return false;
  // one sequence selects k rows per layer; a block takes a G-th of them
  const int max_rows = (std::min(d.k, d.C) + G - 1) / G;  // floor(n (b + 1) / G) - floor(n b / G) <= ceil(n / G)
  if (max_rows > kMaxRows || max_rows > kTmemRows) return false;
  const size_t pstride = (size_t)d.D * 2 + kPad;
  // staging of the down rows, x terms, the peers' partial sums (later this block's outgoing terms), its own outgoing sums
  const size_t fixed = (size_t)(kDS + 3) * pstride + 2 * (size_t)(kCS - 1) * (d.D / kCS) * 4 + (kCS >= 4 ? 0 : 3 * (size_t)(d.D / kCS) * 2) + 1024;
  const size_t budget = 222 * 1024;  // the kernel has about 4 KB of static shared memory besides
  const int run_layers = std::min(kMaxLayers, std::max(1, d.L));
  const size_t slot_bytes = (size_t)run_layers * max_rows * 4;
  if (fixed + slot_bytes + (size_t)(2 * max_rows) * pstride > budget) return false;  // a layer's gate and up rows at once
  g->ns = (int)std::min<size_t>(kMaxSlots, (budget - fixed - slot_bytes) / pstride);
  g->max_rows = max_rows;
  g->run_layers = run_layers;
  g->slot_cache_rows = run_layers * max_rows;
  g->smem = (size_t)g->ns * pstride + fixed - 1024 + slot_bytes;
  return true;
}

template <int KB>
cudaError_t launch_kb(const KArgs& ka, int G, size_t smem, cudaStream_t s, int* max_clusters) {
  cudaError_t e = cudaFuncSetAttribute(k_mlp_rows<KB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(G > 0 ? G : kCS);
  cfg.blockDim = dim3(kBlock);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kCS;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeCooperative;  // every block resident: they wait for one another
  attr[1].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  if (max_clusters) return cudaOccupancyMaxActiveClusters(max_clusters, k_mlp_rows<KB>, &cfg);
  return cudaLaunchKernelEx(&cfg, k_mlp_rows<KB>, ka);
}

cudaError_t dispatch(const Dims& d, const KArgs& ka, int G, size_t smem, cudaStream_t s, int* max_clusters) {
  switch (d.D / 16 / kWarps) {
    case 4: return launch_kb<4>(ka, G, smem, s, max_clusters);
    case 8: return launch_kb<8>(ka, G, smem, s, max_clusters);
    case 12: return launch_kb<12>(ka, G, smem, s, max_clusters);
    case 16: return launch_kb<16>(ka, G, smem, s, max_clusters);
  }
  return cudaErrorInvalidValue;
}

}  // namespace

size_t z_floats(const Dims& d) { return 4 * (size_t)kZR * d.D; }

// How many blocks a launch has: the clusters that can be resident at once, found once per context.
bool prepare(const Dims& d, int sm_count, State* st) {
  st->grid = 0;
  Geometry g;
  // the shared memory does not depend on the grid by much: size it for the smallest grid that could run
  if (!geometry(d, std::max(kCS, sm_count - sm_count % kCS), &g)) return false;
  int ncl = 0;
  KArgs none = {};
  if (dispatch(d, none, 0, g.smem, nullptr, &ncl) != cudaSuccess || ncl < 1) {
    (void)cudaGetLastError();
    return false;
  }
  const int G = std::min(ncl, sm_count / kCS) * kCS;
  if (!geometry(d, G, &g)) return false;
  st->grid = G;
  return true;
}

bool supported(const Dims& d, const State& st) { return st.grid >= kCS; }

int run_layers(const Dims& d, const State& st) {
  Geometry g;
  return geometry(d, st.grid, &g) ? g.run_layers : 0;
}

cudaError_t launch(const Dims& d, const ChainArgs& a, State* st, cudaStream_t s) {
  Geometry g;
  if (st->grid < kCS || !geometry(d, st->grid, &g) || a.dense_rows > 0) return cudaErrorInvalidValue;
  const int NCL = st->grid / kCS;
  for (int l0 = a.l_begin; l0 < a.l_end; l0 += g.run_layers) {
    const int l1 = std::min(a.l_end, l0 + g.run_layers);
    KArgs ka;
    ka.gate = static_cast<const unsigned char*>(a.gate);
    ka.up = static_cast<const unsigned char*>(a.up);
    ka.downT = static_cast<const unsigned char*>(a.downT);
    ka.slots = a.active_slots;
    ka.counters = a.counters;
    // the hand-over between kernels of a chain: x_l = xbuf[(l + 1) & 1] + the copies of zbuf[(l - 1) % 3]
    ka.x_bf16 = l0 == 0 ? static_cast<const uint16_t*>(a.x_bf16) : nullptr;
    ka.x_in = a.xbuf[(l0 + 1) & 1];
    ka.z_in = l0 > 0 ? a.zbuf[(l0 - 1) % 3] : nullptr;
    // ... and at the end x_{l1} = xbuf[(l1 - 1) & 1] + the copies of zbuf[(l1 - 1) % 3], zbuf[l1 % 3] cleared
    ka.x_out = a.xbuf[(l1 - 1) & 1];
    ka.zclr_a = a.zbuf[(l1 - 1) % 3];
    ka.zclr_b = a.zbuf[l1 % 3];
    ka.z4 = st->z4;
    ka.cnt = st->cnt;
    ka.status = a.status;
    ka.cnt_base = st->cnt_base;
    ka.seq = st->seq;
    ka.ns_magic = (unsigned int)((0x100000000ull + (unsigned long long)g.ns - 1) / (unsigned long long)g.ns);
    ka.l_begin = l0;
    ka.l_end = l1;
    ka.D = d.D;
    ka.C = d.C;
    ka.check = a.check;
    ka.ns = g.ns;
    ka.max_rows = g.max_rows;
    ka.slot_cache_rows = g.slot_cache_rows;
    cudaError_t e = dispatch(d, ka, st->grid, g.smem, s, nullptr);
    if (e != cudaSuccess) return e;
    st->cnt_base += (unsigned int)(l1 - l0) * (unsigned int)NCL;
    st->seq += (unsigned int)(l1 - l0);
  }
  return cudaSuccess;
}

}  // namespace chain_rows
}  // namespace npi
