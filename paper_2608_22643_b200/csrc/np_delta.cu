// Stage 3a: delta and residency update (Section 3.4).
//
//   incoming  D_in  = P \ R            (Eq. 2)
//   outgoing  D_out = R \ P            (Eq. 3; all of it under NP_EVICT_EXACT,
//                                       the least recently predicted part of it
//                                       under NP_EVICT_LRU)
//   slot map  S[n] = slot or -1; outgoing rows clear their entry, incoming rows
//             take the freed slots, nothing is compacted or moved.
//
// One block per layer.  Bitmap words are diffed, set bits are turned into
// ascending lists by popcount + block-wide exclusive scan (stream compaction),
// and the i-th incoming row is paired with the i-th free slot.
#include "np_device.cuh"
#include "np_internal.h"
#include "np_pipe.cuh"

namespace npi {
using namespace npd;

constexpr int kDeltaThreads = 1024;

struct DeltaParams {
  Tables t;
  const uint32_t* pred;  // [L][W]
  int32_t* host_lists;   // device alias of the pinned host mirror (may be NULL)
  int L, M, C, W;
  int policy, step, check;
};

// Ascending list of the indices i in [0, n) with flag(i) true; returns the count
// to every thread.  `red` is shared scratch (>= 40 ints).
template <typename Flag, typename Emit>
__device__ __forceinline__ int compact_indices(int n, int* red, Flag flag, Emit emit) {
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nw = blockDim.x >> 5;
  int base = 0;
  for (int i0 = 0; i0 < n; i0 += blockDim.x) {
    const int i = i0 + tid;
    const bool f = i < n && flag(i);
    const uint32_t bal = __ballot_sync(0xffffffffu, f);
    __syncthreads();
    if (lane == 0) red[wid] = __popc(bal);
    __syncthreads();
    if (wid == 0) {
      int c = lane < nw ? red[lane] : 0;
      int inc = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
      }
      red[lane] = inc - c;
      if (lane == 31) red[33] = inc;
    }
    __syncthreads();
    if (f) emit(base + red[wid] + __popc(bal & ((1u << lane) - 1u)), i);
    base += red[33];
  }
  __syncthreads();
  return base;
}

#ifdef NP_TRACE  // development builds only: clock stamps of one block
__device__ long long np_dl_clk[32];
extern "C" int np_debug_dl(void* out) { return (int)cudaMemcpyFromSymbol(out, np_dl_clk, sizeof(np_dl_clk)); }
#define DK(ev) do { if (blockIdx.x == 5 && threadIdx.x == 0) np_dl_clk[ev] = clock64(); } while (0)
#else
#define DK(ev) do { } while (0)
#endif

constexpr int kListCap = 2048;  // list entries held in shared memory; longer lists continue in their global arrays

// List offsets of the set bits of a bitmap by the whole block: off[w] = number of set bits in
// bits[0..w); returns the total to every thread.  wsum: 33 ints of shared scratch.  The caller
// puts a block-wide barrier before off[] is read by other threads (and before wsum is reused).
__device__ __forceinline__ int block_bit_offsets(const uint32_t* bits, int* off, int n, int* wsum, int tid, int lane, int wid) {
  int base = 0;
  for (int w0 = 0; w0 < n; w0 += kDeltaThreads) {  // block-uniform; one round unless the layer has more than 32768 neurons
    if (w0) __syncthreads();
    const int w = w0 + tid;
    const int c = w < n ? __popc(bits[w]) : 0;
    const int inc = block_inclusive_scan_1024(c, wsum, lane, wid);
    if (w < n) off[w] = base + inc - c;
    base += wsum[32];
  }
  return base;
}

// The layer's tables are small and the step is a chain of block-wide phases on one SM: what
// it costs is the instructions of those phases and the memory round trips between them.  So:
//   * list positions are a word's offset (block scan of the words' popcounts; the offsets of
//     the incoming rows, of the candidates and of the predicted rows come out of ONE scan,
//     the first two as 16-bit fields of one integer) plus the rank of the bit inside its word;
//   * the lists are sparse (a tenth of the bits are predicted, a sixtieth arrive or leave), so
//     a thread per word first writes them into shared memory, and then a thread per ENTRY does
//     the work: global loads and stores are one batch, and the lists go out in order
//     (coalesced, also into the host's mirror).  The pass over the predicted rows stamps them,
//     writes the active list (when every incoming row finds a slot, the active set IS the
//     predicted set), copies the slots of the rows that stay and lists the incoming rows;
//   * the free slots are a bitmap (rows that leave set their bit) and a list in shared memory.
// The rare step in which incoming rows find no slot rewrites the active list afterwards.
//
// The resident bitmap and the owner table are read BEFORE the wait on the previous kernel:
// they are written only by kernels of this file and by copies, none of which lets a later
// kernel start early, so they are final once this kernel's blocks run; the predicted bitmap
// may be the previous kernel's and is read after the wait.
__global__ void __launch_bounds__(kDeltaThreads, 1) k_delta(DeltaParams p) {
  extern __shared__ __align__(16) int dsm[];
  const int W = p.W, M = p.M, C = p.C;
  const int CW = (C + 31) >> 5;                        // words of a bitmap over the slots
  uint32_t* w_p = reinterpret_cast<uint32_t*>(dsm);    // [W] predicted
  uint32_t* w_r = w_p + W;                             // [W] resident before the step
  uint32_t* w_in = w_r + W;                            // [W] incoming bits
  uint32_t* w_ev = w_in + W;                           // [W] victim bits
  uint32_t* w_act = w_ev + W;                          // [W] active bits after the update (only when rows found no slot)
  uint32_t* w_free = w_act + W;                        // [CW] free-slot bits
  int* off_in = reinterpret_cast<int*>(w_free + CW);   // [W] list offsets of w_in
  int* off_ev = off_in + W;                            // [W] of w_ev
  int* off_act = off_ev + W;                           // [W] of the active bits
  int* off_free = off_act + W;                         // [CW] of w_free
  int* fl = off_free + CW;                             // [kListCap] the first free slots, ascending
  int* in_list = fl + kListCap;                        // [kListCap] the first incoming rows, ascending
  int* in_apos = in_list + kListCap;                   // [kListCap] their positions in the active list
  int* ev_list = in_apos + kListCap;                   // [kListCap] the first rows that leave, ascending
  int* act_list = ev_list + kListCap;                  // [kListCap] the first predicted rows, ascending
  int* red = act_list + kListCap;                      // [48]
  int* hist = red + 48;                                // [256]
  __shared__ uint32_t s_prefix;
  __shared__ int s_remaining;
  __shared__ int wsum[2][33];

  const int layer = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int T = kDeltaThreads, NW = T >> 5;
  const uint32_t lt = (1u << lane) - 1u;  // the bits below this lane's
  const uint32_t* P = p.pred + (size_t)layer * W;
  uint32_t* R = p.t.resident + (size_t)layer * W;
  int32_t* S = p.t.slot_map + (size_t)layer * M;
  int32_t* owner = p.t.owner + (size_t)layer * C;
  int32_t* stamp = p.t.stamp + (size_t)layer * M;
  int32_t* delta_ids = p.t.delta_ids + (size_t)layer * C;
  int32_t* delta_slots = p.t.delta_slots + (size_t)layer * C;
  int32_t* evict_ids = p.t.evict_ids + (size_t)layer * C;
  int32_t* active_ids = p.t.active_ids + (size_t)layer * C;
  int32_t* active_slots = p.t.active_slots + (size_t)layer * C;
  int32_t* overflow_ids = p.t.overflow_ids + (size_t)layer * M;
  int32_t* free_slots = p.t.free_slots + (size_t)layer * C;
  int32_t* counters = p.t.counters + (size_t)layer * NP_N_COUNTERS;
  // host mirror: [header][layer: counters, delta_ids[C], delta_slots[C]]
  int32_t* h_cnt = nullptr;
  int32_t* h_ids = nullptr;
  int32_t* h_slots = nullptr;
  if (p.host_lists) {
    h_cnt = p.host_lists + kHostHeaderInts + (size_t)layer * (NP_N_COUNTERS + 2 * (size_t)C);
    h_ids = h_cnt + NP_N_COUNTERS;
    h_slots = h_ids + C;
  }
  DK(0);
  for (int w = tid; w < W; w += T) w_r[w] = R[w];
  for (int cw = wid; cw < CW; cw += NW) {
    const int s = cw * 32 + lane;
    const uint32_t fb = __ballot_sync(0xffffffffu, s < C && owner[s] < 0);
    if (lane == 0) w_free[cw] = fb;
  }
  // No early trigger for the kernel behind this one: whatever follows may read the tables.
  npp::pdl_wait_prior();  // the bitmap may be the previous kernel's
  DK(1);

  // ---- 1. diff the bitmaps ------------------------------------------------------------
  for (int w = tid; w < W; w += T) {
    const uint32_t pw = P[w], rw = w_r[w];  // w_r[w]: this thread's own store above
    w_p[w] = pw;
    w_in[w] = pw & ~rw;
    w_ev[w] = rw & ~pw;  // NP_EVICT_EXACT: every candidate leaves; LRU narrows this below
  }
  __syncthreads();
  DK(2);
  // offsets of the incoming rows and of the candidates (two 16-bit fields: a layer has at
  // most 40960 neurons) and of the predicted rows, in one scan
  int n_in, n_cand, n_pred;
  {
    uint32_t base_a = 0u;  // unsigned: the upper field may reach 40960 << 16
    int base_b = 0;
    for (int w0 = 0; w0 < W; w0 += T) {  // block-uniform; one round unless the layer has more than 32768 neurons
      if (w0) __syncthreads();
      const int w = w0 + tid;
      const uint32_t ca = w < W ? ((uint32_t)__popc(w_in[w]) | ((uint32_t)__popc(w_ev[w]) << 16)) : 0u;
      const int cb = w < W ? __popc(w_p[w]) : 0;
      uint32_t ia = ca;
      int ib = cb;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t ta = __shfl_up_sync(0xffffffffu, ia, o);
        const int tb = __shfl_up_sync(0xffffffffu, ib, o);
        if (lane >= o) {
          ia += ta;
          ib += tb;
        }
      }
      if (lane == 31) {
        wsum[0][wid] = (int)ia;
        wsum[1][wid] = ib;
      }
      __syncthreads();
      if (wid < 2) {
        const uint32_t ws = (uint32_t)wsum[wid][lane];
        uint32_t winc = ws;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t t = __shfl_up_sync(0xffffffffu, winc, o);
          if (lane >= o) winc += t;
        }
        wsum[wid][lane] = (int)(winc - ws);
        if (lane == 31) wsum[wid][32] = (int)winc;
      }
      __syncthreads();
      if (w < W) {
        const uint32_t ea = base_a + (uint32_t)wsum[0][wid] + ia - ca;
        off_in[w] = (int)(ea & 0xffffu);
        off_ev[w] = (int)(ea >> 16);
        off_act[w] = base_b + wsum[1][wid] + ib - cb;
      }
      base_a += (uint32_t)wsum[0][32];
      base_b += wsum[1][32];
    }
    n_in = (int)(base_a & 0xffffu);
    n_cand = (int)(base_a >> 16);
    n_pred = base_b;
  }
  const int n_kept = n_pred - n_in;        // P = kept + incoming
  const int n_res_prev = n_kept + n_cand;  // R = kept + candidates
  __syncthreads();  // the offsets are read by other threads
  DK(3);

  // ---- 2. victims under LRU: the `need` candidates with the smallest (stamp, index) -------
  int n_evict = n_cand;
  if (p.policy == NP_EVICT_LRU) {
    const int free_now = C - n_res_prev;
    const int need = max(0, n_in - free_now);
    bool narrowed = false;
    if (need == 0) {
      for (int w = tid; w < W; w += T) w_ev[w] = 0u;
      narrowed = true;
    } else if (need < n_cand) {
      int32_t* cand_ids = p.t.cand_ids + (size_t)layer * C;
      uint32_t* cand_keys = p.t.cand_keys + (size_t)layer * C;
      // candidates as an ascending list with keys stamp + 1 (stamps start at -1); a candidate is
      // not predicted, so its stamp is not one of those written above
      for (int w = wid; w < W; w += NW) {
        const uint32_t m = w_ev[w];
        if ((m >> lane) & 1u) {
          const int pos = off_ev[w] + __popc(m & lt), n = w * 32 + lane;
          cand_ids[pos] = n;
          cand_keys[pos] = (uint32_t)(stamp[n] + 1);
        }
      }
      __syncthreads();
      for (int w = tid; w < W; w += T) w_ev[w] = 0u;
      if (tid == 0) {
        s_prefix = 0u;
        s_remaining = need;
      }
      __syncthreads();
      // radix select, least significant victims first: need-th smallest key
      uint32_t mask = 0u;
      for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        const uint32_t prefix = s_prefix;
        for (int i = tid; i < n_cand; i += T) {
          const uint32_t key = cand_keys[i];
          if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1);
        }
        __syncthreads();
        if (tid == 0) {
          int run = 0, bin = 0;
          const int remaining = s_remaining;
          for (; bin < 256; ++bin) {
            if (run + hist[bin] >= remaining) break;
            run += hist[bin];
          }
          s_prefix = prefix | ((uint32_t)bin << shift);
          s_remaining = remaining - run;
        }
        mask |= 0xffu << shift;
        __syncthreads();
      }
      const uint32_t thr = s_prefix;  // key of the need-th smallest candidate
      const int admit = s_remaining;  // candidates equal to thr that go, lowest index first
      // rank of each threshold-equal candidate among its equals, in list (= index) order
      int base = 0;
      for (int i0 = 0; i0 < n_cand; i0 += T) {
        const int i = i0 + tid;
        const uint32_t key = i < n_cand ? cand_keys[i] : 0xffffffffu;
        const bool eq = i < n_cand && key == thr;
        const uint32_t bal = __ballot_sync(0xffffffffu, eq);
        __syncthreads();
        if (lane == 0) red[wid] = __popc(bal);
        __syncthreads();
        if (wid == 0) {
          int c = lane < NW ? red[lane] : 0;
          int inc = c;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += t;
          }
          red[lane] = inc - c;
          if (lane == 31) red[33] = inc;
        }
        __syncthreads();
        if (i < n_cand) {
          const int rank = base + red[wid] + __popc(bal & lt);
          if (key < thr || (eq && rank < admit)) {
            const int n = cand_ids[i];
            atomicOr(&w_ev[n >> 5], 1u << (n & 31));
          }
        }
        base += red[33];
      }
      narrowed = true;
    }
    // need >= n_cand: every candidate leaves (w_ev and its offsets already hold them)
    if (narrowed) {  // block-uniform: the victims changed, so do their offsets
      __syncthreads();
      n_evict = block_bit_offsets(w_ev, off_ev, W, wsum[0], tid, lane, wid);
      __syncthreads();
    }
  }
  DK(4);

  // ---- 3. one pass over the predicted rows; the rows that leave as a list -------------------
  // 3a. a thread per word: the first kListCap predicted rows and leaving rows as lists
  for (int w = tid; w < W; w += T) {
    uint32_t m = w_p[w];
    int pos = off_act[w];
    while (m && pos < kListCap) {
      act_list[pos++] = w * 32 + __ffs(m) - 1;
      m &= m - 1;
    }
    m = w_ev[w];
    pos = off_ev[w];
    while (m && pos < kListCap) {
      ev_list[pos++] = w * 32 + __ffs(m) - 1;  // rows beyond the shared list are handled bit by bit below
      m &= m - 1;
    }
  }
  __syncthreads();
  // 3b. a thread per predicted row
  auto predicted = [&](int n, int pos) {
    const int w = n >> 5, bit = n & 31;
    stamp[n] = p.step;
    if (pos < C) active_ids[pos] = n;
    const uint32_t in = w_in[w];
    if ((in >> bit) & 1u) {  // arrives: its slot is known below
      const int ipos = off_in[w] + __popc(in & ((1u << bit) - 1u));
      if (ipos < kListCap) {  // rows beyond the shared list are handled bit by bit below
        in_list[ipos] = n;
        in_apos[ipos] = pos;
      }
    } else if (pos < C) {  // stays
      active_slots[pos] = S[n];
    }
  };
  for (int i = tid; i < min(n_pred, kListCap); i += T) predicted(act_list[i], i);
  if (n_pred > kListCap) {  // block-uniform: the rest of a long list, a bit per lane
    for (int w = wid; w < W; w += NW) {
      const uint32_t pw = w_p[w];
      if ((pw >> lane) & 1u) {
        const int pos = off_act[w] + __popc(pw & lt);
        if (pos >= kListCap) predicted(w * 32 + lane, pos);
      }
    }
  }
  __syncthreads();
  DK(5);

  // ---- 4. outgoing rows release their slots; evict list ------------------------------
  auto release = [&](int n, int pos) {
    const int s = S[n];
    if (p.check && (s < 0 || s >= C)) {
      atomicOr(p.t.status, kStatBadSlot);
    } else {
      owner[s] = -1;
      atomicOr(&w_free[s >> 5], 1u << (s & 31));
    }
    S[n] = -1;
    if (pos < C) evict_ids[pos] = n;
  };
  for (int i = tid; i < min(n_evict, kListCap); i += T) release(ev_list[i], i);
  if (n_evict > kListCap) {  // block-uniform: the rest of a long list, a bit per lane
    for (int w = wid; w < W; w += NW) {
      const uint32_t m = w_ev[w];
      if ((m >> lane) & 1u) {
        const int pos = off_ev[w] + __popc(m & lt);
        if (pos >= kListCap) release(w * 32 + lane, pos);
      }
    }
  }
  __syncthreads();  // the free bitmap is complete
  DK(6);

  // ---- 5. free slots, ascending: as many as there are rows to place --------------------
  const int n_avail = block_bit_offsets(w_free, off_free, CW, wsum[0], tid, lane, wid);
  const int n_delta = min(n_in, n_avail);
  __syncthreads();
  DK(7);
  for (int cw = wid; cw < CW; cw += NW) {
    const uint32_t fb = w_free[cw];
    if ((fb >> lane) & 1u) {
      const int pos = off_free[cw] + __popc(fb & lt);
      if (pos < n_delta) {
        if (pos < kListCap) fl[pos] = cw * 32 + lane;
        else free_slots[pos] = cw * 32 + lane;
      }
    }
  }
  __syncthreads();  // the list is read below by other threads
  DK(8);

  // ---- 6. i-th incoming row takes the i-th free slot ---------------------------------
  const bool overflow = n_in > n_avail;  // block-uniform
  auto place = [&](int n, int i, int s) {
    S[n] = s;
    owner[s] = n;
    delta_ids[i] = n;
    delta_slots[i] = s;
    if (h_ids) {
      h_ids[i] = n;
      h_slots[i] = s;
    }
  };
  for (int i = tid; i < min(n_in, kListCap); i += T) {
    const int n = in_list[i];
    if (i < n_avail) {
      const int s = fl[i];
      place(n, i, s);
      const int apos = in_apos[i];
      if (!overflow && apos < C) active_slots[apos] = s;
    } else {
      overflow_ids[i - n_avail] = n;
    }
  }
  if (n_in > kListCap) {  // block-uniform: the rest of a long list, a bit per lane
    for (int w = wid; w < W; w += NW) {
      const uint32_t m = w_in[w];
      if ((m >> lane) & 1u) {
        const int i = off_in[w] + __popc(m & lt), n = w * 32 + lane;
        if (i >= kListCap) {
          if (i < n_avail) place(n, i, free_slots[i]);
          else overflow_ids[i - n_avail] = n;
        }
      }
    }
  }
  for (int w = tid; w < W; w += T) {
    const uint32_t m = w_in[w];
    const uint32_t placed = overflow ? lowest_bits(m, n_avail - off_in[w]) : m;
    const uint32_t rnew = (w_r[w] & ~w_ev[w]) | placed;
    R[w] = rnew;
    if (overflow) w_act[w] = w_p[w] & rnew;
  }
  // every incoming row placed: the active rows are the predicted rows, written above
  int n_active = n_pred;
  if (overflow || n_in > kListCap) {
    // rows without a slot are not active (or the incoming list left shared memory): the
    // active list is written again, from the tables as they now are
    __syncthreads();
    const uint32_t* act = overflow ? w_act : w_p;
    if (overflow) {
      n_active = block_bit_offsets(w_act, off_act, W, wsum[0], tid, lane, wid);
      __syncthreads();
    }
    for (int w = wid; w < W; w += NW) {
      {
        const uint32_t m = act[w];
        if ((m >> lane) & 1u) {
          const int pos = off_act[w] + __popc(m & lt);
          if (pos < C) {
            active_ids[pos] = w * 32 + lane;
            active_slots[pos] = S[w * 32 + lane];
          }
        }
      }
    }
  }
  DK(9);

  if (tid == 0) {
    const int n_resident = n_res_prev - n_evict + n_delta;
    int v[NP_N_COUNTERS];
    v[NP_CNT_PRED] = n_pred;
    v[NP_CNT_KEPT] = n_kept;
    v[NP_CNT_DELTA] = n_delta;
    v[NP_CNT_EVICT] = n_evict;
    v[NP_CNT_OVERFLOW] = n_in - n_delta;
    v[NP_CNT_ACTIVE] = n_active;
    v[NP_CNT_RESIDENT] = n_resident;
    v[NP_CNT_STEP] = p.step;
    if (p.check && (n_active > C || n_resident > C || n_evict > C)) atomicOr(p.t.status, kStatBadCount);
    for (int i = 0; i < NP_N_COUNTERS; ++i) counters[i] = v[i];
    // the host reads its mirror only after an event recorded behind this kernel: no fence needed
    if (h_cnt)
      for (int i = 0; i < NP_N_COUNTERS; ++i) h_cnt[i] = v[i];
  }
  DK(10);
}

// Speculative residency behind a step (the deeper prefetch of the paper's future work, Section 6):
// per layer, the candidates that are not resident, lowest index first, take the free slots in
// ascending order, as many as the budget and the free slots allow.  Nothing leaves, no stamp changes.
__global__ void __launch_bounds__(kDeltaThreads) k_speculate(Tables t, const uint32_t* __restrict__ cand, int32_t* host_lists,
                                                             int M, int C, int W, int budget, int first_layer) {
  extern __shared__ __align__(16) int ssm[];
  uint32_t* w_sp = reinterpret_cast<uint32_t*>(ssm);  // [W] candidate and not resident
  int* scan = reinterpret_cast<int*>(w_sp + W);       // [W]
  int* red = scan + W;                                // [48]
  const int layer = first_layer + blockIdx.x, tid = threadIdx.x;
  uint32_t* R = t.resident + (size_t)layer * W;
  int32_t* S = t.slot_map + (size_t)layer * M;
  int32_t* owner = t.owner + (size_t)layer * C;
  int32_t* free_slots = t.free_slots + (size_t)layer * C;
  int32_t* ids = t.spec_ids + (size_t)layer * C;
  int32_t* slots = t.spec_slots + (size_t)layer * C;
  int32_t* cnt = t.spec_counters + (size_t)layer * NP_N_COUNTERS;
  int32_t* h_cnt = nullptr;
  int32_t* h_ids = nullptr;
  int32_t* h_slots = nullptr;
  if (host_lists) {  // the second list area of the host mirror, laid out like the first
    h_cnt = host_lists + kHostHeaderInts + (size_t)layer * (NP_N_COUNTERS + 2 * (size_t)C);
    h_ids = h_cnt + NP_N_COUNTERS;
    h_slots = h_ids + C;
  }
  const uint32_t* cw = cand + (size_t)layer * W;
  for (int w = tid; w < W; w += blockDim.x) {
    const uint32_t m = cw[w] & ~R[w];
    w_sp[w] = m;
    scan[w] = __popc(m);
  }
  const int n_want = block_exclusive_scan(scan, W, red);
  const int n_avail = compact_indices(
      C, red, [&](int s) { return owner[s] < 0; }, [&](int pos, int s) { free_slots[pos] = s; });
  const int n = max(0, min(budget, min(n_want, n_avail)));
  for (int w = tid; w < W; w += blockDim.x) {
    uint32_t m = w_sp[w];
    int pos = scan[w];
    uint32_t placed = 0u;
    while (m && pos < n) {
      const int bit = __ffs(m) - 1;
      const int nid = w * 32 + bit;
      m &= m - 1;
      const int s = free_slots[pos];
      S[nid] = s;
      owner[s] = nid;
      ids[pos] = nid;
      slots[pos] = s;
      if (h_ids) {
        h_ids[pos] = nid;
        h_slots[pos] = s;
      }
      placed |= 1u << bit;
      ++pos;
    }
    if (placed) R[w] |= placed;
  }
  __syncthreads();
  if (tid == 0) {
    for (int i = 0; i < NP_N_COUNTERS; ++i) cnt[i] = 0;
    cnt[NP_CNT_DELTA] = n;
    t.counters[(size_t)layer * NP_N_COUNTERS + NP_CNT_RESIDENT] += n;
    if (h_cnt) {
      __threadfence_system();  // the list entries of the other threads precede the count the host reads
      for (int i = 0; i < NP_N_COUNTERS; ++i) h_cnt[i] = i == NP_CNT_DELTA ? n : 0;
    }
  }
}

cudaError_t launch_speculate(const Dims& d, const Tables& t, const uint32_t* cand, int budget, int32_t* host_lists_dev,
                             cudaStream_t s) {
  if (d.L <= d.dense) return cudaSuccess;
  const size_t sm = (size_t)d.W * 8 + 48 * 4;
  k_speculate<<<d.L - d.dense, kDeltaThreads, sm, s>>>(t, cand, host_lists_dev, d.M, d.C, d.W, budget, d.dense);
  return cudaGetLastError();
}

__global__ void k_tables_reset(Tables t, int L, int M, int C, int W) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t nLM = (size_t)L * M, nLC = (size_t)L * C, nLW = (size_t)L * W;
  if (i < nLM) {
    t.slot_map[i] = -1;
    t.stamp[i] = -1;
  }
  if (i < nLC) t.owner[i] = -1;
  if (i < nLW) {
    t.resident[i] = 0u;
    t.pred[i] = 0u;
  }
  if (i < (size_t)L * NP_N_COUNTERS) {
    t.counters[i] = 0;
    t.spec_counters[i] = 0;
  }
  if (i < 4) t.status[i] = 0;
}

cudaError_t launch_tables_reset(const Dims& d, const Tables& t, cudaStream_t s) {
  const size_t n = (size_t)d.L * d.M;
  k_tables_reset<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(t, d.L, d.M, d.C, d.W);
  return cudaGetLastError();
}

cudaError_t launch_delta(const Dims& d, const Tables& t, const uint32_t* pred, int policy, int step,
                         int32_t* host_lists_dev, int check, cudaStream_t s) {
  DeltaParams p;
  p.t = t;
  p.pred = pred;
  p.host_lists = host_lists_dev;
  p.L = d.L;
  p.M = d.M;
  p.C = d.C;
  p.W = d.W;
  p.policy = policy;
  p.step = step;
  p.check = check;
  const int CW = (d.C + 31) / 32;
  const size_t sm = ((size_t)d.W * 8 + (size_t)CW * 2 + 5 * kListCap + 48 + 256) * 4;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(d.L);
  cfg.blockDim = dim3(kDeltaThreads);
  cfg.dynamicSmemBytes = sm;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // its blocks are resident when the selection ends
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (sm > 48 * 1024) {
    static size_t allowed[64] = {};  // per device: the attribute sticks to the function, set it when a launch needs more than before
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || sm > allowed[dev]) {
      e = cudaFuncSetAttribute(k_delta, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
      if (e != cudaSuccess) return e;
      if (dev >= 0 && dev < 64) allowed[dev] = sm;
    }
  }
  return cudaLaunchKernelEx(&cfg, k_delta, p);
}

}  // namespace npi
