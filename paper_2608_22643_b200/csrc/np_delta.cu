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

__global__ void __launch_bounds__(kDeltaThreads) k_delta(DeltaParams p) {
  extern __shared__ __align__(16) int dsm[];
  const int W = p.W, M = p.M, C = p.C;
  uint32_t* w_in = reinterpret_cast<uint32_t*>(dsm);  // [W] incoming bits
  uint32_t* w_ev = w_in + W;                          // [W] victim bits
  uint32_t* w_act = w_ev + W;                         // [W] active bits after the update
  int* scan = reinterpret_cast<int*>(w_act + W);      // [W]
  int* red = scan + W;                                // [48]
  int* hist = red + 48;                               // [256]
  __shared__ uint32_t s_prefix;
  __shared__ int s_remaining;

  const int layer = blockIdx.x, tid = threadIdx.x;
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

  // ---- 1. diff the bitmaps, stamp predicted rows --------------------------------
  int c_pred = 0, c_kept = 0, c_res = 0, c_in = 0, c_cand = 0;
  for (int w = tid; w < W; w += blockDim.x) {
    const uint32_t pw = P[w], rw = R[w];
    const uint32_t din = pw & ~rw, cand = rw & ~pw;
    w_in[w] = din;
    w_ev[w] = cand;  // NP_EVICT_EXACT: every candidate leaves; LRU narrows this below
    c_pred += __popc(pw);
    c_kept += __popc(pw & rw);
    c_res += __popc(rw);
    c_in += __popc(din);
    c_cand += __popc(cand);
  }
  // stamps: one warp per word so that the 32 stores of a word coalesce
  for (int w = tid >> 5; w < W; w += blockDim.x >> 5) {
    if ((P[w] >> (tid & 31)) & 1u) stamp[w * 32 + (tid & 31)] = p.step;
  }
  const int n_pred = block_sum_int(c_pred, red);
  const int n_kept = block_sum_int(c_kept, red);
  const int n_res_prev = block_sum_int(c_res, red);
  const int n_in = block_sum_int(c_in, red);
  const int n_cand = block_sum_int(c_cand, red);

  // ---- 2. victims under LRU: the `need` candidates with the smallest (stamp, index) -------
  if (p.policy == NP_EVICT_LRU) {
    const int free_now = C - n_res_prev;
    const int need = max(0, n_in - free_now);
    if (need == 0) {
      for (int w = tid; w < W; w += blockDim.x) w_ev[w] = 0u;
      __syncthreads();
    } else if (need < n_cand) {
      int32_t* cand_ids = p.t.cand_ids + (size_t)layer * C;
      uint32_t* cand_keys = p.t.cand_keys + (size_t)layer * C;
      // candidates as an ascending list with keys stamp + 1 (stamps start at -1)
      for (int w = tid; w < W; w += blockDim.x) scan[w] = __popc(w_ev[w]);
      block_exclusive_scan(scan, W, red);
      for (int w = tid; w < W; w += blockDim.x) {
        uint32_t m = w_ev[w];
        int pos = scan[w];
        while (m) {
          const int n = w * 32 + __ffs(m) - 1;
          m &= m - 1;
          cand_ids[pos] = n;
          cand_keys[pos] = (uint32_t)(stamp[n] + 1);
          ++pos;
        }
      }
      for (int w = tid; w < W; w += blockDim.x) w_ev[w] = 0u;
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
        for (int i = tid; i < n_cand; i += blockDim.x) {
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
      const int lane = tid & 31, wid = tid >> 5, nw = blockDim.x >> 5;
      for (int i0 = 0; i0 < n_cand; i0 += blockDim.x) {
        const int i = i0 + tid;
        const uint32_t key = i < n_cand ? cand_keys[i] : 0xffffffffu;
        const bool eq = i < n_cand && key == thr;
        const uint32_t bal = __ballot_sync(0xffffffffu, eq);
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
        if (i < n_cand) {
          const int rank = base + red[wid] + __popc(bal & ((1u << lane) - 1u));
          if (key < thr || (eq && rank < admit)) {
            const int n = cand_ids[i];
            atomicOr(&w_ev[n >> 5], 1u << (n & 31));
          }
        }
        base += red[33];
      }
      __syncthreads();
    }
    // need >= n_cand: every candidate leaves (w_ev already holds them)
  }

  // ---- 3. outgoing rows release their slots; evict list ------------------------------
  for (int w = tid; w < W; w += blockDim.x) scan[w] = __popc(w_ev[w]);
  const int n_evict = block_exclusive_scan(scan, W, red);
  for (int w = tid; w < W; w += blockDim.x) {
    uint32_t m = w_ev[w];
    int pos = scan[w];
    while (m) {
      const int n = w * 32 + __ffs(m) - 1;
      m &= m - 1;
      const int s = S[n];
      if (p.check && (s < 0 || s >= C)) {
        atomicOr(p.t.status, kStatBadSlot);
      } else {
        owner[s] = -1;
      }
      S[n] = -1;
      if (pos < C) evict_ids[pos] = n;
      ++pos;
    }
  }
  __syncthreads();  // owner[] updates above are read below by other threads

  // ---- 4. free slots, ascending ---------------------------------------------------------
  const int n_avail = compact_indices(
      C, red, [&](int s) { return owner[s] < 0; }, [&](int pos, int s) { free_slots[pos] = s; });

  // ---- 5. i-th incoming row takes the i-th free slot ---------------------------------
  for (int w = tid; w < W; w += blockDim.x) scan[w] = __popc(w_in[w]);
  block_exclusive_scan(scan, W, red);
  const int n_delta = min(n_in, n_avail);
  for (int w = tid; w < W; w += blockDim.x) {
    uint32_t m = w_in[w];
    int pos = scan[w];
    uint32_t placed = 0u;
    while (m) {
      const int bit = __ffs(m) - 1;
      const int n = w * 32 + bit;
      m &= m - 1;
      if (pos < n_avail) {
        const int s = free_slots[pos];
        S[n] = s;
        owner[s] = n;
        delta_ids[pos] = n;
        delta_slots[pos] = s;
        if (h_ids) {
          h_ids[pos] = n;
          h_slots[pos] = s;
        }
        placed |= 1u << bit;
      } else {
        overflow_ids[pos - n_avail] = n;
      }
      ++pos;
    }
    const uint32_t rnew = (R[w] & ~w_ev[w]) | placed;
    R[w] = rnew;
    w_act[w] = P[w] & rnew;
  }
  __syncthreads();  // S[] of placed rows is read below

  // ---- 6. active rows for the sparse MLP: predicted and resident ---------------------
  for (int w = tid; w < W; w += blockDim.x) scan[w] = __popc(w_act[w]);
  const int n_active = block_exclusive_scan(scan, W, red);
  for (int w = tid; w < W; w += blockDim.x) {
    uint32_t m = w_act[w];
    int pos = scan[w];
    while (m) {
      const int n = w * 32 + __ffs(m) - 1;
      m &= m - 1;
      if (pos < C) {
        active_ids[pos] = n;
        active_slots[pos] = S[n];
      }
      ++pos;
    }
  }

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
    if (h_cnt) {
      // list entries above were written by other threads of this block: order them
      // before the counters that tell the host how many entries to read
      __threadfence_system();
      for (int i = 0; i < NP_N_COUNTERS; ++i) h_cnt[i] = v[i];
    }
  }
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
  const size_t sm = (size_t)d.W * 16 + (48 + 256) * 4;
  k_delta<<<d.L, kDeltaThreads, sm, s>>>(p);
  return cudaGetLastError();
}

}  // namespace npi
