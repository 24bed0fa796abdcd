// Internal declarations shared by the translation units of libnp.so.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "np.h"

namespace npi {

constexpr int kMaxBatch = 16;
constexpr int kHostHeaderInts = 16;
constexpr float kRmsEps = 1e-6f;  // x / sqrt(mean(x^2) + eps) in front of every MLP of the chain
#ifndef NP_ZREP
#define NP_ZREP 2
#endif
constexpr int kZRep = NP_ZREP;  // copies of each MLP accumulator vector (spreads same-address adds)  // global header of the host list mirror

// Device-resident tables and lists of all layers (one slab, library-owned).
struct Tables {
  uint32_t* resident;     // [L][W]
  int32_t* slot_map;      // [L][M]
  int32_t* owner;         // [L][C]
  int32_t* stamp;         // [L][M]
  int32_t* delta_ids;     // [L][C]
  int32_t* delta_slots;   // [L][C]
  int32_t* evict_ids;     // [L][C]
  int32_t* active_ids;    // [L][C]
  int32_t* active_slots;  // [L][C]
  int32_t* overflow_ids;  // [L][M]
  int32_t* counters;      // [L][NP_N_COUNTERS]
  int32_t* free_slots;    // [L][C]  scratch of the delta kernel
  int32_t* cand_ids;      // [L][C]  scratch (LRU victim selection)
  uint32_t* cand_keys;    // [L][C]
  uint32_t* pred;         // [L][W]  bitmap of the last np_predict
  int32_t* status;        // [4]     device-side error word(s)
  unsigned int* grid_bar; // [1]     arrival counter of the persistent MLP kernel
  int32_t* identity;      // [M]     0, 1, ..., M-1: the active list of a dense layer
  int32_t* spec_ids;      // [L][C]  rows made resident ahead of time by the last np_speculate
  int32_t* spec_slots;    // [L][C]
  int32_t* spec_counters; // [L][NP_N_COUNTERS] their count sits at NP_CNT_DELTA (the install path reads it there)
  uint32_t* spec_cand;    // [L][W]  candidate bitmap of np_step's own speculation
};

// Carved out of the caller's workspace.
struct Workspace {
  float* hidden;   // [Bmax][H]
  void* hsplit;    // bf16 [48][H]: hidden split into three bf16 terms (tensor-core predictor)
  float* logits;   // [Bmax][L][M]
  float* xbuf[2];  // [Bmax][D] each: x_l of the residual chain, ping-pong
  float* zbuf[3];  // [kZRep][Bmax][D] each: MLP_l(x_l) accumulators, rotating
  float* gu[2];    // [C][2][kMaxBatch] each: gate/up dot products of a layer (batch MLP), alternating
  float* ssq[2];   // [kMaxBatch] each: sum of x_l^2 per sequence
};

struct Dims {
  int L, D, M, H, k, C, W, Bmax;
  int dense;        // leading layers that are dense and fully resident (no selection, no install)
  int rec_int8;     // the store holds 8-bit records (int8 rows + fp32 scales); rec_bytes says how long they are
  int ring_stages;  // cap on shared-memory ring stages of the MLP kernels (0 = as many as fit)
  int Lp;           // layers the record store holds: layer l reads layer l % Lp of it
  size_t rec_bytes;
};

// ---- kernel launchers (each in its own .cu) -------------------------------
cudaError_t launch_tables_reset(const Dims& d, const Tables& t, cudaStream_t s);

cudaError_t launch_pred_l1(const Dims& d, const void* w1, const void* x_bf16, int B, float* hidden,
                           cudaStream_t s);
cudaError_t launch_pred_l2(const Dims& d, const void* w2, const float* hidden, int B, float* logits,
                           int32_t* status, cudaStream_t s, int sm_count);
// whether the ring form of layer 2 (batches without the tensor-core kernel) has room for B hidden vectors of H values
bool pred_l2_ring_fits(int H, int B);
// Tensor-core form of predictor layer 2 for batches (np_predict_tc.cu).
constexpr int kPredL1Parts = 16;  // K ranges (partial sums) of the tensor-core layer 1, at most
struct PredTcState {
  alignas(64) unsigned char map_w2[128];  // CUtensorMap of W2 [L*M][H]
  alignas(64) unsigned char map_h[128];   // CUtensorMap of the split hidden terms [48][H]
  alignas(64) unsigned char map_w1[128];  // CUtensorMap of W1 [H][D]
  void* hsplit;                           // device bf16 [48][H] (workspace)
  float* l1_part;                         // device fp32 [kPredL1Parts][16][H]: layer 1's partial sums per K range
  int n_stages;
  size_t smem;
  int ready;
  int l1_ready, l1_parts, l1_kb_per_block;
};
bool pred_tc_supported(const Dims& d);
bool pred_tc_prepare(const Dims& d, const void* w1, const void* w2, void* hsplit, float* l1_part, int sm_count, PredTcState* st);
cudaError_t launch_pred_l1_tc(const Dims& d, const PredTcState& st, const void* x_bf16, int B, int32_t* status, cudaStream_t s);
cudaError_t launch_pred_l2_tc(const Dims& d, const PredTcState& st, float* hidden, int B, float* logits,
                              int32_t* status, cudaStream_t s, int sm_count, int l1_parts);

cudaError_t launch_topk(const Dims& d, const float* logits, int B, uint32_t* bitmap, cudaStream_t s);

// Centroid heads -> arg-max -> bank lookup -> gate AND up (np_centroid.cu).
cudaError_t launch_centroid_select(const Dims& d, const float* logits, int B, int K, const uint32_t* bank,
                                   int32_t* ids_out, uint32_t* bitmap, cudaStream_t s);

cudaError_t launch_delta(const Dims& d, const Tables& t, const uint32_t* pred, int policy, int step,
                         int32_t* host_lists_dev, int check, cudaStream_t s);
// speculative residency: candidates that are not resident take free slots (np_delta.cu)
cudaError_t launch_speculate(const Dims& d, const Tables& t, const uint32_t* cand, int budget, int32_t* host_lists_dev,
                             cudaStream_t s);

// src_is_store: records are read from the whole-layer store by neuron ID
// (zero-copy); otherwise record r of `src` is the r-th entry of the lists.
cudaError_t launch_scatter(const Dims& d, const void* src, bool src_is_store, const int32_t* ids,
                           const int32_t* slots, const int32_t* count_ptr, int first, int max_rows,
                           void* gate_l, void* up_l, void* downT_l, int32_t* status, int check,
                           cudaStream_t s, int sm_count);

cudaError_t launch_dequant_dense_layer(const Dims& d, const void* store_l, const int32_t* identity, void* dense_l,
                                       int32_t* status, cudaStream_t s, int sm_count);

struct MlpArgs {
  const void* gate_l;
  const void* up_l;
  const void* downT_l;
  const int32_t* active_slots;
  const int32_t* n_active_ptr;  // device counter
  const float* xa;              // x = xa (+ xb)
  const float* xb;              // may be NULL
  float* yacc;                  // [B][D] accumulated with atomics (must hold zeros or a base)
  float* x_store;               // may be NULL: block 0 stores x here
  float* zero_out;              // may be NULL: block 0 clears [B][D] here
  int B;
  int C;
  int check;
  int normalize;     // scale x to unit RMS before the dot products (the chain's pre-MLP norm)
  int force_direct;  // use the direct-load kernel even where the staged one applies
  int32_t* status;
  // tensor-core batch path only (np_mlp_tc.cu); NULL gu keeps the layer on the other kernels
  float* gu;        // [C][2][kMaxBatch] dot-product accumulators of this layer, zero on entry
  float* gu_next;   // the next layer's, cleared by this layer (may be NULL)
  float* ssq;       // [kMaxBatch] sum of x^2 per sequence, zero on entry (needed with normalize)
  float* ssq_next;  // may be NULL
  int gu_rows;      // rows each gu buffer holds (0 = C)
  void* xterms;     // scratch of mlp_tc_xterms_bytes(): x as three bf16 terms for the tcgen05 up kernel (NULL: mma.sync up kernel)
  int dense_rows;   // > 0 (tensor-core path): a dense layer of that many whole records; gate_l / up_l / downT_l point
                    // at the three rows of its first record, active_slots is an identity list, n_active_ptr is not read
};
cudaError_t launch_sparse_mlp(const Dims& d, const MlpArgs& a, cudaStream_t s, int sm_count);
// Batches on tensor cores: two launches per layer (np_mlp_tc.cu).
constexpr int kTcMinBatch = 2;
bool mlp_tc_supported(const Dims& d, int sm_count);
size_t mlp_tc_gu_floats(const Dims& d);
size_t mlp_tc_xterms_bytes(const Dims& d);
bool mlp_tc_up_on_tcgen05(const Dims& d, int sm_count);  // sparse layers of this shape take the tcgen05 up kernel
cudaError_t launch_sparse_mlp_tc(const Dims& d, const MlpArgs& a, cudaStream_t s, int sm_count);

// Arguments of the resident multi-layer kernels for one sequence.
struct ChainArgs {
  const void* gate;  // layer 0 of each row buffer
  const void* up;
  const void* downT;
  const int32_t* active_slots;  // [L][C]
  const int32_t* counters;      // [L][NP_N_COUNTERS]
  const void* x_bf16;  // sliced kernel only, may be NULL: the stack's input, read by the run that starts at layer 0
  float* xbuf[2];
  float* zbuf[3];
  float* x_out;  // may be NULL; a kernel that can leave the stack's result itself (the run ends the stack) does so here
  unsigned int* grid_bar;
  int32_t* status;
  int l_begin, l_end, check;
  int dense_rows;  // > 0 (ALU form only): the layers are dense_rows whole records each, `gate`/`up`/`downT` point
                   // at the three rows of layer 0's first record, active_slots is one identity list
};
namespace dense_chain {  // dense layers, direct loads (np_mlp_dense.cu); same hand-over of x as the other forms
bool supported(const Dims& d, int sm_count);
cudaError_t launch(const Dims& d, const void* rec0, int rows, float* const xbuf[2], float* const zbuf[3],
                   unsigned int* grid_bar, int32_t* status, int l_begin, int l_end, cudaStream_t s, int sm_count);
}  // namespace dense_chain
namespace chain_alu {  // row-partitioned resident kernel (np_mlp_chain_alu.cu): any row width; the sliced kernel's fallback
bool supported(const Dims& d, int sm_count);
cudaError_t launch(const Dims& d, const ChainArgs& a, cudaStream_t s, int sm_count);
}  // namespace chain_alu

namespace chain_slices {  // column-sliced resident form for one sequence (np_mlp_slices.cu); same hand-over of x
struct Plan {
  int R, ks, vg_shift, gw_shift, ng, window, run_layers, slot_cache_rows, max_rows, xch_stride;
  size_t group_bytes, smem;
};
// Library-owned device words and the host's running record of them: the counted sums and the
// exchange stamps only ever grow, so nothing has to be cleared between launches.
struct State {
  unsigned long long* zfix;  // [zfix_words(d)] zero at init / reset
  unsigned int* bars;        // [bar_words()] zero at init / reset
  unsigned long long* xch;   // [xch_words(d, sm_count)] zero at init / reset
  unsigned int bar_base, seq_base;
  int wrote_out;             // the last launch left the stack's result in ChainArgs::x_out
};
bool plan(const Dims& d, int sm_count, Plan* p);
bool supported(const Dims& d, int sm_count);
size_t xch_words(const Dims& d, int sm_count);
bool counted_handover(const Dims& d, int sm_count);  // the sums between layers are counted fixed-point words for this shape
size_t zfix_words(const Dims& d);
size_t bar_words();
cudaError_t launch(const Dims& d, const ChainArgs& a, State* st, cudaStream_t s, int sm_count);
}  // namespace chain_slices

namespace chain_rows {  // whole rows per block, blocks in clusters (np_mlp_rows.cu); same hand-over of x
// Library-owned device words and the host's running record of them: the counters only ever grow
// and the accumulators are used in rotation, so nothing has to be cleared between launches.
struct State {
  float* z4;          // [z_floats(d)] zero at init / reset
  unsigned int* cnt;  // [4] zero at init / reset
  unsigned int cnt_base, seq;
  int grid;           // blocks of a launch (0: the kernel does not apply)
};
size_t z_floats(const Dims& d);
bool prepare(const Dims& d, int sm_count, State* st);
bool supported(const Dims& d, const State& st);
int run_layers(const Dims& d, const State& st);
cudaError_t launch(const Dims& d, const ChainArgs& a, State* st, cudaStream_t s);
}  // namespace chain_rows

cudaError_t launch_selftest_wait(int32_t* status, cudaStream_t s);
cudaError_t launch_widen_bf16(const void* x_bf16, float* out, size_t n, cudaStream_t s);
// out = a + sum of `reps` consecutive copies of b (each n floats)
cudaError_t launch_add_vec(const float* a, const float* b, int reps, float* out, size_t n, cudaStream_t s);

}  // namespace npi
