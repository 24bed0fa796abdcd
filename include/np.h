/*
 * np.h — C ABI of the delta-prefetch sparse-MLP decode path for NVIDIA B200 (sm_100a).
 *
 * One decode step of the method (Section 3.1 of the paper, steps 2-4, in the
 * form the synthetic MLP-stack workload fixes):
 *
 *   np_predict     one predictor pass scores every FFN neuron of every layer and
 *                  keeps the top-k per layer as an active-neuron bitmap
 *   np_delta       compares the predicted sets with the resident rows (Eq. 2-3),
 *                  assigns freed slots to incoming rows, updates the slot map S
 *   np_install     moves only the incoming rows from the neuron-centric record
 *                  store (pinned host memory stands in for the NVMe file) and
 *                  scatters them into the three resident row buffers (Section 3.5)
 *   np_sparse_mlp  SwiGLU MLP over the active resident rows through the slot map
 *   np_step        the four above for one token, with the install of later layers
 *                  overlapped with the MLP of earlier ones
 *
 * Symbols: L layers, D model width, M FFN width, H predictor width, k rows kept
 * per layer per sequence, C resident capacity in rows per layer (the paper's
 * K_max), B sequences, W = M/32 bitmap words per layer, REC = 3*D*2 bytes.
 *
 * Conventions
 *   - Every call returns an int: 0 = NP_OK, < 0 error, > 0 warning (work done).
 *   - "dev" pointers are device global memory, "host" pointers host memory;
 *     "pinned" means page-locked and reachable from the device.
 *   - Streams are passed as void* holding a cudaStream_t (NULL = default stream).
 *     Work is enqueued, not waited for, unless a function says it synchronises.
 *   - The caller owns every large buffer (np_buffers) and keeps it alive and
 *     unchanged in size until np_destroy.  The library owns only its residency
 *     tables, list buffers, events and the context.
 *   - A context is used from one host thread at a time.
 *   - Bitmaps: uint32 words, bit j of word w is neuron 32*w + j.
 *   - bf16 arrays are raw 16-bit patterns; row-major, innermost dimension last.
 *   - There is no CPU fallback: without a CUDA device every compute call fails
 *     with NP_E_CUDA.
 */
#ifndef NP_H_
#define NP_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define NP_VERSION 3

/* return codes */
#define NP_OK           0
#define NP_E_INVAL     -1   /* bad argument or configuration */
#define NP_E_STATE     -2   /* call out of order (e.g. install before delta) */
#define NP_E_CUDA      -3   /* a CUDA runtime call failed; see np_last_error */
#define NP_E_NOMEM     -4   /* allocation of library-owned state failed */
#define NP_E_DEVICE    -5   /* a kernel recorded a status bit (np_last_error prints them): 1 slot, 2 neuron id or
                               4 count out of range; 8 a bounded wait ran out; 16 a block's partial MLP sum was
                               not finite or reached 2^19 in magnitude (the resident one-sequence kernel hands
                               sums between layers in fixed point, resolution 2^-30); state is suspect */
#define NP_E_IO        -6   /* a read of the store file failed or came up short */
#define NP_W_OVERFLOW   1   /* some layer's predicted set did not fit capacity */
#define NP_W_CHUNKED    2   /* some layer's delta exceeded staging and was split */

/* eviction policies (np_config.evict_policy) */
#define NP_EVICT_EXACT  0   /* Eq. 3: every row leaving the predicted set frees its slot */
#define NP_EVICT_LRU    1   /* keep rows while capacity allows; evict least recently predicted,
                               ties by lower neuron index (not in the paper) */

/* how np_install moves records (np_config.transfer_mode) */
#define NP_XFER_MEMCPY_RUNS  0  /* one cudaMemcpyAsync per run of adjacent neuron IDs into
                                   device staging, then the scatter kernel */
#define NP_XFER_HOST_GATHER  1  /* host threads pack records into pinned staging, one
                                   cudaMemcpyAsync per chunk, then the scatter kernel; the
                                   staging buffers are used in up to four parts, round robin */
#define NP_XFER_ZERO_COPY    2  /* the scatter kernel reads the pinned store directly by
                                   neuron ID (the paper's mapped-staging idea); no host sync */
#define NP_XFER_FILE         3  /* the store is a file (Section 3.5): the incoming IDs of a chunk,
                                   already ascending, are coalesced into ranges of adjacent
                                   records and read through io_uring (np_config.io_depth reads
                                   in flight; blocking preads from the host threads where the
                                   kernel offers no io_uring) into parts of the pinned staging,
                                   then one cudaMemcpyAsync per chunk and the scatter kernel as
                                   with HOST_GATHER.  np_buffers.backing is not used;
                                   np_buffers.backing_fd is.  Needs NP_REC_BF16 */

/* how the record store holds a neuron's three rows (np_config.record_format) */
#define NP_REC_BF16  0  /* bf16 rows back to back: gate | up | downT, REC = 3 * D * 2 bytes
                           (Section 3.5) */
#define NP_REC_INT8  1  /* a transfer-path variant the paper leaves as future work: int8 rows
                           gate | up | downT (D bytes each), then their three fp32 scales and 4
                           bytes of padding, REC = 3 * D + 16.  The install path rounds
                           float(q) * scale to bf16 (ties to even) as it places a row, so the
                           resident buffers and the MLP kernels are unchanged and half the
                           bytes cross PCIe.  Needs D % 16 == 0.  Dense layers are rounded the
                           same way once, in np_init */

/* np_config.flags */
#define NP_F_CHECK_BOUNDS    1  /* kernels validate every slot / neuron index and report
                                   through NP_E_DEVICE instead of touching memory */
#define NP_F_DIRECT_LOADS    2  /* sparse MLP: plain 16-byte global loads instead of the
                                   shared-memory staged kernel (for comparison runs) */
#define NP_F_NO_TENSOR_CORES 8  /* np_predict with B > 4: ALU kernel instead of the tcgen05 GEMM
                                   (for comparison runs) */
#define NP_F_LAYER_LAUNCHES  4  /* np_step / np_mlp_chain: one kernel launch per layer instead
                                   of resident kernels spanning runs of layers */
#define NP_F_ROW_CHAIN      32  /* np_step / np_mlp_chain, one sequence: the resident MLP kernel that deals whole rows
                                   to single blocks and reduces through global memory only, instead of the cluster or the
                                   column-sliced one (for comparison runs) */
#define NP_F_CLUSTER_ROWS   64  /* np_step / np_mlp_chain, one sequence: the resident MLP kernel that deals whole rows to
                                   blocks in clusters of four and reduces inside the cluster first (where it applies:
                                   row widths of 1024 to 4096 in steps of 1024), instead of the column-sliced one */
#define NP_F_TCGEN05_BATCH 128  /* batches: the up phase of the sparse MLP as a tcgen05 kernel (rows gathered into
                                   unswizzled K-major tiles, accumulators in tensor memory, x split into bf16 terms
                                   once per layer by a kernel of its own) instead of the mma.sync kernel; applies to
                                   sparse layers whose row width is a multiple of 256, other shapes keep the default.
                                   Results agree with the default to rounding order; measured slower at sixteen
                                   sequences, so off by default */
#define NP_F_MAPPED_STAGING 16  /* NP_XFER_HOST_GATHER / NP_XFER_FILE: no staging copy; the scatter kernel
                                   reads the records in the pinned staging buffer through its device
                                   mapping (Section 3.5: the staging is page-aligned host memory registered
                                   as mapped, so kernels reach it with no copy call in between).  host_staging
                                   must be device-mapped pinned memory; np_buffers.staging is not used */

/* per-layer counters written by np_delta (np_read_counters) */
#define NP_CNT_PRED      0  /* |P|                      */
#define NP_CNT_KEPT      1  /* |P and R_prev|           */
#define NP_CNT_DELTA     2  /* incoming rows given a slot */
#define NP_CNT_EVICT     3  /* rows that released a slot */
#define NP_CNT_OVERFLOW  4  /* incoming rows left without a slot */
#define NP_CNT_ACTIVE    5  /* |P and R| after the update */
#define NP_CNT_RESIDENT  6  /* |R| after the update     */
#define NP_CNT_STEP      7  /* decode step index t of this update */
#define NP_N_COUNTERS    8

typedef struct np_ctx np_ctx;

typedef struct np_config {
  int32_t n_layers;       /* L >= 1 */
  int32_t d_model;        /* D, multiple of 8 */
  int32_t d_ffn;          /* M, multiple of 32 */
  int32_t d_pred;         /* H, multiple of 8 */
  int32_t top_k;          /* k, 0 <= k <= C */
  int32_t capacity;       /* C, 1 <= C <= M */
  int32_t max_batch;      /* largest B any call will pass, 1..16 */
  int32_t evict_policy;   /* NP_EVICT_* */
  int32_t staging_rows;   /* records the staging buffer holds (>= 1); larger deltas are
                             split into chunks (Section 3.5, bounded staging) */
  int32_t transfer_mode;  /* NP_XFER_* */
  int32_t flags;          /* NP_F_* */
  int32_t host_threads;   /* worker threads for NP_XFER_HOST_GATHER (0 = pick) */
  int32_t chain_layers;   /* layers per resident MLP kernel in np_step / np_mlp_chain (0 = runs that
                             shrink towards the end: the last run is an eighth of the stack, the one
                             before it a quarter, the first takes the rest) */
  int32_t ring_stages;    /* cap on the records the MLP kernels stage in shared memory
                             (0 = as many as fit; >= 2 otherwise) */
  int32_t dense_layers;   /* d, 0 <= d <= L: the first d layers are dense (Section 3.1): all M
                             records of each sit in dense_buf (copied from the store by
                             np_init), every row is used, and the layers take no part in
                             selection, delta or install: their rows of every bitmap read as
                             empty and their tables stay empty.  d > 0 excludes
                             NP_F_LAYER_LAUNCHES and NP_F_DIRECT_LOADS, and with max_batch > 1
                             also NP_F_NO_TENSOR_CORES */
  int32_t record_format;  /* NP_REC_*: how the store holds a record */
  int32_t io_depth;       /* NP_XFER_FILE: reads in flight (0 = 256, the paper's queue depth;
                             < 0 = no io_uring, blocking preads from the host threads) */
  int32_t store_layers;   /* Lp, 0 or 1 <= Lp <= L: the store holds Lp layers of records and layer l reads
                             layer l mod Lp of it (0 = L, every layer its own).  For stacks whose whole
                             store the host cannot hold or pin: shapes, row counts and traffic per step
                             stay those of the L-layer stack */
  int32_t spec_rows;      /* s >= 0: np_step / np_step_selected add a speculative prefetch behind every step (see
                             np_speculate): per layer up to s rows ranked k+1 .. k+s by the step's own logits
                             (np_step) become resident in free slots and are transferred after the step's
                             incoming rows.  0 = none */
  int32_t reserved;       /* 0 */
} np_config;

/* Byte counts of the caller-owned buffers for a configuration. */
typedef struct np_sizes {
  uint64_t w1_bytes;          /* bf16 [H][D] */
  uint64_t w2_bytes;          /* bf16 [L*M][H] */
  uint64_t backing_bytes;     /* [Lp][M] records of REC bytes (bf16 [L][M][3][D] with NP_REC_BF16 and store_layers = 0) */
  uint64_t row_buffer_bytes;  /* bf16 [L - d][C][D], each of gate / up / downT (sparse layers only) */
  uint64_t staging_bytes;     /* staging_rows * REC (device; pinned host too for HOST_GATHER) */
  uint64_t workspace_bytes;   /* device scratch */
  uint64_t host_lists_bytes;  /* pinned host area the delta lists are mirrored into */
  uint64_t logits_bytes;      /* fp32 [max_batch][L][M] */
  uint64_t bitmap_bytes;      /* uint32 [L][W] */
  uint64_t record_bytes;      /* REC */
  uint64_t dense_bytes;       /* bf16 [d][M][3][D]: the dense layers' records (0 when d = 0) */
} np_sizes;

typedef struct np_buffers {
  const void* w1;          /* dev  */
  const void* w2;          /* dev  */
  const void* backing;     /* pinned host (cudaHostAlloc or cudaHostRegister); may be NULL with
                              NP_XFER_FILE */
  void* gate_buf;          /* dev  */
  void* up_buf;            /* dev  */
  void* downT_buf;         /* dev  */
  void* staging;           /* dev; unused (may be NULL) with NP_XFER_ZERO_COPY */
  void* host_staging;      /* pinned host, staging_bytes; only for NP_XFER_HOST_GATHER and
                              NP_XFER_FILE */
  void* workspace;         /* dev, 256-byte aligned */
  void* host_lists;        /* pinned host */
  void* dense_buf;         /* dev, dense_bytes; NULL when dense_layers = 0.  Filled by np_init */
  int32_t backing_fd;      /* NP_XFER_FILE: descriptor of the store file, record (l, n) at byte
                              (l*M + n)*REC, open for reading for the life of the context and
                              owned by the caller.  With O_DIRECT (the paper's way; reads then
                              bypass the page cache) REC must suit the file system's alignment
                              rule, commonly a multiple of 512 bytes; the staging parts are
                              4096-byte aligned when host_staging is.  Ignored otherwise */
  int32_t reserved;        /* 0 */
} np_buffers;

/* Device views of one layer's lists from the last np_delta (valid until the next). */
typedef struct np_delta_view {
  const int32_t* delta_ids;     /* dev [n_delta]    incoming neurons, ascending */
  const int32_t* delta_slots;   /* dev [n_delta]    their slots */
  const int32_t* evict_ids;     /* dev [n_evict]    neurons that released their slot, ascending */
  const int32_t* overflow_ids;  /* dev [n_overflow] incoming neurons left non-resident, ascending */
  const int32_t* active_ids;    /* dev [n_active]   predicted and resident, ascending */
  const int32_t* active_slots;  /* dev [n_active] */
  const int32_t* counters;      /* dev [NP_N_COUNTERS] */
} np_delta_view;

/* Library version (NP_VERSION of the build). */
int np_version(void);

/* Fills *out with the buffer sizes `cfg` needs.  Pure host arithmetic (record
 * size: Section 3.5; buffer size: Section 4.3).  NP_E_INVAL on a bad config. */
int np_query_sizes(const np_config* cfg, np_sizes* out);

/* The dense/sparse split's memory rule (Section 3.1: as many leading layers stay
 * dense as the memory budget has room for): the largest d in [0, L] with
 *   d * M * REC + (L - d) * C * REC + fixed_bytes <= budget_bytes,
 * i.e. d dense layers, resident buffers of C records for the rest, next to
 * fixed_bytes of other resident state.  cfg->dense_layers is ignored.
 * *d_out = -1 when not even d = 0 fits.  Pure host arithmetic.  (The paper
 * finds its operating point by a throughput sweep on its device; this is the
 * rule that sweep is described by.)  NP_E_INVAL on a bad config or NULL. */
int np_plan_dense_prefix(const np_config* cfg, uint64_t budget_bytes, uint64_t fixed_bytes, int32_t* d_out);

/* Creates a context with empty residency (the cold-start state of Section 3.4:
 * no row resident, every slot free).  Copies cfg; keeps the pointers in bufs.
 * Allocates the library's tables on the current device and synchronises.
 * Errors: NP_E_INVAL (config, NULL/misaligned/unpinned buffers), NP_E_NOMEM, NP_E_CUDA. */
int np_init(np_ctx** out, const np_config* cfg, const np_buffers* bufs);

/* Waits for the context's outstanding work, frees library-owned memory. */
int np_destroy(np_ctx* ctx);

/* Back to the cold-start state (tables cleared, step counter 0); the row
 * buffers are left as they are.  Enqueued on `stream`. */
int np_reset(np_ctx* ctx, void* stream);

/* Text of the last error of this context (or of the last failed np_init /
 * np_query_sizes when ctx is NULL).  Never NULL; valid until the next call. */
const char* np_last_error(const np_ctx* ctx);

/* Stage 1 + 2: predictor forward and per-layer top-k (Section 3.1 step 2; the
 * workload's predictor is logits = W2 * relu(W1 * x), no biases).
 *   x_bf16       dev bf16 [B][D]   layer-0 hidden states
 *   logits_out   dev fp32 [B][L][M] or NULL (kept internally either way)
 *   bitmap_out   dev uint32 [L][W] or NULL: union over the B sequences of each
 *                sequence's k highest logits per layer; order = fp32 value
 *                descending (+0 above -0), ties to the lower neuron index
 * The bitmap is also kept inside the context for np_delta(ctx, NULL, ...).
 * Dense layers (dense_layers > 0) select nothing: their bitmap rows are zero
 * (with B = 1 they are not even scored and their logits are left untouched).
 * Errors: NP_E_INVAL (NULL x, B outside 1..max_batch), NP_E_CUDA. */
int np_predict(np_ctx* ctx, const void* x_bf16, int32_t B, float* logits_out,
               uint32_t* bitmap_out, void* stream);

/* Stage 2 alone on caller-supplied logits (dev fp32 [B][L][M]) -> bitmap_out
 * (dev uint32 [L][W], required).  Does not touch the context's own bitmap. */
int np_topk(np_ctx* ctx, const float* logits, int32_t B, uint32_t* bitmap_out, void* stream);

/* Stage 2 in the paper's own form (Section 3.3, the heads of the predictor;
 * Section 3.4, the gate/up intersection): per sequence and layer two heads
 * score a vocabulary of K centroids, each head takes its highest-scoring
 * centroid (ties: the lower ID; order as in np_predict), and the layer's
 * active set is gate_mask[id_gate] AND up_mask[id_up], ORed over sequences.
 *   logits      dev fp32 [B][L][2][K]   head 0 = gate, head 1 = up
 *   bank        dev uint32 [L][2][K][W] bit-packed centroid masks (caller-owned,
 *               read only); the sets it yields may have any size up to M
 *   ids_out     dev int32 [B][L][2] chosen centroid IDs, or NULL
 *   bitmap_out  dev uint32 [L][W], required; pass it to np_delta
 * Does not touch the context's own bitmap.  Logits of this shape come from
 * np_predict_logits_noalloc with d_ffn = 2*K, or from any other producer.
 * Errors: NP_E_INVAL (NULL pointer, B outside 1..max_batch, K < 1), NP_E_CUDA. */
int np_centroid_select(np_ctx* ctx, const float* logits, int32_t B, int32_t K, const uint32_t* bank,
                       int32_t* ids_out, uint32_t* bitmap_out, void* stream);

/* Stage 3a: delta and residency update for all layers (Section 3.4, Eq. 2-3).
 *   pred_bitmap  dev uint32 [L][W], or NULL to use the last np_predict's result.
 * Per layer: incoming = P \ R (ascending), victims per the eviction policy,
 * victims' slots cleared in S/owner, i-th incoming row gets the i-th free slot
 * (ascending slot index); rows beyond the free slots are listed as overflow and
 * stay non-resident.  Tables are updated here, before the rows arrive; use
 * np_install before np_sparse_mlp.  Advances the step counter.
 * Does not synchronise.  Warnings are reported by np_install / np_read_counters. */
int np_delta(np_ctx* ctx, const uint32_t* pred_bitmap, void* stream);

/* Stage 3b of the file path on its own, no GPU involved (Section 3.5): reads records
 * ids[0..n) (strictly ascending; record `id` = file bytes [base_offset + id*rec_bytes,
 * +rec_bytes)) into dst + i*rec_bytes, one range per run of adjacent IDs, with io_depth reads
 * in flight (meaning as np_config.io_depth).  Blocks until every read has completed.
 * `dst` is host memory the caller owns (aligned as the descriptor's flags demand).
 * *n_ranges_out (may be NULL) = coalesced ranges; *used_ring_out (may be NULL) = 1 if io_uring
 * carried the reads, 0 if blocking preads did.
 * Errors: NP_E_INVAL (descriptor, sizes, NULL, unsorted ids), NP_E_IO; text in np_last_error(NULL). */
int np_read_records(int32_t fd, uint64_t base_offset, uint64_t rec_bytes, const int32_t* ids, int32_t n, void* dst,
                    int32_t io_depth, int32_t* n_ranges_out, int32_t* used_ring_out);

/* Stage 3b + 3c for layers [layer_begin, layer_end): copy each incoming record
 * (L, n) = bytes [(l*M + n)*REC, +REC) of the store to slot S[n] of the three
 * row buffers, on `copy_stream`, and mark each layer installed (np_sparse_mlp
 * orders itself after that mark).  The copy stream is first ordered after the
 * delta step.  Scatter kernels may run on streams the library owns; those are
 * ordered after the work `copy_stream` held on entry and joined back into it
 * before the call returns, so work queued on `copy_stream` afterwards sees
 * every row installed.  With NP_XFER_MEMCPY_RUNS / NP_XFER_HOST_GATHER / NP_XFER_FILE this
 * call blocks the host until the delta lists of the last np_delta are readable (and, with
 * NP_XFER_FILE, until the last chunk's reads have completed); with NP_XFER_ZERO_COPY it
 * never blocks.  Deltas larger than staging_rows are split
 * into chunks in list order (result unchanged).
 * Returns NP_W_OVERFLOW / NP_W_CHUNKED (OVERFLOW wins) where it can know.
 * Errors: NP_E_STATE (no np_delta since init/reset), NP_E_INVAL, NP_E_CUDA, NP_E_IO (a file
 * read failed: no read is left in flight when the call returns, the layers from the failing
 * chunk on are not marked installed). */
int np_install(np_ctx* ctx, int32_t layer_begin, int32_t layer_end, void* copy_stream);

/* Stage 4 for one layer (Section 3.4): over act = P and R of the last np_delta,
 *   y[b] = sum_{i in act} silu(gate[S[i]].x[b]) * (up[S[i]].x[b]) * downT[S[i]]
 *   x  dev fp32 [B][D],  y  dev fp32 [B][D] (overwritten)
 * bf16 rows, fp32 accumulation; partial sums are combined with floating-point
 * atomics, so the last bits of y can differ between runs.
 * `stream` is first ordered after the layer's install mark.
 * Dense layers run only inside np_mlp_chain / np_step (NP_E_INVAL here).
 * Errors: NP_E_STATE, NP_E_INVAL, NP_E_CUDA. */
int np_sparse_mlp(np_ctx* ctx, int32_t layer, const float* x, int32_t B, float* y, void* stream);

/* One whole decode step: np_predict, np_delta, np_install of every layer on
 * `copy_stream`, and the pre-normalised residual MLP chain
 *   x_{l+1} = x_l + MLP_l(n_l),  n_l = x_l / sqrt(mean(x_l^2) + 1e-6)
 * on `stream`, x_0 = x_bf16 widened to fp32 (the RMS normalisation with unit gain stands
 * for the per-layer norm in front of every MLP block of the paper's models).
 *   x_out  dev fp32 [B][D]  x_L
 * Host-blocking exactly as np_install.  Returns warnings like np_install. */
int np_step(np_ctx* ctx, const void* x_bf16, int32_t B, float* x_out, void* stream,
            void* copy_stream);

/* The same step with the selection taken from the caller: `bitmap` (dev uint32
 * [L][W], e.g. from np_centroid_select) replaces np_predict's top-k result;
 * delta, install and the MLP chain run as in np_step, with the same ordering
 * (a dense prefix is queued before the install).  np_last_step_times then
 * reports 0 for the prediction stage.
 * Errors: as np_step, and NP_E_INVAL for a NULL bitmap. */
int np_step_selected(np_ctx* ctx, const void* x_bf16, int32_t B, const uint32_t* bitmap, float* x_out,
                     void* stream, void* copy_stream);

/* Stage 4 for every layer in order, nothing else: the chain of np_step,
 * x_{l+1} = x_l + MLP_l(x_l / rms(x_l)), over the rows that are active and resident now
 * (Section 3.1: the sparse suffix runs once the delta rows are in place).
 *   x_bf16  dev bf16 [B][D]  x_0,   x_out  dev fp32 [B][D]  x_L
 * Orders `stream` after any pending install marks.  Errors as np_sparse_mlp. */
int np_mlp_chain(np_ctx* ctx, const void* x_bf16, int32_t B, float* x_out, void* stream);

/* Number of kernels this context has launched since np_init (memsets and
 * copies are not counted).  Host counter, no synchronisation. */
int np_launch_count(np_ctx* ctx, uint64_t* out);

/* Failure-detection self-test.  Every device-side wait of this library (mbarrier, grid
 * barrier) is bounded: after a fixed number of polls the kernel records a time-out in the
 * context's device status word and returns, and the next synchronising call reports
 * NP_E_DEVICE.  This call launches a kernel whose wait can never be satisfied (about 25 ms),
 * synchronises `stream` and returns NP_E_DEVICE if the time-out was recorded as it should
 * be (NP_E_STATE if it was not).  The status word stays set until np_reset. */
int np_selftest_bounded_wait(np_ctx* ctx, void* stream);

/* Device pointers to one layer's lists and counters from the last np_delta. */
int np_get_delta(np_ctx* ctx, int32_t layer, np_delta_view* out);

/* Copies all layers' counters to host int32 [L][NP_N_COUNTERS]; synchronises `stream`. */
int np_read_counters(np_ctx* ctx, int32_t* out_host, void* stream);

/* Copies one layer's residency tables to host arrays (any may be NULL) and
 * synchronises `stream`:  slot_map int32 [M] (-1 = not resident), owner int32 [C]
 * (-1 = free), resident uint32 [W], stamp int32 [M] (step of last prediction, -1 never). */
int np_export_state(np_ctx* ctx, int32_t layer, int32_t* slot_map, int32_t* owner,
                    uint32_t* resident, int32_t* stamp, void* stream);

/* Overwrites one layer's tables from host arrays (all required) and sets the
 * step counter; the caller vouches for their consistency.  Synchronises. */
int np_import_state(np_ctx* ctx, int32_t layer, const int32_t* slot_map, const int32_t* owner,
                    const uint32_t* resident, const int32_t* stamp, int32_t step, void* stream);

/* Speculative residency behind a step: the "deeper prefetch pipeline" the paper names as future work
 * (Section 6).  Residency is a cache: a row may be made resident before any token asks for it without
 * changing a result; what changes is the next token's incoming set P \ R (Eq. 2).  After np_delta and
 * before the next one, per layer: of the rows of cand_bitmap (dev uint32 [L][W]) that are not resident,
 * the min(budget, free slots) lowest-indexed become resident; the i-th of them (ascending neuron) takes
 * the i-th free slot (ascending slot), as incoming rows do.  Nothing is evicted, no stamp changes (under
 * NP_EVICT_LRU a speculative row that is never predicted is among the first to leave; under
 * NP_EVICT_EXACT it leaves at the next step).  The rule is this library's: the paper gives none.
 * The lists (np_get_speculative) are mirrored to the host; np_install_speculative transfers the rows
 * exactly as np_install transfers incoming rows (same transfer mode, chunking and per-layer marks), and
 * is meant to be queued after the step's own np_install and MLP launches.  Dense layers take none.
 * Errors: NP_E_STATE (no np_delta yet / np_install_speculative without np_speculate), NP_E_INVAL, NP_E_CUDA. */
int np_speculate(np_ctx* ctx, const uint32_t* cand_bitmap, int32_t budget, void* stream);
int np_install_speculative(np_ctx* ctx, void* copy_stream);
/* Device views of one layer's speculative rows of the last np_speculate: ids and slots (ascending neuron),
 * and their count.  Valid until the next np_speculate. */
int np_get_speculative(np_ctx* ctx, int32_t layer, const int32_t** ids, const int32_t** slots, const int32_t** count);

/* Launches of the resident MLP kernel (sparse layers, one sequence) made by the last np_mlp_chain / np_step:
 * the runs the chain was cut into.  0 when that call ran per-layer or batch kernels.  For reports. */
int np_chain_launches(np_ctx* ctx, int32_t* out);

/* Name of the kernel np_mlp_chain / np_step run the sparse layers' MLP with for B sequences in this
 * context (a static string: "k_mlp_slices", "k_mlp_chain_alu", "k_mlp_tc_up + k_mlp_tc_down",
 * "k_sparse_mlp_pipe" or "k_sparse_mlp").  For reports; NULL if ctx is NULL or B is out of range. */
const char* np_mlp_kernel_name(np_ctx* ctx, int32_t B);

/* Timing of the last np_step in microseconds, host float [4]: predict+top-k,
 * delta, install (copy stream, first enqueue to last mark), MLP chain.
 * Synchronises both streams of that step.  NP_E_STATE if no step ran. */
int np_last_step_times(np_ctx* ctx, float* out_us);

/* Largest B * d_pred np_predict_logits_noalloc accepts, in floats of fixed scratch (enough
 * for 16 sequences at d_pred = 1024).  With its status words the array costs every GPU that
 * loads the library 64 KiB + 256 B of device memory until the process exits. */
#define NP_NOALLOC_MAX_HIDDEN_FLOATS 16384

/* Predictor forward pass (stage 1 only: logits = W2 * relu(W1 * x)) without a context and
 * without any allocation.  The paper has no counterpart; this exists for callers that cannot
 * call cudaMalloc: code that runs under a memory pool which owns all device memory, a decode
 * loop that cannot afford the device-wide synchronisation an allocation may imply, or a process
 * whose device memory is budgeted to the byte.  np_init allocates, so such callers cannot use a
 * context; here the scratch between the two predictor layers is a fixed array inside the library.
 *   w1 dev bf16 [d_pred][d_model], w2 dev bf16 [n_layers*d_ffn][d_pred], x_bf16 dev bf16 [B][d_model]
 *   logits_out dev fp32 [B][n_layers][d_ffn]   (all caller-owned, 16-byte aligned)
 * Bit-identical to np_predict's logits in a context created with NP_F_NO_TENSOR_CORES (the same
 * plain-core kernels); a default context takes the tensor-core kernel for B > 4, whose rounding
 * differs (both are within rel-L2 1e-5 of the exact product).  Calls no cudaMalloc / cudaFree or
 * allocating library routine.  Every call first clears the status words in the scratch; a kernel
 * whose bounded wait runs out records a bit there, leaves part of logits_out unwritten and the
 * call still returns NP_OK (it does not synchronise): np_noalloc_check reports it.  The first call on a device looks up the scratch array's device address
 * (cudaGetSymbolAddress, with that device current); make that first call before any stream
 * capture.  All calls on a device share the one scratch array: calls that may overlap on the GPU
 * (different streams) race on it and must be serialised by the caller.
 * Errors: NP_E_INVAL (NULL / misaligned pointer, shape outside np_config's limits, or
 * B * d_pred > NP_NOALLOC_MAX_HIDDEN_FLOATS), NP_E_CUDA; text in np_noalloc_last_error(). */
int np_predict_logits_noalloc(const void* w1, const void* w2, const void* x_bf16, int32_t B,
                              int32_t n_layers, int32_t d_model, int32_t d_ffn, int32_t d_pred,
                              float* logits_out, void* stream);

/* Waits for `stream` and returns NP_E_DEVICE if the kernels of the last
 * np_predict_logits_noalloc on the current device recorded a status bit (a bounded wait ran
 * out: logits incomplete), NP_OK if not, NP_E_STATE if that entry point never ran on this
 * device.  Allocates nothing (the word is copied to the caller's stack).  The paper has no
 * counterpart. */
int np_noalloc_check(void* stream);

/* Text of the calling thread's last np_predict_logits_noalloc / np_noalloc_check error.  Never NULL. */
const char* np_noalloc_last_error(void);

/* ---- The shared predictor of Section 3.3 (projection blocks -> residual trunk -> centroid
 * heads), for one token.  Stands beside np_predict: its head logits feed np_centroid_select.
 * No context is needed; the caller owns weights, features and workspace (all device memory).
 *
 * Stage 1: feature i (fp32 [feature_dim[i]]) -> Linear -> LayerNorm -> SiLU -> T values; the
 * layer-0 gate centroid ID -> row of the embedding -> Linear -> LayerNorm -> SiLU -> 4T values;
 * concatenated to z (8T).  Stage 2: n_blocks times z <- z + W2 SiLU(LayerNorm(W1 z + b1)) + b2,
 * W1: 8T -> 4T, W2: 4T -> 8T.  Stage 3: head_logits[l][g][k] = heads[(l*2 + g)*K + k] . z for
 * the n_heads sparse layers, g = 0 gate, 1 up (the layout np_centroid_select reads at B = 1).
 * LayerNorm: biased variance, epsilon 1e-5.  Dropout is the identity (inference).
 * Matrices are bf16, row-major [out][in], 16-byte aligned; vectors fp32.  Dimensions that are
 * not multiples of 8 (the scalar norm feature) are passed padded with zeros, their weight rows
 * padded with zero columns. */
#define NP_TRUNK_MAX_BLOCKS 16
typedef struct np_trunk_desc {
  int32_t T;               /* width of a projection block's output, multiple of 8, <= 1024 */
  int32_t n_features;      /* 4 */
  int32_t feature_dim[4];  /* padded to multiples of 8 */
  int32_t K0;              /* layer-0 gate centroid vocabulary (rows of the embedding) */
  int32_t E;               /* embedding width, multiple of 8 */
  int32_t n_blocks;        /* residual blocks, 0..NP_TRUNK_MAX_BLOCKS */
  int32_t n_heads;         /* sparse layers: 2 * n_heads heads */
  int32_t K;               /* centroid vocabulary per head */
  int32_t reserved[5];     /* 0 */
} np_trunk_desc;
typedef struct np_trunk_weights {
  const void* proj_w[4];       /* bf16 [T][feature_dim[i]] */
  const float* proj_b[4];      /* [T] linear bias */
  const float* proj_gain[4];   /* [T] LayerNorm gain */
  const float* proj_bias[4];   /* [T] LayerNorm bias */
  const void* emb;             /* bf16 [K0][E] */
  const void* cproj_w;         /* bf16 [4T][E] */
  const float* cproj_b;        /* [4T] */
  const float* cproj_gain;     /* [4T] */
  const float* cproj_bias;     /* [4T] */
  const void* blk_w1[NP_TRUNK_MAX_BLOCKS];    /* bf16 [4T][8T] */
  const float* blk_b1[NP_TRUNK_MAX_BLOCKS];   /* [4T] */
  const float* blk_gain[NP_TRUNK_MAX_BLOCKS]; /* [4T] */
  const float* blk_bias[NP_TRUNK_MAX_BLOCKS]; /* [4T] */
  const void* blk_w2[NP_TRUNK_MAX_BLOCKS];    /* bf16 [8T][4T] */
  const float* blk_b2[NP_TRUNK_MAX_BLOCKS];   /* [8T] */
  const void* heads;           /* bf16 [n_heads * 2 * K][8T], no bias */
} np_trunk_weights;

/* Floats of device workspace np_trunk_forward needs for `desc` (28 * T).  NP_E_INVAL on a bad T. */
int np_trunk_workspace_floats(const np_trunk_desc* desc, uint64_t* out);

/* Queues the forward pass on `stream` (11 kernel launches at four blocks; no synchronisation,
 * no allocation).  `features`: host array of four device pointers; `centroid_id`: device
 * scalar in [0, K0); `workspace`: device, 16-byte aligned, np_trunk_workspace_floats floats;
 * `head_logits`: device fp32 [n_heads][2][K].
 * Errors: NP_E_INVAL (NULL pointer, dimension outside its range), NP_E_CUDA; text in
 * np_trunk_last_error(). */
int np_trunk_forward(const np_trunk_desc* desc, const np_trunk_weights* weights, const float* const* features,
                     const int32_t* centroid_id, float* workspace, float* head_logits, void* stream);
const char* np_trunk_last_error(void);

#ifdef __cplusplus
}
#endif
#endif  /* NP_H_ */
