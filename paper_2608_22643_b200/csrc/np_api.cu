// C ABI of libnp.so: context, argument checking, stream/event ordering and the
// host side of the install path (run coalescing, chunking, staging).  Every
// arithmetic step runs in the kernels of the sibling .cu files.
#include <algorithm>
#include <atomic>
#include <chrono>
#include <condition_variable>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <functional>
#include <mutex>
#include <new>
#include <deque>
#include <thread>
#if defined(__SSE2__)
#include <emmintrin.h>
#include <xmmintrin.h>
#include <sys/stat.h>
#endif

#include "np_internal.h"
#include "np_io.h"

using namespace npi;

namespace {

thread_local std::string g_last_error = "";

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Packs one record into pinned staging.  The staging lines are written once and read next by
// the copy engine, never by this core: non-temporal stores skip the read-for-ownership a
// cached store would cost (both pointers are 16-byte aligned, n a multiple of 16).
void copy_record_streaming(void* dst, const void* src, size_t n) {
#if defined(__SSE2__)
  const __m128i* s = static_cast<const __m128i*>(src);
  __m128i* d = static_cast<__m128i*>(dst);
  const size_t m = n / 16;
  size_t i = 0;
  for (; i + 4 <= m; i += 4) {
    _mm_prefetch(reinterpret_cast<const char*>(s + i) + 512, _MM_HINT_NTA);
    const __m128i a = _mm_load_si128(s + i), b = _mm_load_si128(s + i + 1);
    const __m128i c = _mm_load_si128(s + i + 2), e = _mm_load_si128(s + i + 3);
    _mm_stream_si128(d + i, a);
    _mm_stream_si128(d + i + 1, b);
    _mm_stream_si128(d + i + 2, c);
    _mm_stream_si128(d + i + 3, e);
  }
  for (; i < m; ++i) _mm_stream_si128(d + i, _mm_load_si128(s + i));
  _mm_sfence();
#else
  memcpy(dst, src, n);
#endif
}

// Small fork-join pool for packing records into pinned staging.  A step issues one short
// job per layer, tens of microseconds apart, so idle workers spin on the job counter for a
// while before they go to sleep on the condition variable (a sleeping thread takes longer
// to wake than a layer's records take to pack).
class Pool {
 public:
  explicit Pool(int n) {
    for (int i = 0; i < n; ++i) threads_.emplace_back([this] { run(); });
  }
  ~Pool() {
    {
      std::lock_guard<std::mutex> lk(m_);
      stop_.store(true);
      ticket_.fetch_add(1ull << 32);
    }
    cv_.notify_all();
    for (auto& t : threads_) t.join();
  }
  // Calls fn(i) for i in [0, count) on the workers and the caller; returns when all are done.
  void parallel_for(int count, const std::function<void(int)>& fn) {
    if (count <= 0) return;
    if (threads_.empty() || count == 1) {
      for (int i = 0; i < count; ++i) fn(i);
      return;
    }
    // Index claims carry the job's generation, so a worker that is late leaving one job can
    // never claim (or count) an index of the next.
    const uint64_t g = (ticket_.load() >> 32) + 1;
    Job& job = jobs_[g & 1];
    job.fn.store(&fn);
    job.count.store(count);
    job.done.store(0);
    {
      std::lock_guard<std::mutex> lk(m_);  // pairs with the sleepers' predicate check
      ticket_.store(g << 32);
    }
    if (sleepers_.load() > 0) cv_.notify_all();
    work(g);
    while (job.done.load(std::memory_order_acquire) < count) cpu_relax();
  }
  int size() const { return (int)threads_.size(); }

 private:
  struct Job {
    std::atomic<const std::function<void(int)>*> fn{nullptr};
    std::atomic<int> count{0};
    std::atomic<int> done{0};
  };
  static void cpu_relax() {
#if defined(__x86_64__) || defined(__i386__)
    __builtin_ia32_pause();
#else
    std::this_thread::yield();
#endif
  }
  void work(uint64_t g) {
    Job& job = jobs_[g & 1];
    const std::function<void(int)>* fn = job.fn.load();
    const int count = job.count.load();
    for (;;) {
      uint64_t t = ticket_.load();
      if ((t >> 32) != g) return;  // the job is over (and fn / count may belong to a later one)
      const int i = (int)(t & 0xffffffffu);
      if (i >= count) return;
      if (!ticket_.compare_exchange_weak(t, t + 1)) continue;
      (*fn)(i);
      job.done.fetch_add(1, std::memory_order_release);
    }
  }
  void run() {
    uint64_t seen = 0;
    for (;;) {
      // spin for roughly a quarter of a millisecond, then sleep
      bool got = false;
      const auto t0 = std::chrono::steady_clock::now();
      for (int spin = 0;; ++spin) {
        if ((ticket_.load(std::memory_order_acquire) >> 32) != seen) {
          got = true;
          break;
        }
        cpu_relax();
        if ((spin & 1023) == 1023 &&
            std::chrono::steady_clock::now() - t0 > std::chrono::microseconds(250))
          break;
      }
      if (!got) {
        std::unique_lock<std::mutex> lk(m_);
        sleepers_.fetch_add(1);
        cv_.wait(lk, [&] { return (ticket_.load() >> 32) != seen; });
        sleepers_.fetch_sub(1);
      }
      seen = ticket_.load(std::memory_order_acquire) >> 32;
      if (stop_.load()) return;
      work(seen);
    }
  }
  std::vector<std::thread> threads_;
  std::mutex m_;
  std::condition_variable cv_;
  std::atomic<bool> stop_{false};
  std::atomic<uint64_t> ticket_{0};  // generation << 32 | next index of that generation's job
  std::atomic<int> sleepers_{0};
  Job jobs_[2];
};

}  // namespace

constexpr int kStageParts = 4;  // most parts the host-gather staging is split into

struct np_ctx {
  np_config cfg;
  np_buffers bufs;
  Dims d;
  Tables t;
  Workspace ws;
  void* slab = nullptr;
  int device = 0;
  int sm_count = 0;
  int32_t* host_lists = nullptr;      // host address
  int32_t* host_lists_dev = nullptr;  // device alias
  const char* backing_dev = nullptr;  // device alias of the record store
  char* hstage_dev = nullptr;         // device alias of the pinned staging (NP_F_MAPPED_STAGING)
  cudaEvent_t ev_delta = nullptr;
  cudaEvent_t ev_spec = nullptr;      // the lists of the last np_speculate are written
  std::vector<cudaEvent_t> ev_installed;
  std::vector<char> install_pending;
  cudaEvent_t ev_half[kStageParts] = {};        // parts of the host / device staging in flight
  // library-owned side streams of the install path: [0] runs the scatter kernels behind the
  // staged copies; in zero-copy mode consecutive layers alternate between the two
  cudaStream_t aux[2] = {nullptr, nullptr};
  cudaEvent_t ev_fork = nullptr, ev_join[2] = {nullptr, nullptr}, ev_copied[kStageParts] = {};
  bool half_pending[kStageParts] = {};
  int next_half = 0;
  cudaEvent_t ev_t[4] = {nullptr, nullptr, nullptr, nullptr};  // compute-stream step timing
  cudaEvent_t ev_c[2] = {nullptr, nullptr};                    // copy-stream step timing
  bool have_delta = false;
  bool have_spec = false;   // np_speculate has run since the last np_delta
  bool have_pred = false;
  bool have_step = false;
  int step = 0;
  uint64_t launches = 0;
  Pool* pool = nullptr;
  RecordReader reader;   // NP_XFER_FILE: reads of the store file
  PredTcState tc = {};
  chain_slices::State slices = {};  // column-sliced resident MLP kernel: its counters, exchange words and their values
  bool use_slices = false;
  void* xterms = nullptr;  // scratch of the tcgen05 up kernel of the batch MLP
  chain_rows::State rows = {};  // cluster form of the resident MLP kernel (whole rows per block): its accumulators and counters
  bool use_rows = false;
  int chain_kernel_launches = 0;    // MLP kernel launches of the last np_mlp_chain / np_step
  size_t gu_bytes = 0;   // both dot-product accumulators of the batch MLP, contiguous
  bool mlp_tc = false;   // batches run the tensor-core MLP kernels
  std::string err;
};

namespace {

int fail(np_ctx* ctx, int code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (ctx) ctx->err = buf;
  g_last_error = buf;
  return code;
}

#define NP_CUDA(ctx, call)                                                                  \
  do {                                                                                      \
    cudaError_t e__ = (call);                                                               \
    if (e__ != cudaSuccess)                                                                 \
      return fail(ctx, NP_E_CUDA, "%s failed: %s (%s:%d)", #call, cudaGetErrorString(e__),  \
                  __FILE__, __LINE__);                                                      \
  } while (0)

// a kernel launch: counted, then checked
#define NP_LAUNCH(ctx, call) \
  do {                       \
    (ctx)->launches += 1;    \
    NP_CUDA(ctx, call);      \
  } while (0)

int check_config(const np_config* c, np_ctx* ctx) {
  if (!c) return fail(ctx, NP_E_INVAL, "config is NULL");
  if (c->n_layers < 1) return fail(ctx, NP_E_INVAL, "n_layers must be >= 1");
  if (c->d_model < 8 || c->d_model % 8 || c->d_model > 16384)
    return fail(ctx, NP_E_INVAL, "d_model must be a multiple of 8 in [8, 16384]");
  if (c->d_ffn < 32 || c->d_ffn % 32 || c->d_ffn > 40960)
    return fail(ctx, NP_E_INVAL, "d_ffn must be a multiple of 32 in [32, 40960]");
  if (c->d_pred < 8 || c->d_pred % 8 || c->d_pred > 4096)
    return fail(ctx, NP_E_INVAL, "d_pred must be a multiple of 8 in [8, 4096]");
  if (c->capacity < 1 || c->capacity > c->d_ffn) return fail(ctx, NP_E_INVAL, "capacity must be in [1, d_ffn]");
  if (c->top_k < 0 || c->top_k > c->capacity) return fail(ctx, NP_E_INVAL, "top_k must be in [0, capacity]");
  if (c->max_batch < 1 || c->max_batch > kMaxBatch) return fail(ctx, NP_E_INVAL, "max_batch must be in [1, 16]");
  if (c->evict_policy != NP_EVICT_EXACT && c->evict_policy != NP_EVICT_LRU)
    return fail(ctx, NP_E_INVAL, "unknown evict_policy");
  if (c->transfer_mode < NP_XFER_MEMCPY_RUNS || c->transfer_mode > NP_XFER_FILE)
    return fail(ctx, NP_E_INVAL, "unknown transfer_mode");
  if (c->staging_rows < 1) return fail(ctx, NP_E_INVAL, "staging_rows must be >= 1");
  if ((c->transfer_mode == NP_XFER_HOST_GATHER || c->transfer_mode == NP_XFER_FILE) && c->staging_rows < 2)
    return fail(ctx, NP_E_INVAL, "host gather and file reads need staging_rows >= 2 (at least two parts)");
  if (c->transfer_mode == NP_XFER_FILE && c->record_format != NP_REC_BF16)
    return fail(ctx, NP_E_INVAL, "NP_XFER_FILE needs NP_REC_BF16 records");
  if (c->io_depth < -1 || c->io_depth > 4096) return fail(ctx, NP_E_INVAL, "io_depth must be in [-1, 4096]");
  if (c->flags & ~(NP_F_CHECK_BOUNDS | NP_F_DIRECT_LOADS | NP_F_LAYER_LAUNCHES | NP_F_NO_TENSOR_CORES | NP_F_MAPPED_STAGING | NP_F_ROW_CHAIN | NP_F_CLUSTER_ROWS | NP_F_TCGEN05_BATCH)) return fail(ctx, NP_E_INVAL, "unknown flag bits");
  if (c->host_threads < 0 || c->host_threads > 256) return fail(ctx, NP_E_INVAL, "host_threads out of range");
  if (c->chain_layers < 0) return fail(ctx, NP_E_INVAL, "chain_layers must be >= 0");
  if (c->ring_stages < 0 || c->ring_stages == 1) return fail(ctx, NP_E_INVAL, "ring_stages must be 0 or >= 2");
  if (c->dense_layers < 0 || c->dense_layers > c->n_layers)
    return fail(ctx, NP_E_INVAL, "dense_layers must be in [0, n_layers]");
  if (c->dense_layers > 0 && c->max_batch > 1 && (c->flags & NP_F_NO_TENSOR_CORES))
    return fail(ctx, NP_E_INVAL, "dense_layers > 0 with batches needs the tensor-core kernels");
  if (c->dense_layers > 0 && (c->flags & (NP_F_LAYER_LAUNCHES | NP_F_DIRECT_LOADS)))
    return fail(ctx, NP_E_INVAL, "dense_layers > 0 excludes NP_F_LAYER_LAUNCHES and NP_F_DIRECT_LOADS");
  if (c->record_format != NP_REC_BF16 && c->record_format != NP_REC_INT8)
    return fail(ctx, NP_E_INVAL, "unknown record_format");
  if (c->spec_rows < 0 || c->spec_rows > c->capacity) return fail(ctx, NP_E_INVAL, "spec_rows must be in [0, capacity]");
  if (c->reserved != 0) return fail(ctx, NP_E_INVAL, "reserved must be 0");
  if (c->store_layers < 0 || c->store_layers > c->n_layers)
    return fail(ctx, NP_E_INVAL, "store_layers must be 0 or in [1, n_layers]");
  if (c->record_format == NP_REC_INT8 && c->d_model % 16)
    return fail(ctx, NP_E_INVAL, "8-bit records need d_model % 16 == 0");
  {
    // batches the tensor-core predictor does not take (B <= 4, no tensor cores, or a width
    // outside its K blocks) run the ring kernel, whose shared memory holds the batch's hidden
    // vectors beside at least two stages of W2 rows
    Dims pd = {};
    pd.H = c->d_pred;
    const bool tc = c->max_batch > 4 && !(c->flags & NP_F_NO_TENSOR_CORES) && pred_tc_supported(pd);
    const int b_ring = tc ? 4 : c->max_batch;
    if (b_ring >= 2 && !pred_l2_ring_fits(c->d_pred, b_ring))
      return fail(ctx, NP_E_INVAL, "max_batch=%d with d_pred=%d: the hidden vectors of %d sequences do not fit the "
                  "predictor kernel's shared memory", c->max_batch, c->d_pred, b_ring);
  }
  return NP_OK;
}

size_t record_bytes_of(const np_config& c) {
  return c.record_format == NP_REC_INT8 ? 3ull * c.d_model + 16 : 3ull * c.d_model * 2;
}

struct WsLayout {
  size_t hidden, hsplit, logits, xbuf, zbuf, gu, gu_each, total;
};

WsLayout ws_layout(const np_config& c) {
  WsLayout w;
  size_t off = 0;
  w.hidden = off;
  off = align_up(off + (size_t)c.max_batch * c.d_pred * 4, 256);
  w.hsplit = off;
  off = align_up(off + (size_t)48 * c.d_pred * 2, 256);
  w.logits = off;
  off = align_up(off + (size_t)c.max_batch * c.n_layers * c.d_ffn * 4, 256);
  const size_t vec = align_up((size_t)c.max_batch * c.d_model * 4, 256);
  w.xbuf = off;
  off += 2 * vec;
  w.zbuf = off;
  off += 3 * kZRep * vec;
  // batch MLP: two dot-product accumulators, each followed by its per-sequence sums of squares
  w.gu = off;
  const size_t gu_rows = c.dense_layers > 0 ? c.d_ffn : c.capacity;  // a dense layer has M active rows
  w.gu_each = align_up((gu_rows * 2 * kMaxBatch + kMaxBatch) * 4, 256);
  off += 2 * w.gu_each;
  w.total = off;
  return w;
}

// one list area of the host mirror: [header][layer: counters, ids[C], slots[C]]
size_t host_area_ints(const np_config& c) {
  return kHostHeaderInts + (size_t)c.n_layers * (NP_N_COUNTERS + 2 * (size_t)c.capacity);
}
// two areas: the incoming rows of np_delta, then the speculative rows of np_speculate
size_t host_lists_ints(const np_config& c) { return 2 * host_area_ints(c); }

cudaStream_t as_stream(void* s) { return static_cast<cudaStream_t>(s); }

int check_device_status(np_ctx* ctx, cudaStream_t s) {
  int32_t st[4];
  NP_CUDA(ctx, cudaMemcpyAsync(st, ctx->t.status, sizeof st, cudaMemcpyDeviceToHost, s));
  NP_CUDA(ctx, cudaStreamSynchronize(s));
  if (st[0]) return fail(ctx, NP_E_DEVICE, "kernel bounds check tripped (status bits 0x%x)", st[0]);
  return NP_OK;
}

}  // namespace

extern "C" {

int np_version(void) { return NP_VERSION; }

const char* np_last_error(const np_ctx* ctx) { return ctx ? ctx->err.c_str() : g_last_error.c_str(); }

int np_query_sizes(const np_config* cfg, np_sizes* out) {
  if (!out) return fail(nullptr, NP_E_INVAL, "out is NULL");
  int rc = check_config(cfg, nullptr);
  if (rc) return rc;
  const np_config& c = *cfg;
  const uint64_t rec = record_bytes_of(c);
  out->record_bytes = rec;
  out->w1_bytes = 2ull * c.d_pred * c.d_model;
  out->w2_bytes = 2ull * c.n_layers * c.d_ffn * c.d_pred;
  out->backing_bytes = rec * (c.store_layers > 0 ? c.store_layers : c.n_layers) * c.d_ffn;
  out->row_buffer_bytes = 2ull * (c.n_layers - c.dense_layers) * c.capacity * c.d_model;
  out->dense_bytes = (uint64_t)c.dense_layers * c.d_ffn * 3 * c.d_model * 2;  // bf16 whatever the store holds
  out->staging_bytes = rec * c.staging_rows;
  out->workspace_bytes = ws_layout(c).total;
  out->host_lists_bytes = host_lists_ints(c) * 4;
  out->logits_bytes = 4ull * c.max_batch * c.n_layers * c.d_ffn;
  out->bitmap_bytes = 4ull * c.n_layers * (c.d_ffn / 32);
  return NP_OK;
}

int np_plan_dense_prefix(const np_config* cfg, uint64_t budget_bytes, uint64_t fixed_bytes, int32_t* d_out) {
  if (!d_out) return fail(nullptr, NP_E_INVAL, "d_out is NULL");
  if (!cfg) return fail(nullptr, NP_E_INVAL, "config is NULL");
  np_config c = *cfg;
  c.dense_layers = 0;  // the field is the answer, not an input
  int rc = check_config(&c, nullptr);
  if (rc) return rc;
  const uint64_t rec = 3ull * c.d_model * 2;  // device-resident rows are bf16 whatever the store holds
  const uint64_t dense = (uint64_t)c.d_ffn * rec, sparse = (uint64_t)c.capacity * rec;
  *d_out = -1;
  for (int d = 0; d <= c.n_layers; ++d) {
    const uint64_t need = (uint64_t)d * dense + (uint64_t)(c.n_layers - d) * sparse;
    if (need <= budget_bytes && fixed_bytes <= budget_bytes - need) *d_out = d;
  }
  return NP_OK;
}

int np_destroy(np_ctx* ctx) {
  if (!ctx) return NP_OK;
  cudaDeviceSynchronize();
  ctx->reader.close();  // nothing may be in flight when the pool and the buffers go
  delete ctx->pool;
  if (ctx->slab) cudaFree(ctx->slab);
  if (ctx->ev_delta) cudaEventDestroy(ctx->ev_delta);
  if (ctx->ev_spec) cudaEventDestroy(ctx->ev_spec);
  for (auto e : ctx->ev_installed)
    if (e) cudaEventDestroy(e);
  for (auto e : ctx->ev_half)
    if (e) cudaEventDestroy(e);
  for (auto e : ctx->ev_copied)
    if (e) cudaEventDestroy(e);
  for (int i = 0; i < 2; ++i) {
    if (ctx->ev_join[i]) cudaEventDestroy(ctx->ev_join[i]);
    if (ctx->aux[i]) cudaStreamDestroy(ctx->aux[i]);
  }
  if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
  for (auto e : ctx->ev_t)
    if (e) cudaEventDestroy(e);
  for (auto e : ctx->ev_c)
    if (e) cudaEventDestroy(e);
  delete ctx;
  return NP_OK;
}

int np_init(np_ctx** out, const np_config* cfg, const np_buffers* b) {
  if (!out) return fail(nullptr, NP_E_INVAL, "out is NULL");
  *out = nullptr;
  int rc = check_config(cfg, nullptr);
  if (rc) return rc;
  if (!b) return fail(nullptr, NP_E_INVAL, "buffers is NULL");
  const bool mapped_staging = (cfg->flags & NP_F_MAPPED_STAGING) &&
                              (cfg->transfer_mode == NP_XFER_HOST_GATHER || cfg->transfer_mode == NP_XFER_FILE);
  const bool need_staging = cfg->transfer_mode != NP_XFER_ZERO_COPY && !mapped_staging;
  const bool any_sparse = cfg->dense_layers < cfg->n_layers;
  const bool from_file = cfg->transfer_mode == NP_XFER_FILE;
  if (!b->w1 || !b->w2 || (!b->backing && !from_file) || !b->workspace || !b->host_lists ||
      (any_sparse && (!b->gate_buf || !b->up_buf || !b->downT_buf)) || (need_staging && !b->staging) ||
      ((cfg->transfer_mode == NP_XFER_HOST_GATHER || from_file) && !b->host_staging) ||
      (cfg->dense_layers > 0 && !b->dense_buf))
    return fail(nullptr, NP_E_INVAL, "a required buffer pointer is NULL");
  if (from_file) {
    struct stat st;
    if (b->backing_fd < 0 || fstat(b->backing_fd, &st) != 0)
      return fail(nullptr, NP_E_INVAL, "backing_fd is not an open file");
    const uint64_t need = (uint64_t)(cfg->store_layers > 0 ? cfg->store_layers : cfg->n_layers) * cfg->d_ffn * record_bytes_of(*cfg);
    if (S_ISREG(st.st_mode) && (uint64_t)st.st_size < need)
      return fail(nullptr, NP_E_INVAL, "the store file holds %llu bytes, the configuration needs %llu",
                  (unsigned long long)st.st_size, (unsigned long long)need);
  }
  const void* aligned16[] = {b->w1, b->w2, b->backing, b->gate_buf, b->up_buf, b->downT_buf, b->staging,
                             b->host_staging, b->dense_buf};
  for (const void* p : aligned16)
    if ((uintptr_t)p % 16) return fail(nullptr, NP_E_INVAL, "weight, row and staging buffers must be 16-byte aligned");
  if ((uintptr_t)b->workspace % 256) return fail(nullptr, NP_E_INVAL, "workspace must be 256-byte aligned");
  if ((uintptr_t)b->host_lists % 16) return fail(nullptr, NP_E_INVAL, "host_lists must be 16-byte aligned");

  np_ctx* ctx = new (std::nothrow) np_ctx();
  if (!ctx) return fail(nullptr, NP_E_NOMEM, "out of host memory");
  ctx->cfg = *cfg;
  ctx->bufs = *b;
  Dims& d = ctx->d;
  d.L = cfg->n_layers;
  d.D = cfg->d_model;
  d.M = cfg->d_ffn;
  d.H = cfg->d_pred;
  d.k = cfg->top_k;
  d.C = cfg->capacity;
  d.W = cfg->d_ffn / 32;
  d.Bmax = cfg->max_batch;
  d.ring_stages = cfg->ring_stages;
  d.Lp = cfg->store_layers > 0 ? cfg->store_layers : cfg->n_layers;
  d.rec_bytes = record_bytes_of(*cfg);
  d.rec_int8 = cfg->record_format == NP_REC_INT8;
  d.dense = cfg->dense_layers;

#define NP_INIT_CUDA(call)                                                                   \
  do {                                                                                       \
    cudaError_t e__ = (call);                                                                \
    if (e__ != cudaSuccess) {                                                                \
      int rc__ = fail(nullptr, e__ == cudaErrorMemoryAllocation ? NP_E_NOMEM : NP_E_CUDA,    \
                      "%s failed: %s", #call, cudaGetErrorString(e__));                      \
      np_destroy(ctx);                                                                       \
      return rc__;                                                                           \
    }                                                                                        \
  } while (0)

  NP_INIT_CUDA(cudaGetDevice(&ctx->device));
  NP_INIT_CUDA(cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device));

  // pinned host areas must be reachable from the device
  void* dev_alias = nullptr;
  if (cudaHostGetDevicePointer(&dev_alias, b->host_lists, 0) != cudaSuccess) {
    cudaGetLastError();
    np_destroy(ctx);
    return fail(nullptr, NP_E_INVAL, "host_lists is not pinned, device-mapped host memory");
  }
  ctx->host_lists = static_cast<int32_t*>(b->host_lists);
  ctx->host_lists_dev = static_cast<int32_t*>(dev_alias);
  if (mapped_staging) {
    if (cudaHostGetDevicePointer(&dev_alias, b->host_staging, 0) != cudaSuccess) {
      cudaGetLastError();
      np_destroy(ctx);
      return fail(nullptr, NP_E_INVAL, "host_staging is not pinned, device-mapped host memory (NP_F_MAPPED_STAGING)");
    }
    ctx->hstage_dev = static_cast<char*>(dev_alias);
  }
  if (!from_file) {
    if (cudaHostGetDevicePointer(&dev_alias, const_cast<void*>(b->backing), 0) != cudaSuccess) {
      cudaGetLastError();
      np_destroy(ctx);
      return fail(nullptr, NP_E_INVAL, "backing store is not pinned, device-mapped host memory");
    }
    ctx->backing_dev = static_cast<const char*>(dev_alias);
  }

  // library-owned slab: residency tables, lists, scratch
  const size_t LM = (size_t)d.L * d.M, LC = (size_t)d.L * d.C, LW = (size_t)d.L * d.W;
  size_t off = 0;
  auto take = [&](size_t ints) {
    size_t o = off;
    off = align_up(off + ints * 4, 256);
    return o;
  };
  const size_t o_res = take(LW), o_slot = take(LM), o_owner = take(LC), o_stamp = take(LM);
  const size_t o_did = take(LC), o_dsl = take(LC), o_eid = take(LC), o_aid = take(LC), o_asl = take(LC);
  const size_t o_ovf = take(LM), o_cnt = take((size_t)d.L * NP_N_COUNTERS), o_free = take(LC);
  const size_t o_cid = take(LC), o_ckey = take(LC), o_pred = take(LW), o_stat = take(4), o_bar = take(4);
  const size_t o_ident = take(d.dense > 0 ? (size_t)d.M : 1);
  const size_t o_spid = take(LC), o_spsl = take(LC), o_spcnt = take((size_t)d.L * NP_N_COUNTERS), o_spcand = take(LW);
  const size_t o_sfix = take(2 * chain_slices::zfix_words(d)), o_sbar = take(chain_slices::bar_words()), o_sxch = take(2 * chain_slices::xch_words(d, ctx->sm_count));
  const size_t o_rz = take(chain_rows::z_floats(d)), o_rcnt = take(4);
  const size_t o_l1p = take(cfg->max_batch > 4 ? (size_t)kPredL1Parts * 16 * d.H : 1);
  const size_t o_xt = take(cfg->max_batch >= kTcMinBatch ? mlp_tc_xterms_bytes(d) / 4 : 1);
  NP_INIT_CUDA(cudaMalloc(&ctx->slab, off));
  char* base = static_cast<char*>(ctx->slab);
  Tables& t = ctx->t;
  t.resident = reinterpret_cast<uint32_t*>(base + o_res);
  t.slot_map = reinterpret_cast<int32_t*>(base + o_slot);
  t.owner = reinterpret_cast<int32_t*>(base + o_owner);
  t.stamp = reinterpret_cast<int32_t*>(base + o_stamp);
  t.delta_ids = reinterpret_cast<int32_t*>(base + o_did);
  t.delta_slots = reinterpret_cast<int32_t*>(base + o_dsl);
  t.evict_ids = reinterpret_cast<int32_t*>(base + o_eid);
  t.active_ids = reinterpret_cast<int32_t*>(base + o_aid);
  t.active_slots = reinterpret_cast<int32_t*>(base + o_asl);
  t.overflow_ids = reinterpret_cast<int32_t*>(base + o_ovf);
  t.counters = reinterpret_cast<int32_t*>(base + o_cnt);
  t.free_slots = reinterpret_cast<int32_t*>(base + o_free);
  t.cand_ids = reinterpret_cast<int32_t*>(base + o_cid);
  t.cand_keys = reinterpret_cast<uint32_t*>(base + o_ckey);
  t.pred = reinterpret_cast<uint32_t*>(base + o_pred);
  t.status = reinterpret_cast<int32_t*>(base + o_stat);
  t.grid_bar = reinterpret_cast<unsigned int*>(base + o_bar);
  t.identity = reinterpret_cast<int32_t*>(base + o_ident);
  t.spec_ids = reinterpret_cast<int32_t*>(base + o_spid);
  t.spec_slots = reinterpret_cast<int32_t*>(base + o_spsl);
  t.spec_counters = reinterpret_cast<int32_t*>(base + o_spcnt);
  t.spec_cand = reinterpret_cast<uint32_t*>(base + o_spcand);
  ctx->slices.zfix = reinterpret_cast<unsigned long long*>(base + o_sfix);
  ctx->slices.bars = reinterpret_cast<unsigned int*>(base + o_sbar);
  ctx->slices.xch = reinterpret_cast<unsigned long long*>(base + o_sxch);
  ctx->slices.seq_base = ctx->slices.bar_base = 0;
  NP_INIT_CUDA(cudaMemset(ctx->slices.zfix, 0, chain_slices::zfix_words(ctx->d) * 8));
  NP_INIT_CUDA(cudaMemset(ctx->slices.bars, 0, chain_slices::bar_words() * 4));
  NP_INIT_CUDA(cudaMemset(ctx->slices.xch, 0, chain_slices::xch_words(ctx->d, ctx->sm_count) * 8));
  ctx->use_slices = !(cfg->flags & NP_F_ROW_CHAIN) && chain_slices::supported(d, ctx->sm_count);
  ctx->xterms = base + o_xt;
  ctx->rows.z4 = reinterpret_cast<float*>(base + o_rz);
  ctx->rows.cnt = reinterpret_cast<unsigned int*>(base + o_rcnt);
  ctx->rows.cnt_base = ctx->rows.seq = 0;
  NP_INIT_CUDA(cudaMemset(ctx->rows.z4, 0, chain_rows::z_floats(d) * 4));
  NP_INIT_CUDA(cudaMemset(ctx->rows.cnt, 0, 4 * 4));
  ctx->use_rows = (cfg->flags & NP_F_CLUSTER_ROWS) && !(cfg->flags & NP_F_ROW_CHAIN) && d.dense < d.L && chain_rows::prepare(d, ctx->sm_count, &ctx->rows);

  const WsLayout wl = ws_layout(*cfg);
  char* wsb = static_cast<char*>(b->workspace);
  const size_t vec = align_up((size_t)d.Bmax * d.D * 4, 256);
  ctx->ws.hidden = reinterpret_cast<float*>(wsb + wl.hidden);
  ctx->ws.hsplit = wsb + wl.hsplit;
  ctx->ws.logits = reinterpret_cast<float*>(wsb + wl.logits);
  for (int i = 0; i < 2; ++i) ctx->ws.xbuf[i] = reinterpret_cast<float*>(wsb + wl.xbuf + i * vec);
  for (int i = 0; i < 3; ++i) ctx->ws.zbuf[i] = reinterpret_cast<float*>(wsb + wl.zbuf + i * kZRep * vec);
  for (int i = 0; i < 2; ++i) {
    ctx->ws.gu[i] = reinterpret_cast<float*>(wsb + wl.gu + i * wl.gu_each);
    ctx->ws.ssq[i] = ctx->ws.gu[i] + (size_t)(cfg->dense_layers > 0 ? cfg->d_ffn : cfg->capacity) * 2 * kMaxBatch;
  }
  ctx->gu_bytes = 2 * wl.gu_each;

  NP_INIT_CUDA(cudaEventCreateWithFlags(&ctx->ev_delta, cudaEventDisableTiming));
  NP_INIT_CUDA(cudaEventCreateWithFlags(&ctx->ev_spec, cudaEventDisableTiming));
  ctx->ev_installed.assign(d.L, nullptr);
  ctx->install_pending.assign(d.L, 0);
  for (int l = 0; l < d.L; ++l)
    NP_INIT_CUDA(cudaEventCreateWithFlags(&ctx->ev_installed[l], cudaEventDisableTiming));
  for (auto& e : ctx->ev_half) NP_INIT_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  for (auto& e : ctx->ev_copied) NP_INIT_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  for (int i = 0; i < 2; ++i) {
    NP_INIT_CUDA(cudaStreamCreateWithFlags(&ctx->aux[i], cudaStreamNonBlocking));
    NP_INIT_CUDA(cudaEventCreateWithFlags(&ctx->ev_join[i], cudaEventDisableTiming));
  }
  NP_INIT_CUDA(cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming));
  for (auto& e : ctx->ev_t) NP_INIT_CUDA(cudaEventCreate(&e));
  for (auto& e : ctx->ev_c) NP_INIT_CUDA(cudaEventCreate(&e));

  if (cfg->transfer_mode == NP_XFER_HOST_GATHER || from_file) {
    int n = cfg->host_threads;
    if (n == 0) {
      // the packing is what bounds the transfer (steps/s kept rising up to 14 of 16 cores); two
      // cores stay with the caller's thread and the driver
      const unsigned hc = std::thread::hardware_concurrency();
      n = (int)std::max(1u, std::min(16u, hc > 8 ? hc - 2 : hc));
    }
    ctx->pool = new (std::nothrow) Pool(n - 1);  // the caller's thread works too
  }
  if (from_file) {
    Pool* pool = ctx->pool;
    std::string note;
    ctx->reader.open(b->backing_fd, cfg->io_depth,
                     [pool](int count, const std::function<void(int)>& fn) {
                       if (pool) pool->parallel_for(count, fn);
                       else for (int i = 0; i < count; ++i) fn(i);
                     },
                     &note);
    if (!note.empty()) ctx->err = note;  // readable through np_last_error: why the ring is not in use
  }

  // tensor-core predictor for batches: tensor maps over W2 and the split hidden terms
  ctx->mlp_tc = cfg->max_batch >= kTcMinBatch && !(cfg->flags & (NP_F_NO_TENSOR_CORES | NP_F_DIRECT_LOADS)) &&
                mlp_tc_supported(d, ctx->sm_count);
  if (cfg->max_batch > 4 && !(cfg->flags & NP_F_NO_TENSOR_CORES))
    pred_tc_prepare(d, b->w1, b->w2, ctx->ws.hsplit, reinterpret_cast<float*>(static_cast<char*>(ctx->slab) + o_l1p), ctx->sm_count, &ctx->tc);
  {
    // batches the tensor-core predictor does not take go through the ring kernel, whose shared
    // memory holds the batch's hidden vectors beside at least two stages of W2 rows
    const int b_ring = ctx->tc.ready ? std::min(cfg->max_batch, 4) : cfg->max_batch;
    if (b_ring >= 2 && !pred_l2_ring_fits(d.H, b_ring)) {
      np_destroy(ctx);
      return fail(nullptr, NP_E_INVAL,
                  "max_batch=%d with d_pred=%d: the hidden vectors of %d sequences do not fit the predictor kernel's "
                  "shared memory%s", cfg->max_batch, d.H, b_ring,
                  (cfg->flags & NP_F_NO_TENSOR_CORES) ? " (NP_F_NO_TENSOR_CORES is set)" : "");
    }
  }
  memset(ctx->host_lists, 0, host_lists_ints(*cfg) * 4);
  if (d.dense > 0 && cfg->max_batch > 1 && !ctx->mlp_tc) {
    np_destroy(ctx);
    return fail(nullptr, NP_E_INVAL, "dense_layers > 0 with batches: this width is outside the tensor-core batch kernels");
  }
  if (d.dense > 0) {
    Dims dd = d;
    dd.k = dd.C = d.M;
    if ((!dense_chain::supported(d, ctx->sm_count) && !chain_alu::supported(dd, ctx->sm_count)) || (d.dense < d.L && !chain_slices::supported(d, ctx->sm_count) && !chain_alu::supported(d, ctx->sm_count))) {
      np_destroy(ctx);
      return fail(nullptr, NP_E_INVAL, "dense_layers > 0: this shape is outside what the resident MLP kernels cover");
    }
    // the dense layers' records move to the device once; their active list is 0 .. M-1
    std::vector<int32_t> ident(d.M);
    for (int i = 0; i < d.M; ++i) ident[i] = i;
    NP_INIT_CUDA(cudaMemcpy(t.identity, ident.data(), (size_t)d.M * 4, cudaMemcpyHostToDevice));
    const size_t dense_layer_bytes = (size_t)d.M * 3 * d.D * 2;
    if (d.rec_int8) {
      // 8-bit store: the same rounding as the install path, once, straight from the pinned store
      for (int l = 0; l < d.dense; ++l)
        NP_INIT_CUDA(launch_dequant_dense_layer(d, ctx->backing_dev + (size_t)(l % d.Lp) * d.M * d.rec_bytes, t.identity,
                                                static_cast<char*>(b->dense_buf) + l * dense_layer_bytes, t.status,
                                                nullptr, ctx->sm_count));
    } else if (from_file) {
      // through the pinned staging, a staging buffer's worth at a time
      const size_t total = (size_t)d.dense * dense_layer_bytes, step = (size_t)cfg->staging_rows * d.rec_bytes;
      const size_t file_bytes = (size_t)d.Lp * dense_layer_bytes;  // the file holds Lp layers; later layers wrap around
      size_t off = 0;
      while (off < total) {
        const size_t foff = off % file_bytes;
        const size_t n = std::min(std::min(step, total - off), file_bytes - foff);
        if (!ctx->reader.submit(b->host_staging, n, foff, 0) || !ctx->reader.wait_group(0)) {
          const int e = ctx->reader.last_error();
          np_destroy(ctx);
          return fail(nullptr, NP_E_IO, "reading the dense layers from the store file failed: %s", strerror(e));
        }
        NP_INIT_CUDA(cudaMemcpy(static_cast<char*>(b->dense_buf) + off, b->host_staging, n, cudaMemcpyHostToDevice));
        off += n;
      }
    } else {
      for (int l = 0; l < d.dense; ++l)
        NP_INIT_CUDA(cudaMemcpy(static_cast<char*>(b->dense_buf) + l * dense_layer_bytes,
                                static_cast<const char*>(b->backing) + (size_t)(l % d.Lp) * dense_layer_bytes,
                                dense_layer_bytes, cudaMemcpyHostToDevice));
    }
  }
  NP_INIT_CUDA(launch_tables_reset(d, t, nullptr));
  NP_INIT_CUDA(cudaDeviceSynchronize());
#undef NP_INIT_CUDA

  *out = ctx;
  return NP_OK;
}

int np_reset(np_ctx* ctx, void* stream) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  NP_LAUNCH(ctx, launch_tables_reset(ctx->d, ctx->t, as_stream(stream)));
  // a launch that gave up may have left the sliced kernel's counters and stamps anywhere
  NP_CUDA(ctx, cudaMemsetAsync(ctx->slices.zfix, 0, chain_slices::zfix_words(ctx->d) * 8, as_stream(stream)));
  NP_CUDA(ctx, cudaMemsetAsync(ctx->slices.bars, 0, chain_slices::bar_words() * 4, as_stream(stream)));
  NP_CUDA(ctx, cudaMemsetAsync(ctx->slices.xch, 0, chain_slices::xch_words(ctx->d, ctx->sm_count) * 8, as_stream(stream)));
  ctx->slices.seq_base = ctx->slices.bar_base = 0;
  NP_CUDA(ctx, cudaMemsetAsync(ctx->rows.z4, 0, chain_rows::z_floats(ctx->d) * 4, as_stream(stream)));
  NP_CUDA(ctx, cudaMemsetAsync(ctx->rows.cnt, 0, 4 * 4, as_stream(stream)));
  ctx->rows.cnt_base = ctx->rows.seq = 0;
  ctx->have_delta = ctx->have_pred = ctx->have_step = ctx->have_spec = false;
  std::fill(ctx->install_pending.begin(), ctx->install_pending.end(), 0);
  ctx->step = 0;
  return NP_OK;
}

int np_predict(np_ctx* ctx, const void* x_bf16, int32_t B, float* logits_out, uint32_t* bitmap_out,
               void* stream) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  if (!x_bf16) return fail(ctx, NP_E_INVAL, "x is NULL");
  if (B < 1 || B > ctx->d.Bmax) return fail(ctx, NP_E_INVAL, "B=%d outside [1, max_batch=%d]", B, ctx->d.Bmax);
  if ((uintptr_t)x_bf16 % 16) return fail(ctx, NP_E_INVAL, "x must be 16-byte aligned");
  cudaStream_t s = as_stream(stream);
  const Dims& d = ctx->d;
  // batches: both layers on the tensor cores where the shapes allow (layer 1 leaves partial sums that layer 2's
  // split kernel adds up)
  const bool l1_tc = B > 4 && ctx->tc.ready && ctx->tc.l1_ready && d.dense == 0;
  if (l1_tc)
    NP_LAUNCH(ctx, launch_pred_l1_tc(d, ctx->tc, x_bf16, B, ctx->t.status, s));
  else
    NP_LAUNCH(ctx, launch_pred_l1(d, ctx->bufs.w1, x_bf16, B, ctx->ws.hidden, s));
  // Dense layers are not scored: the sparse layers are a contiguous suffix of W2, of the logits
  // and of the bitmap (a dense prefix implies B = 1, so the per-sequence stride does not matter).
  // With several sequences the per-sequence stride of the logits keeps all L layers, so every
  // layer is scored and the dense layers' bitmap rows are cleared afterwards.
  Dims ds = d;
  const int skip_layers = B == 1 ? d.dense : 0;
  ds.L = d.L - skip_layers;
  const size_t skip_rows = (size_t)skip_layers * d.M;
  float* logits = ctx->ws.logits + skip_rows;
  if (ds.L > 0) {
    if (B > 4 && ctx->tc.ready) {
      ctx->launches += 1;  // split kernel + GEMM kernel
      NP_LAUNCH(ctx, launch_pred_l2_tc(d, ctx->tc, ctx->ws.hidden, B, ctx->ws.logits, ctx->t.status, s, ctx->sm_count,
                                       l1_tc ? ctx->tc.l1_parts : 0));
    } else {
      NP_LAUNCH(ctx, launch_pred_l2(ds, static_cast<const char*>(ctx->bufs.w2) + skip_rows * d.H * 2, ctx->ws.hidden,
                                  B, logits, ctx->t.status, s, ctx->sm_count));
    }
    NP_LAUNCH(ctx, launch_topk(ds, logits, B, ctx->t.pred + (size_t)skip_layers * d.W, s));
  }
  if (d.dense > 0) NP_CUDA(ctx, cudaMemsetAsync(ctx->t.pred, 0, (size_t)d.dense * d.W * 4, s));
  const size_t nlog = (size_t)B * ds.L * d.M * 4, nbm = (size_t)d.L * d.W * 4;
  if (logits_out && nlog)
    NP_CUDA(ctx, cudaMemcpyAsync(logits_out + skip_rows, logits, nlog, cudaMemcpyDeviceToDevice, s));
  if (bitmap_out) NP_CUDA(ctx, cudaMemcpyAsync(bitmap_out, ctx->t.pred, nbm, cudaMemcpyDeviceToDevice, s));
  ctx->have_pred = true;
  return NP_OK;
}

int np_topk(np_ctx* ctx, const float* logits, int32_t B, uint32_t* bitmap_out, void* stream) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  if (!logits || !bitmap_out) return fail(ctx, NP_E_INVAL, "logits or bitmap_out is NULL");
  if (B < 1 || B > ctx->d.Bmax) return fail(ctx, NP_E_INVAL, "B=%d outside [1, max_batch=%d]", B, ctx->d.Bmax);
  const Dims& d = ctx->d;
  Dims ds = d;
  const int skip_layers = B == 1 ? d.dense : 0;  // dense layers select nothing: their rows of the bitmap are zero
  ds.L = d.L - skip_layers;
  if (ds.L > 0)
    NP_LAUNCH(ctx, launch_topk(ds, logits + (size_t)skip_layers * d.M, B, bitmap_out + (size_t)skip_layers * d.W,
                               as_stream(stream)));
  if (d.dense > 0) NP_CUDA(ctx, cudaMemsetAsync(bitmap_out, 0, (size_t)d.dense * d.W * 4, as_stream(stream)));
  return NP_OK;
}

int np_centroid_select(np_ctx* ctx, const float* logits, int32_t B, int32_t K, const uint32_t* bank,
                       int32_t* ids_out, uint32_t* bitmap_out, void* stream) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  if (!logits || !bank || !bitmap_out) return fail(ctx, NP_E_INVAL, "logits, bank or bitmap_out is NULL");
  if (B < 1 || B > ctx->d.Bmax) return fail(ctx, NP_E_INVAL, "B=%d outside [1, max_batch=%d]", B, ctx->d.Bmax);
  if (K < 1) return fail(ctx, NP_E_INVAL, "K=%d must be positive", K);
  NP_LAUNCH(ctx, launch_centroid_select(ctx->d, logits, B, K, bank, ids_out, bitmap_out, as_stream(stream)));
  if (ctx->d.dense > 0)  // dense layers select nothing
    NP_CUDA(ctx, cudaMemsetAsync(bitmap_out, 0, (size_t)ctx->d.dense * ctx->d.W * 4, as_stream(stream)));
  return NP_OK;
}

int np_delta(np_ctx* ctx, const uint32_t* pred_bitmap, void* stream) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  if (!pred_bitmap) {
    if (!ctx->have_pred) return fail(ctx, NP_E_STATE, "np_delta(NULL) needs a prior np_predict");
    pred_bitmap = ctx->t.pred;
  }
  cudaStream_t s = as_stream(stream);
  if (ctx->d.dense > 0 && pred_bitmap != ctx->t.pred) {
    // a caller's bitmap may name rows of dense layers; those layers select nothing
    const size_t skip = (size_t)ctx->d.dense * ctx->d.W;
    NP_CUDA(ctx, cudaMemsetAsync(ctx->t.pred, 0, skip * 4, s));
    NP_CUDA(ctx, cudaMemcpyAsync(ctx->t.pred + skip, pred_bitmap + skip, ((size_t)ctx->d.L * ctx->d.W - skip) * 4,
                                 cudaMemcpyDeviceToDevice, s));
    pred_bitmap = ctx->t.pred;
  }
  // the previous step's installs must have landed before tables and slots are reused
  for (int l = 0; l < ctx->d.L; ++l) {
    if (ctx->install_pending[l]) {
      NP_CUDA(ctx, cudaStreamWaitEvent(s, ctx->ev_installed[l], 0));
      ctx->install_pending[l] = 0;
    }
  }
  NP_LAUNCH(ctx, launch_delta(ctx->d, ctx->t, pred_bitmap, ctx->cfg.evict_policy, ctx->step, ctx->host_lists_dev,
                            ctx->cfg.flags & NP_F_CHECK_BOUNDS, s));
  NP_CUDA(ctx, cudaEventRecord(ctx->ev_delta, s));
  ctx->step += 1;
  ctx->have_delta = true;
  ctx->have_spec = false;
  return NP_OK;
}

// NP_XFER_FILE: per chunk of a layer's incoming rows, the ranges of adjacent records are read
// from the store file into a part of the pinned staging, copied to the device and scattered.
// The reads of the next chunk are queued before the previous chunk is waited for, so the
// device queue does not drain at chunk boundaries.
static int install_from_file(np_ctx* ctx, int layer_begin, int layer_end, cudaStream_t cs, int* warn) {
  const Dims& d = ctx->d;
  const size_t rec = d.rec_bytes, row_bytes = (size_t)d.D * 2;
  const int check = ctx->cfg.flags & NP_F_CHECK_BOUNDS;
  char* staging = static_cast<char*>(ctx->bufs.staging);
  char* hstage = static_cast<char*>(ctx->bufs.host_staging);
  const size_t per_layer = NP_N_COUNTERS + 2 * (size_t)d.C;
  const int parts = std::min(kStageParts, std::max(2, ctx->cfg.staging_rows / std::max(1, d.k / 4 + 1)));
  const int part_rows = ctx->cfg.staging_rows / parts;
  struct Chunk {
    int l, first, rows, h;
    bool last;
  };
  std::deque<Chunk> queued;  // reads queued, copy not yet issued
  auto finish = [&](const Chunk& c) -> int {
    if (!ctx->reader.wait_group(c.h)) {
      const int e = ctx->reader.last_error();
      ctx->reader.drain();
      return fail(ctx, NP_E_IO, "layer %d: reading the store file failed: %s", c.l, strerror(e));
    }
    char* hbuf = hstage + (size_t)c.h * part_rows * rec;
    char* dbuf = staging + (size_t)c.h * part_rows * rec;
    if (ctx->hstage_dev) {
      // mapped staging (the paper's way): the scatter kernel reads the staged records over the bus itself
      dbuf = ctx->hstage_dev + (size_t)c.h * part_rows * rec;
    } else {
      NP_CUDA(ctx, cudaMemcpyAsync(dbuf, hbuf, (size_t)c.rows * rec, cudaMemcpyHostToDevice, cs));
      NP_CUDA(ctx, cudaEventRecord(ctx->ev_copied[c.h], cs));
      NP_CUDA(ctx, cudaStreamWaitEvent(ctx->aux[0], ctx->ev_copied[c.h], 0));
    }
    NP_LAUNCH(ctx, launch_scatter(d, dbuf, false, nullptr, ctx->t.delta_slots + (size_t)c.l * d.C,
                                ctx->t.counters + (size_t)c.l * NP_N_COUNTERS + NP_CNT_DELTA, c.first, c.rows,
                                static_cast<char*>(ctx->bufs.gate_buf) + (size_t)(c.l - d.dense) * d.C * row_bytes,
                                static_cast<char*>(ctx->bufs.up_buf) + (size_t)(c.l - d.dense) * d.C * row_bytes,
                                static_cast<char*>(ctx->bufs.downT_buf) + (size_t)(c.l - d.dense) * d.C * row_bytes,
                                ctx->t.status, check, ctx->aux[0], ctx->sm_count));
    NP_CUDA(ctx, cudaEventRecord(ctx->ev_half[c.h], ctx->aux[0]));  // both copies of the part are free again
    ctx->half_pending[c.h] = true;
    if (c.last) {
      NP_CUDA(ctx, cudaEventRecord(ctx->ev_installed[c.l], ctx->aux[0]));
      ctx->install_pending[c.l] = 1;
    }
    return NP_OK;
  };
  auto give_up = [&](int rc) {
    ctx->reader.drain();
    return rc;
  };
  for (int l = layer_begin; l < layer_end; ++l) {
    const int32_t* cnt = ctx->host_lists + kHostHeaderInts + (size_t)l * per_layer;
    const int32_t* ids = cnt + NP_N_COUNTERS;
    const int n = cnt[NP_CNT_DELTA];
    if (n < 0 || n > d.C) return give_up(fail(ctx, NP_E_DEVICE, "layer %d: delta count %d outside [0, %d]", l, n, d.C));
    if (cnt[NP_CNT_OVERFLOW] > 0) *warn = NP_W_OVERFLOW;
    if (n > part_rows && *warn == NP_OK) *warn = NP_W_CHUNKED;
    if (n == 0) {  // nothing to read: the layer is installed once the earlier chunks are
      while (!queued.empty()) {
        const int rc = finish(queued.front());
        queued.pop_front();
        if (rc < 0) return give_up(rc);
      }
      NP_CUDA(ctx, cudaEventRecord(ctx->ev_installed[l], ctx->aux[0]));
      ctx->install_pending[l] = 1;
      continue;
    }
    for (int first = 0; first < n; first += part_rows) {
      const int rows = std::min(part_rows, n - first);
      const int h = ctx->next_half % parts;
      ctx->next_half = (h + 1) % parts;
      // a part is taken again only after its earlier chunk has been copied and scattered
      while (!queued.empty() && ((int)queued.size() >= parts - 1 || queued.front().h == h)) {
        const int rc = finish(queued.front());
        queued.pop_front();
        if (rc < 0) return give_up(rc);
      }
      if (ctx->half_pending[h]) {
        NP_CUDA(ctx, cudaEventSynchronize(ctx->ev_half[h]));
        ctx->half_pending[h] = false;
      }
      char* hbuf = hstage + (size_t)h * part_rows * rec;
      // ascending IDs: adjacent IDs are adjacent records of the file -> one range per run
      int r = 0;
      while (r < rows) {
        int len = 1;
        while (r + len < rows && ids[first + r + len] == ids[first + r] + len) ++len;
        const int id = ids[first + r];
        if (id < 0 || id + len > d.M) return give_up(fail(ctx, NP_E_DEVICE, "layer %d: neuron id %d out of range", l, id));
        if (!ctx->reader.submit(hbuf + (size_t)r * rec, (size_t)len * rec, ((uint64_t)(l % d.Lp) * d.M + (uint64_t)id) * rec, h))
          return give_up(fail(ctx, NP_E_IO, "layer %d: queueing a read failed: %s", l, strerror(ctx->reader.last_error())));
        r += len;
      }
      queued.push_back(Chunk{l, first, rows, h, first + rows >= n});
      // keep one chunk's reads queued behind the one that is waited for
      while (queued.size() > 1) {
        const int rc = finish(queued.front());
        queued.pop_front();
        if (rc < 0) return give_up(rc);
      }
    }
  }
  while (!queued.empty()) {
    const int rc = finish(queued.front());
    queued.pop_front();
    if (rc < 0) return give_up(rc);
  }
  return NP_OK;
}

// NP_XFER_HOST_GATHER: the pool packs the incoming records into a part of the pinned staging,
// one cudaMemcpyAsync moves the part, scatter kernels place its rows.  The parts are used round
// robin: one is packed while earlier ones are copied and scattered (the scatter kernels can fall
// behind while a resident MLP launch holds the device; spare parts keep the host and the copy
// engine going).  A part takes the rows of up to kGatherLayers consecutive layers: a copy has a
// start-up cost, and a steady-state layer fills only a fraction of a part.
constexpr int kGatherLayers = 2;

static int install_host_gather(np_ctx* ctx, int layer_begin, int layer_end, cudaStream_t cs, int* warn) {
  const Dims& d = ctx->d;
  const size_t rec = d.rec_bytes, row_bytes = (size_t)d.D * 2;
  const int check = ctx->cfg.flags & NP_F_CHECK_BOUNDS;
  const char* store = static_cast<const char*>(ctx->bufs.backing);
  char* staging = static_cast<char*>(ctx->bufs.staging);
  char* hstage = static_cast<char*>(ctx->bufs.host_staging);
  const size_t per_layer = NP_N_COUNTERS + 2 * (size_t)d.C;
  const int parts = std::min(kStageParts, std::max(2, ctx->cfg.staging_rows / std::max(1, d.k / 4 + 1)));
  const int part_rows = ctx->cfg.staging_rows / parts;
  struct Piece {
    int l, first, rows, at;  // rows [first, first + rows) of layer l's list sit at row `at` of the part
    bool last;               // the layer is complete with this piece
  };
  std::vector<Piece> batch;
  int h = -1, used = 0, layers_in = 0, last_l = -1;
  int flushed = 0;  // parts handed to the copy engine by this call
  const int first_small = 1;  // the first part takes one layer: the copy engine starts sooner
  auto open_part = [&]() -> int {
    h = ctx->next_half % parts;
    ctx->next_half = (h + 1) % parts;
    if (ctx->half_pending[h]) {
      NP_CUDA(ctx, cudaEventSynchronize(ctx->ev_half[h]));
      ctx->half_pending[h] = false;
    }
    used = 0;
    layers_in = 0;
    last_l = -1;
    return NP_OK;
  };
  auto flush = [&]() -> int {
    if (batch.empty()) return NP_OK;
    char* hbuf = hstage + (size_t)h * part_rows * rec;
    char* dbuf = staging + (size_t)h * part_rows * rec;
    if (used > 0) {
      bool bad = false;
      const int nthreads = ctx->pool ? ctx->pool->size() + 1 : 1;
      const int jobs = std::min(used, nthreads * 4);
      auto body = [&](int job) {
        const int lo = (int)((long long)used * job / jobs), hi = (int)((long long)used * (job + 1) / jobs);
        size_t pi = 0;
        for (int r = lo; r < hi; ++r) {
          while (r >= batch[pi].at + batch[pi].rows) ++pi;  // pieces are in row order; empty ones are skipped
          const Piece& pc = batch[pi];
          const int32_t* ids = ctx->host_lists + kHostHeaderInts + (size_t)pc.l * per_layer + NP_N_COUNTERS;
          const int id = ids[pc.first + (r - pc.at)];
          if (id < 0 || id >= d.M) {
            bad = true;
            continue;
          }
          copy_record_streaming(hbuf + (size_t)r * rec, store + ((size_t)(pc.l % d.Lp) * d.M + id) * rec, rec);
        }
      };
      if (ctx->pool) ctx->pool->parallel_for(jobs, body);
      else for (int job = 0; job < jobs; ++job) body(job);
      if (bad) return fail(ctx, NP_E_DEVICE, "layer %d: neuron id out of range", batch.front().l);
      // the copies queue back to back on the caller's stream; the scatter kernels follow them
      // on a side stream, so a copy never waits for the previous part's kernels
      if (ctx->hstage_dev) {
        dbuf = ctx->hstage_dev + (size_t)h * part_rows * rec;  // mapped staging: no staging copy
      } else {
        NP_CUDA(ctx, cudaMemcpyAsync(dbuf, hbuf, (size_t)used * rec, cudaMemcpyHostToDevice, cs));
        NP_CUDA(ctx, cudaEventRecord(ctx->ev_copied[h], cs));
        NP_CUDA(ctx, cudaStreamWaitEvent(ctx->aux[0], ctx->ev_copied[h], 0));
      }
    }
    for (const Piece& pc : batch) {
      if (pc.rows > 0)
        NP_LAUNCH(ctx, launch_scatter(d, dbuf + (size_t)pc.at * rec, false, nullptr, ctx->t.delta_slots + (size_t)pc.l * d.C,
                                    ctx->t.counters + (size_t)pc.l * NP_N_COUNTERS + NP_CNT_DELTA, pc.first, pc.rows,
                                    static_cast<char*>(ctx->bufs.gate_buf) + (size_t)(pc.l - d.dense) * d.C * row_bytes,
                                    static_cast<char*>(ctx->bufs.up_buf) + (size_t)(pc.l - d.dense) * d.C * row_bytes,
                                    static_cast<char*>(ctx->bufs.downT_buf) + (size_t)(pc.l - d.dense) * d.C * row_bytes,
                                    ctx->t.status, check, ctx->aux[0], ctx->sm_count));
      if (pc.last) {
        NP_CUDA(ctx, cudaEventRecord(ctx->ev_installed[pc.l], ctx->aux[0]));
        ctx->install_pending[pc.l] = 1;
      }
    }
    if (used > 0) {
      NP_CUDA(ctx, cudaEventRecord(ctx->ev_half[h], ctx->aux[0]));  // both copies of the part are free again
      ctx->half_pending[h] = true;
    }
    batch.clear();
    h = -1;
    ++flushed;
    return NP_OK;
  };
  for (int l = layer_begin; l < layer_end; ++l) {
    const int32_t* cnt = ctx->host_lists + kHostHeaderInts + (size_t)l * per_layer;
    const int n = cnt[NP_CNT_DELTA];
    if (n < 0 || n > d.C) return fail(ctx, NP_E_DEVICE, "layer %d: delta count %d outside [0, %d]", l, n, d.C);
    if (cnt[NP_CNT_OVERFLOW] > 0) *warn = NP_W_OVERFLOW;
    if (n > part_rows && *warn == NP_OK) *warn = NP_W_CHUNKED;
    int first = 0;
    do {
      const int rows = std::min(part_rows, n - first);
      if (h >= 0 && (used + rows > part_rows || (l != last_l && layers_in >= (flushed < first_small ? 1 : kGatherLayers)))) {
        const int rc = flush();
        if (rc < 0) return rc;
      }
      if (h < 0) {
        const int rc = open_part();
        if (rc < 0) return rc;
      }
      if (l != last_l) {
        ++layers_in;
        last_l = l;
      }
      batch.push_back(Piece{l, first, rows, used, first + rows >= n});
      used += rows;
      first += rows;
    } while (first < n);
  }
  return flush();
}

int np_install(np_ctx* ctx, int32_t layer_begin, int32_t layer_end, void* copy_stream) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  const Dims& d = ctx->d;
  if (layer_begin < 0 || layer_end > d.L || layer_begin > layer_end)
    return fail(ctx, NP_E_INVAL, "layer range [%d, %d) outside [0, %d)", layer_begin, layer_end, d.L);
  if (!ctx->have_delta) return fail(ctx, NP_E_STATE, "np_install needs a prior np_delta");
  layer_begin = std::max(layer_begin, d.dense);  // dense layers hold all their rows already
  layer_end = std::max(layer_end, layer_begin);
  cudaStream_t cs = as_stream(copy_stream);
  const int check = ctx->cfg.flags & NP_F_CHECK_BOUNDS;
  const int mode = ctx->cfg.transfer_mode;
  const size_t rec = d.rec_bytes;
  const size_t row_bytes = (size_t)d.D * 2;
  NP_CUDA(ctx, cudaStreamWaitEvent(cs, ctx->ev_delta, 0));
  int warn = NP_OK;
  // Side streams: ordered after everything the caller's copy stream holds so far, and joined
  // back into it at the end, so the caller sees one stream's worth of ordering.
  const bool forked = mode != NP_XFER_MEMCPY_RUNS;
  if (forked) {
    NP_CUDA(ctx, cudaEventRecord(ctx->ev_fork, cs));
    for (int i = 0; i < 2; ++i) NP_CUDA(ctx, cudaStreamWaitEvent(ctx->aux[i], ctx->ev_fork, 0));
  }
  auto join = [&]() -> cudaError_t {
    for (int i = 0; i < 2; ++i) {
      cudaError_t e = cudaEventRecord(ctx->ev_join[i], ctx->aux[i]);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(cs, ctx->ev_join[i], 0);
      if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
  };

  if (mode == NP_XFER_ZERO_COPY) {
    // consecutive layers alternate between the two side streams: one kernel's tail (its last
    // reads are still crossing PCIe) overlaps the next kernel's start
    const int max_rows = d.C;
    for (int l = layer_begin; l < layer_end; ++l) {
      cudaStream_t zs = ctx->aux[l & 1];
      const char* store_l = ctx->backing_dev + (size_t)(l % d.Lp) * d.M * rec;
      NP_LAUNCH(ctx, launch_scatter(d, store_l, true, ctx->t.delta_ids + (size_t)l * d.C,
                                  ctx->t.delta_slots + (size_t)l * d.C,
                                  ctx->t.counters + (size_t)l * NP_N_COUNTERS + NP_CNT_DELTA, 0, max_rows,
                                  static_cast<char*>(ctx->bufs.gate_buf) + (size_t)(l - d.dense) * d.C * row_bytes,
                                  static_cast<char*>(ctx->bufs.up_buf) + (size_t)(l - d.dense) * d.C * row_bytes,
                                  static_cast<char*>(ctx->bufs.downT_buf) + (size_t)(l - d.dense) * d.C * row_bytes,
                                  ctx->t.status, check, zs, ctx->sm_count));
      NP_CUDA(ctx, cudaEventRecord(ctx->ev_installed[l], zs));
      ctx->install_pending[l] = 1;
    }
    NP_CUDA(ctx, join());
    return NP_OK;
  }

  // the host plans the copies: wait until the delta lists are readable
  NP_CUDA(ctx, cudaEventSynchronize(ctx->ev_delta));
  if (mode == NP_XFER_FILE || mode == NP_XFER_HOST_GATHER) {
    const int rc = mode == NP_XFER_FILE ? install_from_file(ctx, layer_begin, layer_end, cs, &warn)
                                        : install_host_gather(ctx, layer_begin, layer_end, cs, &warn);
    if (rc < 0) return rc;
    NP_CUDA(ctx, join());
    return warn;
  }
  const char* store = static_cast<const char*>(ctx->bufs.backing);
  char* staging = static_cast<char*>(ctx->bufs.staging);
  const size_t per_layer = NP_N_COUNTERS + 2 * (size_t)d.C;
  for (int l = layer_begin; l < layer_end; ++l) {
    const int32_t* cnt = ctx->host_lists + kHostHeaderInts + (size_t)l * per_layer;
    const int32_t* ids = cnt + NP_N_COUNTERS;
    const int n = cnt[NP_CNT_DELTA];
    if (n < 0 || n > d.C) return fail(ctx, NP_E_DEVICE, "layer %d: delta count %d outside [0, %d]", l, n, d.C);
    if (cnt[NP_CNT_OVERFLOW] > 0) warn = NP_W_OVERFLOW;
    const char* store_l = store + (size_t)(l % d.Lp) * d.M * rec;
    char* gate_l = static_cast<char*>(ctx->bufs.gate_buf) + (size_t)(l - d.dense) * d.C * row_bytes;
    char* up_l = static_cast<char*>(ctx->bufs.up_buf) + (size_t)(l - d.dense) * d.C * row_bytes;
    char* down_l = static_cast<char*>(ctx->bufs.downT_buf) + (size_t)(l - d.dense) * d.C * row_bytes;
    const int32_t* slots_dev = ctx->t.delta_slots + (size_t)l * d.C;
    const int32_t* count_dev = ctx->t.counters + (size_t)l * NP_N_COUNTERS + NP_CNT_DELTA;

    if (mode == NP_XFER_MEMCPY_RUNS) {
      const int cap = ctx->cfg.staging_rows;
      if (n > cap && warn == NP_OK) warn = NP_W_CHUNKED;
      for (int first = 0; first < n; first += cap) {
        const int rows = std::min(cap, n - first);
        // ascending IDs: adjacent IDs are adjacent records of the store -> one copy per run
        int r = 0;
        while (r < rows) {
          int len = 1;
          while (r + len < rows && ids[first + r + len] == ids[first + r] + len) ++len;
          const int id = ids[first + r];
          if (id < 0 || id + len > d.M) return fail(ctx, NP_E_DEVICE, "layer %d: neuron id %d out of range", l, id);
          NP_CUDA(ctx, cudaMemcpyAsync(staging + (size_t)r * rec, store_l + (size_t)id * rec, (size_t)len * rec,
                                       cudaMemcpyHostToDevice, cs));
          r += len;
        }
        NP_LAUNCH(ctx, launch_scatter(d, staging, false, nullptr, slots_dev, count_dev, first, rows, gate_l, up_l,
                                    down_l, ctx->t.status, check, cs, ctx->sm_count));
      }
    }
    NP_CUDA(ctx, cudaEventRecord(ctx->ev_installed[l], cs));
    ctx->install_pending[l] = 1;
  }
  if (forked) NP_CUDA(ctx, join());
  return warn;
}

// Orders `s` after a layer's install mark; marks that have already completed need no wait.
static cudaError_t wait_install(np_ctx* ctx, int layer, cudaStream_t s) {
  const cudaError_t q = cudaEventQuery(ctx->ev_installed[layer]);
  if (q == cudaSuccess) {
    ctx->install_pending[layer] = 0;  // landed: later calls need not ask again
    return cudaSuccess;
  }
  if (q != cudaErrorNotReady) return q;
  (void)cudaGetLastError();
  return cudaStreamWaitEvent(s, ctx->ev_installed[layer], 0);
}

// gu_sel: which of the two dot-product accumulators this layer uses (the batch kernels clear the
// other one for the next layer); -1 = a single layer outside a chain
static int mlp_layer(np_ctx* ctx, int layer, const float* xa, const float* xb, float* yacc, float* x_store,
                     float* zero_out, int B, int normalize, int gu_sel, cudaStream_t s) {
  const Dims& d = ctx->d;
  const size_t row_bytes = (size_t)d.D * 2;
  MlpArgs a;
  const bool dense_layer = layer < d.dense;
  if (dense_layer) {  // whole records, every row active (tensor-core batch kernels only)
    const char* rec0 = static_cast<const char*>(ctx->bufs.dense_buf) + (size_t)layer * d.M * 3 * d.D * 2;
    a.gate_l = rec0;
    a.up_l = rec0 + row_bytes;
    a.downT_l = rec0 + 2 * row_bytes;
    a.active_slots = ctx->t.identity;
  } else {
    a.gate_l = static_cast<const char*>(ctx->bufs.gate_buf) + (size_t)(layer - d.dense) * d.C * row_bytes;
    a.up_l = static_cast<const char*>(ctx->bufs.up_buf) + (size_t)(layer - d.dense) * d.C * row_bytes;
    a.downT_l = static_cast<const char*>(ctx->bufs.downT_buf) + (size_t)(layer - d.dense) * d.C * row_bytes;
    a.active_slots = ctx->t.active_slots + (size_t)layer * d.C;
  }
  a.dense_rows = dense_layer ? d.M : 0;
  a.gu_rows = d.dense > 0 ? d.M : d.C;
  a.n_active_ptr = ctx->t.counters + (size_t)layer * NP_N_COUNTERS + NP_CNT_ACTIVE;
  a.xa = xa;
  a.xb = xb;
  a.yacc = yacc;
  a.x_store = x_store;
  a.zero_out = zero_out;
  a.B = B;
  a.C = d.C;
  a.check = ctx->cfg.flags & NP_F_CHECK_BOUNDS;
  a.normalize = normalize;
  a.force_direct = (ctx->cfg.flags & NP_F_DIRECT_LOADS) ? 1 : 0;
  a.status = ctx->t.status;
  a.gu = a.gu_next = a.ssq = a.ssq_next = nullptr;
  a.xterms = (ctx->cfg.flags & NP_F_TCGEN05_BATCH) ? ctx->xterms : nullptr;
  if (ctx->install_pending[layer]) NP_CUDA(ctx, cudaStreamWaitEvent(s, ctx->ev_installed[layer], 0));
  if (ctx->mlp_tc && B >= kTcMinBatch && !a.force_direct) {
    const int cur = gu_sel < 0 ? 0 : gu_sel;
    a.gu = ctx->ws.gu[cur];
    a.ssq = ctx->ws.ssq[cur];
    if (gu_sel >= 0) {
      a.gu_next = ctx->ws.gu[cur ^ 1];
      a.ssq_next = ctx->ws.ssq[cur ^ 1];
    }
    // two kernels per layer; three where the tcgen05 up kernel runs (x is split by a kernel of its own)
    ctx->launches += (a.xterms && !dense_layer && mlp_tc_up_on_tcgen05(d, ctx->sm_count)) ? 2 : 1;
    NP_LAUNCH(ctx, launch_sparse_mlp_tc(d, a, s, ctx->sm_count));
    return NP_OK;
  }
  if (dense_layer) return fail(ctx, NP_E_STATE, "dense layer %d reached a kernel that cannot run it", layer);
  NP_LAUNCH(ctx, launch_sparse_mlp(d, a, s, ctx->sm_count));
  return NP_OK;
}

// residual chain: x_l = xbuf[(l+1)&1] + zbuf[(l-1)%3]; layer l accumulates MLP_l(x_l) into
// zbuf[l%3], stores x_l to xbuf[l&1] and clears zbuf[(l+1)%3] for the next layer
// `part`: kChainAll = the whole chain; kChainHead = its start up to the end of the dense prefix
// (nothing there waits for an install, so np_step queues it before the host packs any rows);
// kChainTail = the sparse layers and the result.
enum { kChainAll = 0, kChainHead = 1, kChainTail = 2 };
static int mlp_chain(np_ctx* ctx, const void* x_bf16, int B, float* x_out, cudaStream_t s, int part = kChainAll) {
  const Dims& d = ctx->d;
  const size_t n = (size_t)B * d.D;
  const bool persistent = B == 1 && !(ctx->cfg.flags & (NP_F_DIRECT_LOADS | NP_F_LAYER_LAUNCHES)) &&
                          (ctx->use_rows || ctx->use_slices || chain_alu::supported(d, ctx->sm_count));
  const bool tc_batch = !persistent && ctx->mlp_tc && B >= kTcMinBatch && !(ctx->cfg.flags & NP_F_DIRECT_LOADS);
  if (part != kChainTail) ctx->chain_kernel_launches = 0;
  // the sliced kernel widens the stack's bf16 input itself when it runs layer 0
  const bool fold_widen = persistent && (ctx->use_rows || ctx->use_slices) && d.dense == 0;
  // Where the sliced kernel hands its sums over as counted words, layer 0's fp32 accumulator is used only by a
  // first launch of one layer that does not end the stack: the clearing waits until the runs are known.
  const bool lazy_clear = fold_widen && ctx->use_slices && !ctx->use_rows && chain_slices::counted_handover(d, ctx->sm_count);
  bool out_written = false;  // the last resident launch left x_out itself
  if (part != kChainTail) {
    if (!fold_widen) NP_LAUNCH(ctx, launch_widen_bf16(x_bf16, ctx->ws.xbuf[1], n, s));
    // the accumulator of layer 0 starts at zero (later ones are cleared one layer ahead)
    if (!lazy_clear) NP_CUDA(ctx, cudaMemsetAsync(ctx->ws.zbuf[0], 0, (persistent ? (size_t)kZRep * d.D : n) * 4, s));
  }
  if (persistent) {
    // runs of layers in one resident kernel each; a run starts once its layers are installed,
    // so the install of later runs still overlaps the compute of earlier ones
    const int run = std::max(1, ctx->cfg.chain_layers > 0 ? ctx->cfg.chain_layers : (d.L + 3) / 4);
    const size_t row_bytes = (size_t)d.D * 2;
    ChainArgs a;
    for (int i = 0; i < 2; ++i) a.xbuf[i] = ctx->ws.xbuf[i];
    for (int i = 0; i < 3; ++i) a.zbuf[i] = ctx->ws.zbuf[i];
    a.grid_bar = ctx->t.grid_bar;
    a.status = ctx->t.status;
    a.check = ctx->cfg.flags & NP_F_CHECK_BOUNDS;
    a.counters = ctx->t.counters;
    a.x_bf16 = fold_widen ? x_bf16 : nullptr;
    a.x_out = nullptr;
    // the dense prefix first: whole records, every row active, nothing to wait for (it also
    // widens the window in which the sparse layers' rows arrive)
    if (d.dense > 0 && part != kChainTail) {
      const char* dense = static_cast<const char*>(ctx->bufs.dense_buf);
      a.gate = dense;
      a.up = dense + row_bytes;
      a.downT = dense + 2 * row_bytes;
      a.active_slots = ctx->t.identity;
      a.dense_rows = d.M;
      // Runs, not one launch: while a resident launch is on the device the install's scatter
      // kernels do not run beside it (its blocks hold the register file), so the installs of the
      // sparse layers advance between runs.  The fewer sparse layers wait for rows, the longer a
      // run may be (measured at the 7B shape: d = 20: 697 steps/s with runs of 3, 648 with 6;
      // d = 24: 711 / 755 / 702 / 594 with runs of 3 / 6 / 8 / 24; d = 28: 682 / 710 / 725 with
      // 3 / 6 / 12).
      const int dense_run = d.dense < d.L ? std::max(3, std::min(12, 2 * d.dense / (d.L - d.dense))) : 12;
      for (int l0 = 0; l0 < d.dense; l0 += dense_run) {
        a.l_begin = l0;
        a.l_end = std::min(d.dense, l0 + dense_run);
        if (dense_chain::supported(d, ctx->sm_count))
          NP_LAUNCH(ctx, dense_chain::launch(d, dense, d.M, a.xbuf, a.zbuf, a.grid_bar, a.status, a.l_begin, a.l_end, s,
                                             ctx->sm_count));
        else
          NP_LAUNCH(ctx, chain_alu::launch(d, a, s, ctx->sm_count));
      }
    }
    // the sparse layers' buffers start at layer d; the kernels index them by absolute layer
    const size_t shift = (size_t)d.dense * d.C * row_bytes;
    a.gate = static_cast<const char*>(ctx->bufs.gate_buf) - shift;
    a.up = static_cast<const char*>(ctx->bufs.up_buf) - shift;
    a.downT = static_cast<const char*>(ctx->bufs.downT_buf) - shift;
    a.active_slots = ctx->t.active_slots;
    a.dense_rows = 0;
    // Runs of the sparse layers.  A run starts once its layers are installed, so what the step waits for
    // after its last row has landed is the last run: with chain_layers = 0 the runs shrink towards the end
    // (the tail is an eighth of the stack, the run before it a quarter, the first run takes the rest), which
    // also makes fewer launches than equal runs of a quarter each.
    std::vector<int> runs;
    if (part != kChainHead) {
      // layers whose rows have all landed already need no run of their own to wait in: they go into one
      // first run (the whole stack when nothing is pending, as in np_mlp_chain on resident rows)
      int landed = d.dense;
      while (landed < d.L) {
        if (ctx->install_pending[landed]) {
          const cudaError_t q = cudaEventQuery(ctx->ev_installed[landed]);
          if (q == cudaErrorNotReady) {
            (void)cudaGetLastError();
            break;
          }
          if (q != cudaSuccess) return fail(ctx, NP_E_CUDA, "cudaEventQuery failed: %s", cudaGetErrorString(q));
          ctx->install_pending[landed] = 0;
        }
        ++landed;
      }
      const int ns = d.L - landed;  // layers that still wait for rows
      if (ctx->cfg.chain_layers > 0) {
        for (int l0 = d.dense; l0 < d.L; l0 += run) runs.push_back(std::min(run, d.L - l0));
      } else {
        if (landed > d.dense) runs.push_back(landed - d.dense);
        if (ns > 0) {
          const int unit = std::max(1, (d.L - d.dense) / 8);
          const int tail = std::min(ns, unit), mid = std::min(ns - tail, 2 * unit), first = ns - tail - mid;
          if (first > 0) runs.push_back(first);
          if (mid > 0) runs.push_back(mid);
          runs.push_back(tail);
        }
      }
    }
    int l0 = d.dense;
    for (size_t ri = 0; ri < runs.size() && part != kChainHead; ++ri) {
      const int l1 = l0 + runs[ri];
      for (int l = l0; l < l1; ++l)
        if (ctx->install_pending[l]) NP_CUDA(ctx, wait_install(ctx, l, s));
      a.l_begin = l0;
      a.l_end = l1;
      if (ctx->use_rows) {
        const int rl = chain_rows::run_layers(d, ctx->rows);
        ctx->chain_kernel_launches += (l1 - l0 + rl - 1) / rl;
        NP_LAUNCH(ctx, chain_rows::launch(d, a, &ctx->rows, s));
      } else if (ctx->use_slices) {
        chain_slices::Plan sp;
        chain_slices::plan(d, ctx->sm_count, &sp);
        ctx->chain_kernel_launches += (l1 - l0 + sp.run_layers - 1) / sp.run_layers;
        a.x_out = l1 == d.L ? x_out : nullptr;  // the run that ends the stack may leave the result itself
        if (lazy_clear && l0 == 0 && std::min(l1, sp.run_layers) == 1 && l1 != d.L)
          NP_CUDA(ctx, cudaMemsetAsync(ctx->ws.zbuf[0], 0, (size_t)kZRep * d.D * 4, s));
        NP_LAUNCH(ctx, chain_slices::launch(d, a, &ctx->slices, s, ctx->sm_count));
        out_written = a.x_out && ctx->slices.wrote_out;
      } else {
        ctx->chain_kernel_launches += 1;
        NP_LAUNCH(ctx, chain_alu::launch(d, a, s, ctx->sm_count));
      }
      l0 = l1;
    }
  } else {
    if (part != kChainTail && ctx->mlp_tc && B >= kTcMinBatch)
      NP_CUDA(ctx, cudaMemsetAsync(ctx->ws.gu[0], 0, ctx->gu_bytes, s));
    const int lo = part == kChainTail ? d.dense : 0, hi = part == kChainHead ? d.dense : d.L;
    for (int l = lo; l < hi; ++l) {
      int rc;
      if (tc_batch) {
        // The tensor-core pair keeps x in the accumulator itself: the up kernel stores x_l into
        // zbuf[l % 3] (its blocks of row block 0, one K slice each), the down kernel adds
        // MLP_l(x_l) on top, and the next layer reads x_{l+1} from there: one vector to read per
        // block instead of two, nothing to clear.
        rc = mlp_layer(ctx, l, l > 0 ? ctx->ws.zbuf[(l - 1) % 3] : ctx->ws.xbuf[1], nullptr, ctx->ws.zbuf[l % 3],
                       ctx->ws.zbuf[l % 3], nullptr, B, 1, l & 1, s);
      } else {
        rc = mlp_layer(ctx, l, ctx->ws.xbuf[(l + 1) & 1], l > 0 ? ctx->ws.zbuf[(l - 1) % 3] : nullptr,
                       ctx->ws.zbuf[l % 3], ctx->ws.xbuf[l & 1], ctx->ws.zbuf[(l + 1) % 3], B, 1, l & 1, s);
      }
      if (rc < 0) return rc;
    }
  }
  if (part != kChainHead && !out_written) {
    if (tc_batch)  // the last accumulator holds the result
      NP_LAUNCH(ctx, launch_add_vec(ctx->ws.zbuf[(d.L - 1) % 3], nullptr, 0, x_out, n, s));
    else
      NP_LAUNCH(ctx, launch_add_vec(ctx->ws.xbuf[(d.L - 1) & 1], ctx->ws.zbuf[(d.L - 1) % 3], persistent ? kZRep : 1,
                                    x_out, n, s));
  }
  return NP_OK;
}

int np_mlp_chain(np_ctx* ctx, const void* x_bf16, int32_t B, float* x_out, void* stream) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  if (!x_bf16 || !x_out) return fail(ctx, NP_E_INVAL, "x or x_out is NULL");
  if ((uintptr_t)x_out % 16) return fail(ctx, NP_E_INVAL, "x_out must be 16-byte aligned");
  if (B < 1 || B > ctx->d.Bmax) return fail(ctx, NP_E_INVAL, "B=%d outside [1, max_batch=%d]", B, ctx->d.Bmax);
  if (!ctx->have_delta) return fail(ctx, NP_E_STATE, "np_mlp_chain needs a prior np_delta");
  return mlp_chain(ctx, x_bf16, B, x_out, as_stream(stream));
}

int np_selftest_bounded_wait(np_ctx* ctx, void* stream) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  cudaStream_t s = as_stream(stream);
  NP_LAUNCH(ctx, launch_selftest_wait(ctx->t.status, s));
  const int rc = check_device_status(ctx, s);
  return rc == NP_E_DEVICE ? NP_E_DEVICE : (rc < 0 ? rc : fail(ctx, NP_E_STATE, "the wait did not time out"));
}

int np_speculate(np_ctx* ctx, const uint32_t* cand_bitmap, int32_t budget, void* stream) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  if (!cand_bitmap) return fail(ctx, NP_E_INVAL, "cand_bitmap is NULL");
  if (budget < 0) return fail(ctx, NP_E_INVAL, "budget must be >= 0");
  if (!ctx->have_delta) return fail(ctx, NP_E_STATE, "np_speculate needs a prior np_delta");
  cudaStream_t s = as_stream(stream);
  // rows brought in ahead of time by an earlier call must have landed before their tables move again
  for (int l = 0; l < ctx->d.L; ++l)
    if (ctx->have_spec && ctx->install_pending[l]) NP_CUDA(ctx, cudaStreamWaitEvent(s, ctx->ev_installed[l], 0));
  NP_LAUNCH(ctx, launch_speculate(ctx->d, ctx->t, cand_bitmap, std::min(budget, ctx->d.C),
                                  ctx->host_lists_dev + host_area_ints(ctx->cfg), s));
  NP_CUDA(ctx, cudaEventRecord(ctx->ev_spec, s));
  ctx->have_spec = true;
  return NP_OK;
}

int np_install_speculative(np_ctx* ctx, void* copy_stream) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  if (!ctx->have_spec) return fail(ctx, NP_E_STATE, "np_install_speculative needs a prior np_speculate");
  // The speculative rows take the very path of the incoming rows: for the length of this call the
  // install code is pointed at the second list area (host mirror, device lists, counts, event).
  struct Saved {
    int32_t *host, *ids, *slots, *counters;
    cudaEvent_t ev;
  } keep = {ctx->host_lists, ctx->t.delta_ids, ctx->t.delta_slots, ctx->t.counters, ctx->ev_delta};
  ctx->host_lists += host_area_ints(ctx->cfg);
  ctx->t.delta_ids = ctx->t.spec_ids;
  ctx->t.delta_slots = ctx->t.spec_slots;
  ctx->t.counters = ctx->t.spec_counters;
  ctx->ev_delta = ctx->ev_spec;
  const int rc = np_install(ctx, 0, ctx->d.L, copy_stream);
  ctx->host_lists = keep.host;
  ctx->t.delta_ids = keep.ids;
  ctx->t.delta_slots = keep.slots;
  ctx->t.counters = keep.counters;
  ctx->ev_delta = keep.ev;
  return rc;
}

int np_get_speculative(np_ctx* ctx, int32_t layer, const int32_t** ids, const int32_t** slots, const int32_t** count) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  if (layer < 0 || layer >= ctx->d.L) return fail(ctx, NP_E_INVAL, "layer %d outside [0, %d)", layer, ctx->d.L);
  if (!ctx->have_spec) return fail(ctx, NP_E_STATE, "np_get_speculative needs a prior np_speculate");
  if (ids) *ids = ctx->t.spec_ids + (size_t)layer * ctx->d.C;
  if (slots) *slots = ctx->t.spec_slots + (size_t)layer * ctx->d.C;
  if (count) *count = ctx->t.spec_counters + (size_t)layer * NP_N_COUNTERS + NP_CNT_DELTA;
  return NP_OK;
}

int np_chain_launches(np_ctx* ctx, int32_t* out) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  if (!out) return fail(ctx, NP_E_INVAL, "out is NULL");
  *out = ctx->chain_kernel_launches;
  return NP_OK;
}

const char* np_mlp_kernel_name(np_ctx* ctx, int32_t B) {
  if (!ctx || B < 1 || B > ctx->d.Bmax) return nullptr;
  const Dims& d = ctx->d;
  const int flags = ctx->cfg.flags;
  if (B == 1 && !(flags & (NP_F_DIRECT_LOADS | NP_F_LAYER_LAUNCHES))) {
    if (ctx->use_rows) return "k_mlp_rows";
    if (ctx->use_slices) return "k_mlp_slices";
    if (chain_alu::supported(d, ctx->sm_count)) return "k_mlp_chain_alu";
  }
  if (ctx->mlp_tc && B >= kTcMinBatch && !(flags & NP_F_DIRECT_LOADS))
    return ((flags & NP_F_TCGEN05_BATCH) && mlp_tc_up_on_tcgen05(d, ctx->sm_count)) ? "k_mlp_up5 + k_mlp_tc_down" : "k_mlp_tc_up + k_mlp_tc_down";
  return (flags & NP_F_DIRECT_LOADS) ? "k_sparse_mlp" : "k_sparse_mlp_pipe";
}

int np_launch_count(np_ctx* ctx, uint64_t* out) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  if (!out) return fail(ctx, NP_E_INVAL, "out is NULL");
  *out = ctx->launches;
  return NP_OK;
}

int np_sparse_mlp(np_ctx* ctx, int32_t layer, const float* x, int32_t B, float* y, void* stream) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  const Dims& d = ctx->d;
  if (layer < 0 || layer >= d.L) return fail(ctx, NP_E_INVAL, "layer %d outside [0, %d)", layer, d.L);
  if (layer < d.dense) return fail(ctx, NP_E_INVAL, "layer %d is dense: it runs only inside np_mlp_chain / np_step", layer);
  if (!x || !y) return fail(ctx, NP_E_INVAL, "x or y is NULL");
  if ((uintptr_t)x % 16 || (uintptr_t)y % 16) return fail(ctx, NP_E_INVAL, "x and y must be 16-byte aligned");
  if (B < 1 || B > d.Bmax) return fail(ctx, NP_E_INVAL, "B=%d outside [1, max_batch=%d]", B, d.Bmax);
  if (!ctx->have_delta) return fail(ctx, NP_E_STATE, "np_sparse_mlp needs a prior np_delta");
  cudaStream_t s = as_stream(stream);
  NP_CUDA(ctx, cudaMemsetAsync(y, 0, (size_t)B * d.D * 4, s));
  if (ctx->mlp_tc && B >= kTcMinBatch) NP_CUDA(ctx, cudaMemsetAsync(ctx->ws.gu[0], 0, ctx->gu_bytes / 2, s));
  return mlp_layer(ctx, layer, x, nullptr, y, nullptr, nullptr, B, 0, -1, s);
}

// One decode step; `selected` = NULL runs the library's own predictor and top-k, otherwise the
// caller's bitmap takes their place.
static int step_impl(np_ctx* ctx, const void* x_bf16, int32_t B, const uint32_t* selected, float* x_out,
                     void* stream, void* copy_stream) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  if (!x_bf16 || !x_out) return fail(ctx, NP_E_INVAL, "x or x_out is NULL");
  if ((uintptr_t)x_out % 16) return fail(ctx, NP_E_INVAL, "x_out must be 16-byte aligned");
  if (B < 1 || B > ctx->d.Bmax) return fail(ctx, NP_E_INVAL, "B=%d outside [1, max_batch=%d]", B, ctx->d.Bmax);
  if (stream == copy_stream) return fail(ctx, NP_E_INVAL, "a step needs two different streams");
  const Dims& d = ctx->d;
  cudaStream_t s = as_stream(stream), cs = as_stream(copy_stream);
  NP_CUDA(ctx, cudaEventRecord(ctx->ev_t[0], s));
  int rc = NP_OK;
  if (!selected) rc = np_predict(ctx, x_bf16, B, nullptr, nullptr, stream);
  if (rc < 0) return rc;
  NP_CUDA(ctx, cudaEventRecord(ctx->ev_t[1], s));
  rc = np_delta(ctx, selected, stream);
  if (rc < 0) return rc;
  NP_CUDA(ctx, cudaEventRecord(ctx->ev_t[2], s));
  // Speculative prefetch behind the step (Section 6's future work).  Its candidates are the rows ranked
  // k+1 .. k+s by this step's own logits (a caller's selection has no ranking to extend: the caller then
  // calls np_speculate itself).  The second selection and the table update run right behind the delta
  // step (the MLP launches read only the step's active lists and their slots, which a speculative row
  // never takes); the transfer is queued last, behind the incoming rows and the MLP launches.
  const bool spec = ctx->cfg.spec_rows > 0 && !selected;
  if (spec) {
    Dims ds = d;
    const int skip_layers = B == 1 ? d.dense : 0;
    ds.L = d.L - skip_layers;
    ds.k = std::min(d.M, d.k + ctx->cfg.spec_rows);
    if (ds.L > 0)
      NP_LAUNCH(ctx, launch_topk(ds, ctx->ws.logits + (size_t)skip_layers * d.M, B,
                                 ctx->t.spec_cand + (size_t)skip_layers * d.W, s));
    if (d.dense > 0) NP_CUDA(ctx, cudaMemsetAsync(ctx->t.spec_cand, 0, (size_t)d.dense * d.W * 4, s));
    rc = np_speculate(ctx, ctx->t.spec_cand, ctx->cfg.spec_rows, stream);
    if (rc < 0) return rc;
  }
  // the dense prefix waits for no install: it is queued before the host starts on the rows
  const bool head_first = d.dense > 0;
  if (head_first) {
    rc = mlp_chain(ctx, x_bf16, B, x_out, s, kChainHead);
    if (rc < 0) return rc;
  }
  // the copy stream is ordered after the delta step inside np_install
  NP_CUDA(ctx, cudaStreamWaitEvent(cs, ctx->ev_delta, 0));
  NP_CUDA(ctx, cudaEventRecord(ctx->ev_c[0], cs));
  const int warn = np_install(ctx, 0, d.L, copy_stream);
  if (warn < 0) return warn;
  NP_CUDA(ctx, cudaEventRecord(ctx->ev_c[1], cs));

  rc = mlp_chain(ctx, x_bf16, B, x_out, s, head_first ? kChainTail : kChainAll);
  if (rc < 0) return rc;
  NP_CUDA(ctx, cudaEventRecord(ctx->ev_t[3], s));
  ctx->have_step = true;
  if (spec) {
    // the guessed rows cross behind the step's own rows, while its MLP launches run
    rc = np_install_speculative(ctx, copy_stream);
    if (rc < 0) return rc;
  }
  return warn;
}

int np_step(np_ctx* ctx, const void* x_bf16, int32_t B, float* x_out, void* stream, void* copy_stream) {
  return step_impl(ctx, x_bf16, B, nullptr, x_out, stream, copy_stream);
}

int np_step_selected(np_ctx* ctx, const void* x_bf16, int32_t B, const uint32_t* bitmap, float* x_out, void* stream,
                     void* copy_stream) {
  if (ctx && !bitmap) return fail(ctx, NP_E_INVAL, "bitmap is NULL");
  return step_impl(ctx, x_bf16, B, bitmap, x_out, stream, copy_stream);
}

int np_last_step_times(np_ctx* ctx, float* out_us) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  if (!out_us) return fail(ctx, NP_E_INVAL, "out is NULL");
  if (!ctx->have_step) return fail(ctx, NP_E_STATE, "no np_step has run");
  NP_CUDA(ctx, cudaEventSynchronize(ctx->ev_t[3]));
  NP_CUDA(ctx, cudaEventSynchronize(ctx->ev_c[1]));
  float ms[4];
  NP_CUDA(ctx, cudaEventElapsedTime(&ms[0], ctx->ev_t[0], ctx->ev_t[1]));
  NP_CUDA(ctx, cudaEventElapsedTime(&ms[1], ctx->ev_t[1], ctx->ev_t[2]));
  NP_CUDA(ctx, cudaEventElapsedTime(&ms[2], ctx->ev_c[0], ctx->ev_c[1]));
  NP_CUDA(ctx, cudaEventElapsedTime(&ms[3], ctx->ev_t[2], ctx->ev_t[3]));
  for (int i = 0; i < 4; ++i) out_us[i] = ms[i] * 1000.f;
  return NP_OK;
}

int np_get_delta(np_ctx* ctx, int32_t layer, np_delta_view* out) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  if (!out) return fail(ctx, NP_E_INVAL, "out is NULL");
  const Dims& d = ctx->d;
  if (layer < 0 || layer >= d.L) return fail(ctx, NP_E_INVAL, "layer %d outside [0, %d)", layer, d.L);
  if (!ctx->have_delta) return fail(ctx, NP_E_STATE, "np_get_delta needs a prior np_delta");
  out->delta_ids = ctx->t.delta_ids + (size_t)layer * d.C;
  out->delta_slots = ctx->t.delta_slots + (size_t)layer * d.C;
  out->evict_ids = ctx->t.evict_ids + (size_t)layer * d.C;
  out->overflow_ids = ctx->t.overflow_ids + (size_t)layer * d.M;
  out->active_ids = ctx->t.active_ids + (size_t)layer * d.C;
  out->active_slots = ctx->t.active_slots + (size_t)layer * d.C;
  out->counters = ctx->t.counters + (size_t)layer * NP_N_COUNTERS;
  return NP_OK;
}

int np_read_counters(np_ctx* ctx, int32_t* out_host, void* stream) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  if (!out_host) return fail(ctx, NP_E_INVAL, "out is NULL");
  cudaStream_t s = as_stream(stream);
  NP_CUDA(ctx, cudaMemcpyAsync(out_host, ctx->t.counters, (size_t)ctx->d.L * NP_N_COUNTERS * 4,
                               cudaMemcpyDeviceToHost, s));
  return check_device_status(ctx, s);
}

int np_export_state(np_ctx* ctx, int32_t layer, int32_t* slot_map, int32_t* owner, uint32_t* resident,
                    int32_t* stamp, void* stream) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  const Dims& d = ctx->d;
  if (layer < 0 || layer >= d.L) return fail(ctx, NP_E_INVAL, "layer %d outside [0, %d)", layer, d.L);
  cudaStream_t s = as_stream(stream);
  if (slot_map)
    NP_CUDA(ctx, cudaMemcpyAsync(slot_map, ctx->t.slot_map + (size_t)layer * d.M, (size_t)d.M * 4,
                                 cudaMemcpyDeviceToHost, s));
  if (owner)
    NP_CUDA(ctx, cudaMemcpyAsync(owner, ctx->t.owner + (size_t)layer * d.C, (size_t)d.C * 4, cudaMemcpyDeviceToHost, s));
  if (resident)
    NP_CUDA(ctx, cudaMemcpyAsync(resident, ctx->t.resident + (size_t)layer * d.W, (size_t)d.W * 4,
                                 cudaMemcpyDeviceToHost, s));
  if (stamp)
    NP_CUDA(ctx, cudaMemcpyAsync(stamp, ctx->t.stamp + (size_t)layer * d.M, (size_t)d.M * 4, cudaMemcpyDeviceToHost, s));
  return check_device_status(ctx, s);
}

int np_import_state(np_ctx* ctx, int32_t layer, const int32_t* slot_map, const int32_t* owner,
                    const uint32_t* resident, const int32_t* stamp, int32_t step, void* stream) {
  if (!ctx) return fail(nullptr, NP_E_INVAL, "ctx is NULL");
  const Dims& d = ctx->d;
  if (layer < 0 || layer >= d.L) return fail(ctx, NP_E_INVAL, "layer %d outside [0, %d)", layer, d.L);
  if (!slot_map || !owner || !resident || !stamp) return fail(ctx, NP_E_INVAL, "a state array is NULL");
  if (step < 0) return fail(ctx, NP_E_INVAL, "step must be >= 0");
  cudaStream_t s = as_stream(stream);
  NP_CUDA(ctx, cudaMemcpyAsync(ctx->t.slot_map + (size_t)layer * d.M, slot_map, (size_t)d.M * 4,
                               cudaMemcpyHostToDevice, s));
  NP_CUDA(ctx, cudaMemcpyAsync(ctx->t.owner + (size_t)layer * d.C, owner, (size_t)d.C * 4, cudaMemcpyHostToDevice, s));
  NP_CUDA(ctx, cudaMemcpyAsync(ctx->t.resident + (size_t)layer * d.W, resident, (size_t)d.W * 4,
                               cudaMemcpyHostToDevice, s));
  NP_CUDA(ctx, cudaMemcpyAsync(ctx->t.stamp + (size_t)layer * d.M, stamp, (size_t)d.M * 4, cudaMemcpyHostToDevice, s));
  NP_CUDA(ctx, cudaStreamSynchronize(s));
  ctx->step = step;
  return NP_OK;
}

int np_read_records(int32_t fd, uint64_t base_offset, uint64_t rec_bytes, const int32_t* ids, int32_t n, void* dst,
                    int32_t io_depth, int32_t* n_ranges_out, int32_t* used_ring_out) {
  if (fd < 0 || !rec_bytes || n < 0 || (n > 0 && (!ids || !dst)))
    return fail(nullptr, NP_E_INVAL, "np_read_records: bad descriptor, record size, count or NULL pointer");
  if (io_depth < -1 || io_depth > 4096) return fail(nullptr, NP_E_INVAL, "io_depth must be in [-1, 4096]");
  for (int i = 0; i < n; ++i)
    if (ids[i] < 0 || (i > 0 && ids[i] <= ids[i - 1]))
      return fail(nullptr, NP_E_INVAL, "np_read_records: ids must be non-negative and strictly ascending");
  RecordReader reader;
  std::string note;
  if (!reader.open(fd, io_depth, nullptr, &note)) return fail(nullptr, NP_E_IO, "np_read_records: cannot use the descriptor");
  int ranges = 0, r = 0;
  bool ok = true;
  while (r < n && ok) {
    int len = 1;
    while (r + len < n && ids[r + len] == ids[r] + len) ++len;
    ok = reader.submit(static_cast<char*>(dst) + (size_t)r * rec_bytes, (size_t)len * rec_bytes,
                       base_offset + (uint64_t)ids[r] * rec_bytes, ranges % RecordReader::kGroups);
    ++ranges;
    r += len;
  }
  ok = reader.drain() && ok;
  if (n_ranges_out) *n_ranges_out = ranges;
  if (used_ring_out) *used_ring_out = reader.uses_ring() ? 1 : 0;
  if (!ok) return fail(nullptr, NP_E_IO, "np_read_records: a read failed: %s", strerror(reader.last_error()));
  return NP_OK;
}

}  // extern "C"
