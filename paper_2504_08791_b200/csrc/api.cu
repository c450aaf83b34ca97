// C ABI of the layer-window decoder: context, weight loading, window execution, output layer.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "../../include/prima.h"
#include "common.cuh"

using namespace prima;

namespace {

thread_local std::string g_tls_error;

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
    ok = cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

struct Layer {
  TiledMat qkv, o, gu, down;
  float* g_attn = nullptr;
  float* g_ffn = nullptr;
  float gmax_attn = 1.f, gmax_ffn = 1.f;
  uint32_t have = 0;   // bit per tensor id
  __half* k = nullptr;        // cache of sequence 0 (the only one that prima_forward_window uses)
  __half* v = nullptr;
  std::vector<__half*> k_seq, v_seq;   // caches of sequences 1.. (index seq - 1), allocated on first use
  uint8_t* host = nullptr;    // streamed layers: the four tiled matrices in pinned host memory (qkv | o | gate/up | down)
};

// A device buffer that holds the matrices of ONE streamed layer at a time.
struct StreamSlot {
  uint8_t* dev = nullptr;
  int layer = -1;              // layer whose copy was queued into the slot (or -1)
  bool waited = false;         // the compute stream already waits for that copy
  bool used = false;           // a compute pass over the slot's content has been queued (compute_done is recorded)
  cudaEvent_t copy_done = nullptr, compute_done = nullptr;
};
struct CopySpan { cudaEvent_t t0, t1; };      // around one layer's copy, for the statistics

constexpr uint32_t kLayerMask = (1u << 9) - 1;
constexpr uint32_t kMatrixMask = kLayerMask & ~((1u << PRIMA_ATTN_NORM) | (1u << PRIMA_FFN_NORM));

}  // namespace

struct prima_ctx {
  prima_model_config cfg{};
  cudaStream_t stream = nullptr;
  int sm_count = 0;
  std::vector<Layer> layers;
  float* g_out = nullptr;
  float gmax_out = 1.f;
  TiledMat head;
  uint8_t* embd = nullptr;
  bool have_out_norm = false, have_head = false, have_embd = false;

  // fixed-point accumulators of the products, [max_n_tok][padded rows] each; all zero between calls
  acc_t* acc_qkv = nullptr;  // QKV and head products
  acc_t* acc_o = nullptr;    // O product
  acc_t* acc_gu = nullptr;   // gate/up product
  acc_t* acc_down = nullptr; // down product
  int64_t n_acc_qkv = 0, n_acc_o = 0, n_acc_gu = 0, n_acc_down = 0;
  float* h_a = nullptr;      // residual stream entering a layer / leaving its feed-forward block
  float* h_b = nullptr;      // residual stream after the attention block
  float* obuf = nullptr;
  SumSq ssq_attn, ssq_ffn, ssq_out;
  float2* rope_tab = nullptr;
  AttnScratch attn{};
  uint8_t* staging = nullptr;
  size_t staging_bytes = 0;
  int32_t* d_tokens = nullptr;
  float* am_val = nullptr;
  int32_t* am_idx = nullptr;
  int32_t* am_out = nullptr;
  int* status = nullptr;

  // ---- layers streamed from pinned host memory (PRIMA_OPT_RESIDENT_LAYERS) ----
  int n_resident = -1;                 // -1: every layer lives on the device
  int n_slots = 2;
  std::vector<StreamSlot> slots;
  cudaStream_t copy_stream = nullptr;
  size_t off_o = 0, off_gu = 0, off_down = 0, layer_bytes = 0;
  int loading_layer = -1;              // streamed layer being assembled in slot 0
  int64_t streamed_bytes = 0;
  double copy_ms = 0;
  std::vector<void*> pinned;
  std::vector<CopySpan> spans_pending, spans_free;

  std::vector<void*> allocs;
  std::string err;
  int64_t launches = 0;
  // Lowest cache position appended since the host last waited for the stream (INT_MAX: none).  Entries below it are
  // known to be in memory and may be read by the attention kernels before their dependency wait.
  int unsynced_min_pos = 0x7fffffff;
  uint32_t first_wait_polls = 0;   // PRIMA_OPT_FIRST_WAIT_POLLS (0: the ordinary limit)
  int64_t l2_ahead_bytes = -1;     // PRIMA_OPT_L2_AHEAD_BYTES (-1: a sixteenth of the gate/up matrix)
  int64_t l2_ahead_o_bytes = -1;   // PRIMA_OPT_L2_AHEAD_O_BYTES
  int64_t fail_after = -1;         // PRIMA_OPT_FAIL_AFTER_LAUNCHES: launch steps still allowed before an injected failure (-1: off)

  // optional per-class device timing (prima_profile_*): mode 1 = a pair of events around every launch,
  // mode 2 = in-situ stamps written by the kernels themselves
  bool profiling = false;
  struct Span { cudaEvent_t a, b; int klass; int64_t bytes; int launches; };
  std::vector<Span> spans;
  bool stamping = false;
  unsigned long long* stamp_t0 = nullptr;   // device, [kMaxStamps]
  unsigned long long* stamp_t1 = nullptr;
  struct StampInfo { int klass; int sub; int64_t bytes; int launches; };
  std::vector<StampInfo> stamp_info;
};

struct prima_gemv_plan {
  int device = 0;
  int sm_count = 0;
  int max_n_cols = 1;
  TiledMat w;
  acc_t* acc = nullptr;
  int* status = nullptr;
};

namespace {

int fail(prima_ctx* c, int code, const std::string& msg) {
  if (c) c->err = msg;
  else g_tls_error = msg;
  return code;
}

int cuda_fail(prima_ctx* c, cudaError_t e, const char* what) {
  std::string msg = std::string(what) + ": " + cudaGetErrorString(e);
  return fail(c, e == cudaErrorMemoryAllocation ? PRIMA_ERR_NOMEM : PRIMA_ERR_CUDA, msg);
}

template <typename T>
int dev_alloc(prima_ctx* c, T** p, size_t count, bool zero = false) {
  void* raw = nullptr;
  cudaError_t e = cudaMalloc(&raw, std::max<size_t>(count * sizeof(T), 16));
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaMalloc");
  if (zero) {
    e = cudaMemsetAsync(raw, 0, std::max<size_t>(count * sizeof(T), 16), c->stream);
    if (e != cudaSuccess) {
      cudaFree(raw);
      return cuda_fail(c, e, "cudaMemsetAsync");
    }
  }
  c->allocs.push_back(raw);
  *p = static_cast<T*>(raw);
  return PRIMA_OK;
}

TiledMat shape_tiled(int64_t rows, int64_t cols) {
  TiledMat t;
  t.rows = rows;
  t.cols = cols;
  t.n_rt = (rows + kRowsPerTile - 1) / kRowsPerTile;
  t.n_sb = cols / 256;
  return t;
}

int ensure_tiled(prima_ctx* c, TiledMat* t, int64_t rows, int64_t cols) {
  if (t->data) return PRIMA_OK;
  TiledMat s = shape_tiled(rows, cols);
  int rc = dev_alloc(c, &s.data, s.bytes(), true);
  if (rc != PRIMA_OK) return rc;
  *t = s;
  return PRIMA_OK;
}

bool is_streamed(const prima_ctx* c, int layer) { return c->n_resident >= 0 && layer >= c->n_resident; }

// Shapes and offsets of a layer's four matrices inside a slot / a pinned host copy.
void stream_layout(prima_ctx* c, TiledMat* qkv, TiledMat* o, TiledMat* gu, TiledMat* down) {
  const prima_model_config& g = c->cfg;
  *qkv = shape_tiled(static_cast<int64_t>(g.n_q_heads + 2 * g.n_kv_heads) * kHeadDim, g.hidden);
  *o = shape_tiled(g.hidden, static_cast<int64_t>(g.n_q_heads) * kHeadDim);
  *gu = shape_tiled(2 * static_cast<int64_t>(g.ffn), g.hidden);
  *down = shape_tiled(g.hidden, g.ffn);
  c->off_o = qkv->bytes();
  c->off_gu = c->off_o + o->bytes();
  c->off_down = c->off_gu + gu->bytes();
  c->layer_bytes = c->off_down + down->bytes();
}

void point_layer_at(prima_ctx* c, Layer& L, uint8_t* base) {
  TiledMat qkv, o, gu, down;
  stream_layout(c, &qkv, &o, &gu, &down);
  qkv.data = base;
  o.data = base ? base + c->off_o : nullptr;
  gu.data = base ? base + c->off_gu : nullptr;
  down.data = base ? base + c->off_down : nullptr;
  L.qkv = qkv; L.o = o; L.gu = gu; L.down = down;
}

// Slots and the copy stream, created when the first streamed layer is loaded.
int ensure_slots(prima_ctx* c) {
  if (!c->slots.empty()) return PRIMA_OK;
  TiledMat a, b, d, e2;
  stream_layout(c, &a, &b, &d, &e2);
  cudaError_t e = cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking);
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaStreamCreate(copy stream)");
  c->slots.resize(c->n_slots);
  for (auto& sl : c->slots) {
    int rc = dev_alloc(c, &sl.dev, c->layer_bytes);
    if (rc != PRIMA_OK) return rc;
    e = cudaEventCreateWithFlags(&sl.copy_done, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&sl.compute_done, cudaEventDisableTiming);
    if (e != cudaSuccess) return cuda_fail(c, e, "cudaEventCreate(slot)");
  }
  return PRIMA_OK;
}

// Add the times of the copies that have completed to the statistics; never waits unless asked to.
void harvest_copy_times(prima_ctx* c, bool wait) {
  size_t kept = 0;
  for (size_t i = 0; i < c->spans_pending.size(); ++i) {
    CopySpan sp = c->spans_pending[i];
    cudaError_t q = wait ? cudaEventSynchronize(sp.t1) : cudaEventQuery(sp.t1);
    if (q == cudaSuccess) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, sp.t0, sp.t1) == cudaSuccess) c->copy_ms += ms;
      c->spans_free.push_back(sp);
    } else {
      c->spans_pending[kept++] = sp;
    }
  }
  c->spans_pending.resize(kept);
}

// Queue, on the copy stream, the copy of streamed layer `l` into slot `s`: after the compute pass that last used
// the slot, one cudaMemcpyAsync per matrix, then the slot's copy_done event.
int queue_layer_copy(prima_ctx* c, int l, int s) {
  StreamSlot& sl = c->slots[s];
  Layer& L = c->layers[l];
  harvest_copy_times(c, false);
  CopySpan sp{nullptr, nullptr};
  cudaError_t e = cudaSuccess;
  if (!c->spans_free.empty()) {
    sp = c->spans_free.back();
    c->spans_free.pop_back();
  } else {
    e = cudaEventCreate(&sp.t0);
    if (e == cudaSuccess) e = cudaEventCreate(&sp.t1);
    if (e != cudaSuccess) return cuda_fail(c, e, "cudaEventCreate(copy span)");
  }
  if (sl.used) e = cudaStreamWaitEvent(c->copy_stream, sl.compute_done, 0);
  if (e == cudaSuccess) e = cudaEventRecord(sp.t0, c->copy_stream);
  const size_t off[5] = {0, c->off_o, c->off_gu, c->off_down, c->layer_bytes};
  for (int i = 0; i < 4 && e == cudaSuccess; ++i)
    e = cudaMemcpyAsync(sl.dev + off[i], L.host + off[i], off[i + 1] - off[i], cudaMemcpyHostToDevice, c->copy_stream);
  if (e == cudaSuccess) e = cudaEventRecord(sp.t1, c->copy_stream);
  if (e == cudaSuccess) e = cudaEventRecord(sl.copy_done, c->copy_stream);
  c->spans_pending.push_back(sp);
  if (e != cudaSuccess) return cuda_fail(c, e, "queueing the copy of a streamed layer");
  sl.layer = l;
  sl.waited = false;
  sl.used = false;
  c->streamed_bytes += static_cast<int64_t>(c->layer_bytes);
  return PRIMA_OK;
}

int slot_of_layer(const prima_ctx* c, int l) {
  for (size_t s = 0; s < c->slots.size(); ++s)
    if (c->slots[s].layer == l) return static_cast<int>(s);
  return -1;
}

// The streamed layer that follows l in the order in which a decoding loop visits them (cyclic).
int next_streamed(const prima_ctx* c, int l) { return l + 1 < c->cfg.n_layers ? l + 1 : c->n_resident; }

// Make streamed layer l's matrices available to the compute stream; returns the slot in *slot.
int acquire_layer(prima_ctx* c, int l, int* slot) {
  int s = slot_of_layer(c, l);
  if (s < 0) {
    // not queued yet (first use, or layers visited out of order): take the slot whose layer comes last in the cyclic
    // order that starts at l
    int best = 0, best_d = -1;
    const int n_str = c->cfg.n_layers - c->n_resident;
    for (size_t i = 0; i < c->slots.size(); ++i) {
      const int other = c->slots[i].layer;
      const int d = other < 0 ? 1 << 30 : ((other - l) % n_str + n_str) % n_str;
      if (d > best_d) { best_d = d; best = static_cast<int>(i); }
    }
    s = best;
    const int rc = queue_layer_copy(c, l, s);
    if (rc != PRIMA_OK) return rc;
  }
  StreamSlot& sl = c->slots[s];
  if (!sl.waited) {
    const cudaError_t e = cudaStreamWaitEvent(c->stream, sl.copy_done, 0);
    if (e != cudaSuccess) return cuda_fail(c, e, "cudaStreamWaitEvent(copy done)");
    sl.waited = true;
  }
  point_layer_at(c, c->layers[l], sl.dev);
  *slot = s;
  return PRIMA_OK;
}

// After layer l's kernels were queued: mark its slot and queue the copies of the streamed layers that follow
// it, as many as there are other slots, so that they stream in while l and its successors compute.
int release_and_prefetch(prima_ctx* c, int l, int slot) {
  StreamSlot& sl = c->slots[slot];
  cudaError_t e = cudaEventRecord(sl.compute_done, c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaEventRecord(compute done)");
  sl.used = true;
  const int n_str = c->cfg.n_layers - c->n_resident;
  int nxt = l;
  for (int k = 1; k < static_cast<int>(c->slots.size()) && k < n_str; ++k) {
    nxt = next_streamed(c, nxt);
    if (slot_of_layer(c, nxt) >= 0) continue;
    // victim: not the slot that layer l is being computed from (a copy into it would have to wait for that
    // computation, and nothing would overlap); of the others, the one whose layer is needed last
    int best = -1, best_d = -1;
    for (size_t i = 0; i < c->slots.size(); ++i) {
      if (static_cast<int>(i) == slot) continue;
      const int other = c->slots[i].layer;
      const int d = other < 0 ? 1 << 30 : ((other - l - 1) % n_str + n_str) % n_str;
      if (d > best_d) { best_d = d; best = static_cast<int>(i); }
    }
    const int rc = queue_layer_copy(c, nxt, best);
    if (rc != PRIMA_OK) return rc;
  }
  return PRIMA_OK;
}

int ensure_kv(prima_ctx* c, int layer) {
  Layer& L = c->layers[layer];
  if (L.k) return PRIMA_OK;
  const size_t n = static_cast<size_t>(c->cfg.n_kv_heads) * c->cfg.kv_capacity * kHeadDim;
  int rc = dev_alloc(c, &L.k, n, true);
  if (rc != PRIMA_OK) return rc;
  return dev_alloc(c, &L.v, n, true);
}

constexpr int kMaxSeqs = 64;

// Cache pointers of (layer, sequence); allocates the sequence's cache on first use.
int ensure_kv_seq(prima_ctx* c, int layer, int seq, __half** k, __half** v) {
  int rc = ensure_kv(c, layer);
  if (rc != PRIMA_OK) return rc;
  Layer& L = c->layers[layer];
  if (seq == 0) {
    *k = L.k;
    *v = L.v;
    return PRIMA_OK;
  }
  if (static_cast<int>(L.k_seq.size()) < seq) {
    L.k_seq.resize(seq, nullptr);
    L.v_seq.resize(seq, nullptr);
  }
  if (!L.k_seq[seq - 1]) {
    const size_t n = static_cast<size_t>(c->cfg.n_kv_heads) * c->cfg.kv_capacity * kHeadDim;
    rc = dev_alloc(c, &L.k_seq[seq - 1], n, true);
    if (rc == PRIMA_OK) rc = dev_alloc(c, &L.v_seq[seq - 1], n, true);
    if (rc != PRIMA_OK) return rc;
  }
  *k = L.k_seq[seq - 1];
  *v = L.v_seq[seq - 1];
  return PRIMA_OK;
}

// Copy a standard-layout matrix (host or device) through the staging buffer and re-tile it.
int load_tiled(prima_ctx* c, TiledMat& dst, const uint8_t* data, int64_t rows, int64_t n_sb, int64_t row0, int64_t stride) {
  const int64_t row_bytes = n_sb * kBlockBytes;
  int64_t rows_per_chunk = std::max<int64_t>(1, static_cast<int64_t>(c->staging_bytes) / row_bytes);
  for (int64_t r = 0; r < rows; r += rows_per_chunk) {
    const int64_t n = std::min(rows_per_chunk, rows - r);
    cudaError_t e = cudaMemcpyAsync(c->staging, data + r * row_bytes, static_cast<size_t>(n * row_bytes), cudaMemcpyDefault, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemcpyAsync(weights)");
    int k = launch_retile(c->staging, n, n_sb, dst, row0 + r * stride, stride, c->stream);
    if (k < 0) return cuda_fail(c, static_cast<cudaError_t>(-k), "retile kernel");
  }
  cudaError_t e = cudaStreamSynchronize(c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaStreamSynchronize(load)");
  return PRIMA_OK;
}

int load_norm(prima_ctx* c, float** dst, float* gmax, const void* data, int64_t cols) {
  std::vector<float> host(static_cast<size_t>(cols));
  cudaError_t e = cudaMemcpy(host.data(), data, static_cast<size_t>(cols) * 4, cudaMemcpyDefault);
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemcpy(norm)");
  float m = 0.f;
  for (float v : host) m = std::max(m, std::fabs(v));
  if (!*dst) {
    int rc = dev_alloc(c, dst, static_cast<size_t>(cols));
    if (rc != PRIMA_OK) return rc;
  }
  e = cudaMemcpy(*dst, host.data(), static_cast<size_t>(cols) * 4, cudaMemcpyHostToDevice);
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemcpy(norm upload)");
  *gmax = m;
  return PRIMA_OK;
}

// Host-side fault injection (PRIMA_OPT_FAIL_AFTER_LAUNCHES): stands in for a launch that the runtime refuses.
inline bool injected_failure(prima_ctx* c) {
  if (c->fail_after < 0) return false;
  if (c->fail_after == 0) {
    c->fail_after = -1;
    return true;
  }
  --c->fail_after;
  return false;
}

#define LAUNCH(c, expr, what)                                                       \
  do {                                                                              \
    if (injected_failure(c)) return fail((c), PRIMA_ERR_CUDA, std::string(what) + ": injected launch failure"); \
    int k_ = (expr);                                                                \
    if (k_ < 0) return cuda_fail((c), static_cast<cudaError_t>(-k_), what);         \
    (c)->launches += k_;                                                            \
  } while (0)

// Same, bracketed by a pair of events when profiling is on.
#define LAUNCH_P(c, klass_, bytes_, expr, what)                                     \
  do {                                                                              \
    prima_ctx::Span sp_{nullptr, nullptr, (klass_), (bytes_), 0};                   \
    if (injected_failure(c)) return fail((c), PRIMA_ERR_CUDA, std::string(what) + ": injected launch failure"); \
    if ((c)->profiling) {                                                           \
      cudaEventCreate(&sp_.a);                                                      \
      cudaEventCreate(&sp_.b);                                                      \
      cudaEventRecord(sp_.a, (c)->stream);                                          \
    }                                                                               \
    int k_ = (expr);                                                                \
    if (k_ < 0) return cuda_fail((c), static_cast<cudaError_t>(-k_), what);         \
    (c)->launches += k_;                                                            \
    if ((c)->profiling) {                                                           \
      cudaEventRecord(sp_.b, (c)->stream);                                          \
      sp_.launches = k_;                                                            \
      (c)->spans.push_back(sp_);                                                    \
    }                                                                               \
  } while (0)

int64_t q4k_bytes(const TiledMat& t) { return t.rows * t.n_sb * kBlockBytes; }

constexpr size_t kMaxStamps = 1 << 15;

// The stamp words of the next launch of a profiled class (mode 2), or nothing.
Stamp next_stamp(prima_ctx* c, int klass, int64_t bytes, int launches, int sub = 0) {
  Stamp s;
  if (!c->stamping || c->stamp_info.size() >= kMaxStamps) return s;
  s.t0 = c->stamp_t0 + c->stamp_info.size();
  s.t1 = c->stamp_t1 + c->stamp_info.size();
  c->stamp_info.push_back({klass, sub, bytes, launches});
  return s;
}

// Queue the clearing of the four accumulator arrays and of the status word: restores the "all zero
// between calls" state after a step that failed half-way or whose kernels reported a failed self-check.
void queue_reset(prima_ctx* c) {
  cudaMemsetAsync(c->acc_qkv, 0, static_cast<size_t>(c->n_acc_qkv) * sizeof(acc_t), c->stream);
  cudaMemsetAsync(c->acc_o, 0, static_cast<size_t>(c->n_acc_o) * sizeof(acc_t), c->stream);
  cudaMemsetAsync(c->acc_gu, 0, static_cast<size_t>(c->n_acc_gu) * sizeof(acc_t), c->stream);
  cudaMemsetAsync(c->acc_down, 0, static_cast<size_t>(c->n_acc_down) * sizeof(acc_t), c->stream);
  cudaMemsetAsync(c->status, 0, sizeof(int), c->stream);
  cudaMemsetAsync(c->attn.tickets, 0, static_cast<size_t>(kMaxTok) * c->cfg.n_kv_heads * sizeof(int), c->stream);
}

}  // namespace

// =============================================================================================
extern "C" {

int prima_ctx_create(const prima_model_config* cfg, void* cuda_stream, prima_ctx** out) {
  if (out) *out = nullptr;
  if (!cfg || !out) return fail(nullptr, PRIMA_ERR_ARG, "prima_ctx_create: null argument");
  const prima_model_config& g = *cfg;
  if (g.n_layers < 1 || g.hidden < 256 || g.hidden % 256 || g.ffn < 256 || g.ffn % 256 || g.head_dim != kHeadDim ||
      g.n_q_heads < 1 || g.n_kv_heads < 1 || g.n_q_heads % g.n_kv_heads || g.n_q_heads / g.n_kv_heads > 8 ||
      g.n_q_heads > kMaxStatBlocks || g.vocab < 1 || g.kv_capacity < 1 || g.max_n_tok < 1 || g.max_n_tok > PRIMA_MAX_N_SEQ ||
      !(g.rms_eps >= 0.f) || !(g.rope_theta > 0.f) || (g.rope_mode != 0 && g.rope_mode != 1) || g.device < 0)
    return fail(nullptr, PRIMA_ERR_ARG, "prima_ctx_create: inconsistent model shape");
  int n_dev = 0;
  cudaError_t e = cudaGetDeviceCount(&n_dev);
  if (e != cudaSuccess) return cuda_fail(nullptr, e, "cudaGetDeviceCount");
  if (g.device >= n_dev) return fail(nullptr, PRIMA_ERR_ARG, "prima_ctx_create: no such device");
  DeviceGuard guard(g.device);
  if (!guard.ok) return fail(nullptr, PRIMA_ERR_CUDA, "cudaSetDevice failed");

  prima_ctx* c = new (std::nothrow) prima_ctx();
  if (!c) return fail(nullptr, PRIMA_ERR_NOMEM, "out of host memory");
  c->cfg = g;
  c->stream = static_cast<cudaStream_t>(cuda_stream);
  c->layers.resize(g.n_layers);
  cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, g.device);

  const int64_t n = g.max_n_tok;
  const int64_t e_ = g.hidden, H = g.n_q_heads, G = g.n_kv_heads, F = g.ffn;
  auto pad8 = [](int64_t r) { return (r + 7) / 8 * 8; };
  c->n_acc_qkv = n * std::max(pad8((H + 2 * G) * kHeadDim), pad8(g.vocab));
  c->n_acc_o = n * pad8(e_);
  c->n_acc_gu = n * pad8(2 * F);
  c->n_acc_down = n * pad8(e_);
  c->attn.max_chunks = (g.kv_capacity + attention_chunk_len() - 1) / attention_chunk_len();
  c->staging_bytes = 256u << 20;

  int rc = PRIMA_OK;
  auto A = [&](int r) { if (rc == PRIMA_OK) rc = r; };
  A(dev_alloc(c, &c->acc_qkv, static_cast<size_t>(c->n_acc_qkv), true));
  A(dev_alloc(c, &c->acc_o, static_cast<size_t>(c->n_acc_o), true));
  A(dev_alloc(c, &c->acc_gu, static_cast<size_t>(c->n_acc_gu), true));
  A(dev_alloc(c, &c->acc_down, static_cast<size_t>(c->n_acc_down), true));
  A(dev_alloc(c, &c->h_a, static_cast<size_t>(n * e_)));
  A(dev_alloc(c, &c->h_b, static_cast<size_t>(n * e_)));
  A(dev_alloc(c, &c->obuf, static_cast<size_t>(n * H * kHeadDim)));
  A(dev_alloc(c, &c->ssq_attn.data, static_cast<size_t>(kMaxTok) * kMaxStatBlocks, true));
  A(dev_alloc(c, &c->ssq_ffn.data, static_cast<size_t>(kMaxTok) * kMaxStatBlocks, true));
  A(dev_alloc(c, &c->ssq_out.data, static_cast<size_t>(kMaxTok) * kMaxStatBlocks, true));
  A(dev_alloc(c, &c->rope_tab, static_cast<size_t>(kMaxTok) * (kHeadDim / 2)));
  A(dev_alloc(c, &c->attn.o_part, static_cast<size_t>(n * H) * c->attn.max_chunks * kHeadDim));
  A(dev_alloc(c, &c->attn.ml_part, static_cast<size_t>(n * H) * c->attn.max_chunks));
  A(dev_alloc(c, &c->attn.tickets, static_cast<size_t>(kMaxTok) * G, true));
  A(dev_alloc(c, &c->staging, c->staging_bytes));
  A(dev_alloc(c, &c->d_tokens, static_cast<size_t>(kMaxTok)));
  A(dev_alloc(c, &c->am_val, static_cast<size_t>(kMaxTok) * kArgmaxBlocks));
  A(dev_alloc(c, &c->am_idx, static_cast<size_t>(kMaxTok) * kArgmaxBlocks));
  A(dev_alloc(c, &c->am_out, static_cast<size_t>(kMaxTok)));
  A(dev_alloc(c, &c->status, 1, true));
  c->attn.status = c->status;
  if (rc != PRIMA_OK) {
    g_tls_error = c->err;
    for (void* p : c->allocs) cudaFree(p);
    delete c;
    return rc;
  }
  *out = c;
  return PRIMA_OK;
}

int prima_ctx_destroy(prima_ctx* c) {
  if (!c) return PRIMA_OK;
  DeviceGuard guard(c->cfg.device);
  cudaStreamSynchronize(c->stream);
  for (auto& sp : c->spans) {
    cudaEventDestroy(sp.a);
    cudaEventDestroy(sp.b);
  }
  if (c->copy_stream) {
    cudaStreamSynchronize(c->copy_stream);
    cudaStreamDestroy(c->copy_stream);
  }
  for (auto& sl : c->slots) {
    if (sl.copy_done) cudaEventDestroy(sl.copy_done);
    if (sl.compute_done) cudaEventDestroy(sl.compute_done);
  }
  for (auto* v : {&c->spans_pending, &c->spans_free})
    for (auto& sp : *v) {
      cudaEventDestroy(sp.t0);
      cudaEventDestroy(sp.t1);
    }
  for (void* p : c->pinned) cudaFreeHost(p);
  for (void* p : c->allocs) cudaFree(p);
  delete c;
  return PRIMA_OK;
}

int prima_load_q4k_weights(prima_ctx* c, int layer, int tensor_id, const void* data, int64_t rows, int64_t cols,
                           int64_t nbytes) {
  if (!c) return fail(nullptr, PRIMA_ERR_ARG, "prima_load_q4k_weights: null context");
  if (!data) return fail(c, PRIMA_ERR_ARG, "prima_load_q4k_weights: null data");
  if (tensor_id < PRIMA_ATTN_NORM || tensor_id > PRIMA_TOK_EMBD) return fail(c, PRIMA_ERR_ARG, "unknown tensor id");
  const prima_model_config& g = c->cfg;
  const bool global = tensor_id >= PRIMA_OUT_NORM;
  if (global ? layer != -1 : (layer < 0 || layer >= g.n_layers)) return fail(c, PRIMA_ERR_ARG, "layer out of range");
  const int64_t e_ = g.hidden, H = g.n_q_heads, G = g.n_kv_heads, F = g.ffn, V = g.vocab;
  int64_t want_rows = 1, want_cols = e_;
  bool is_norm = false;
  switch (tensor_id) {
    case PRIMA_ATTN_NORM: case PRIMA_FFN_NORM: case PRIMA_OUT_NORM: is_norm = true; break;
    case PRIMA_WQ: want_rows = H * kHeadDim; break;
    case PRIMA_WK: case PRIMA_WV: want_rows = G * kHeadDim; break;
    case PRIMA_WO: want_rows = e_; want_cols = H * kHeadDim; break;
    case PRIMA_W_GATE: case PRIMA_W_UP: want_rows = F; break;
    case PRIMA_W_DOWN: want_rows = e_; want_cols = F; break;
    case PRIMA_W_HEAD: case PRIMA_TOK_EMBD: want_rows = V; break;
  }
  if (cols % 256 != 0 && !is_norm) return fail(c, PRIMA_ERR_ARG, "cols must be a multiple of 256");
  if (rows != want_rows || cols != want_cols) return fail(c, PRIMA_ERR_ARG, "tensor shape disagrees with the model config");
  const int64_t want_bytes = is_norm ? cols * 4 : rows * (cols / 256) * kBlockBytes;
  if (nbytes != want_bytes) return fail(c, PRIMA_ERR_ARG, "nbytes disagrees with rows and cols");
  DeviceGuard guard(g.device);

  const uint8_t* bytes = static_cast<const uint8_t*>(data);
  const int64_t n_sb = cols / 256;
  int rc = PRIMA_OK;
  if (global) {
    if (tensor_id == PRIMA_OUT_NORM) {
      rc = load_norm(c, &c->g_out, &c->gmax_out, data, cols);
      if (rc == PRIMA_OK) c->have_out_norm = true;
    } else if (tensor_id == PRIMA_W_HEAD) {
      rc = ensure_tiled(c, &c->head, V, e_);
      if (rc == PRIMA_OK) rc = load_tiled(c, c->head, bytes, rows, n_sb, 0, 1);
      if (rc == PRIMA_OK) c->have_head = true;
    } else {
      if (!c->embd) rc = dev_alloc(c, &c->embd, static_cast<size_t>(nbytes));
      if (rc == PRIMA_OK) {
        cudaError_t e = cudaMemcpy(c->embd, data, static_cast<size_t>(nbytes), cudaMemcpyDefault);
        if (e != cudaSuccess) rc = cuda_fail(c, e, "cudaMemcpy(embedding)");
      }
      if (rc == PRIMA_OK) c->have_embd = true;
    }
    return rc;
  }
  Layer& L = c->layers[layer];
  rc = ensure_kv(c, layer);
  if (rc != PRIMA_OK) return rc;
  const bool matrix = tensor_id != PRIMA_ATTN_NORM && tensor_id != PRIMA_FFN_NORM;
  if (is_streamed(c, layer) && matrix) {
    // A streamed layer is assembled in slot 0 and moved to pinned host memory when its seventh matrix has arrived.
    rc = ensure_slots(c);
    if (rc != PRIMA_OK) return rc;
    if (c->loading_layer != layer) {
      if (c->loading_layer >= 0)
        return fail(c, PRIMA_ERR_STATE, "the matrices of a streamed layer must be loaded layer by layer: layer " +
                                            std::to_string(c->loading_layer) + " is not complete yet");
      cudaError_t e = cudaStreamSynchronize(c->stream);
      if (e == cudaSuccess) e = cudaStreamSynchronize(c->copy_stream);
      if (e == cudaSuccess) e = cudaMemsetAsync(c->slots[0].dev, 0, c->layer_bytes, c->stream);
      if (e != cudaSuccess) return cuda_fail(c, e, "preparing the assembly slot");
      harvest_copy_times(c, true);
      c->slots[0].layer = -1;
      c->slots[0].used = false;
      c->loading_layer = layer;
      L.have &= ~kMatrixMask;
    }
    point_layer_at(c, L, c->slots[0].dev);
  }
  switch (tensor_id) {
    case PRIMA_ATTN_NORM: rc = load_norm(c, &L.g_attn, &L.gmax_attn, data, cols); break;
    case PRIMA_FFN_NORM: rc = load_norm(c, &L.g_ffn, &L.gmax_ffn, data, cols); break;
    case PRIMA_WQ: case PRIMA_WK: case PRIMA_WV: {
      rc = ensure_tiled(c, &L.qkv, (H + 2 * G) * kHeadDim, e_);
      const int64_t row0 = tensor_id == PRIMA_WQ ? 0 : tensor_id == PRIMA_WK ? H * kHeadDim : (H + G) * kHeadDim;
      if (rc == PRIMA_OK) rc = load_tiled(c, L.qkv, bytes, rows, n_sb, row0, 1);
      break;
    }
    case PRIMA_WO:
      rc = ensure_tiled(c, &L.o, e_, H * kHeadDim);
      if (rc == PRIMA_OK) rc = load_tiled(c, L.o, bytes, rows, n_sb, 0, 1);
      break;
    case PRIMA_W_GATE: case PRIMA_W_UP:
      rc = ensure_tiled(c, &L.gu, 2 * F, e_);
      if (rc == PRIMA_OK) rc = load_tiled(c, L.gu, bytes, rows, n_sb, tensor_id == PRIMA_W_GATE ? 0 : 1, 2);
      break;
    case PRIMA_W_DOWN:
      rc = ensure_tiled(c, &L.down, e_, F);
      if (rc == PRIMA_OK) rc = load_tiled(c, L.down, bytes, rows, n_sb, 0, 1);
      break;
  }
  if (rc == PRIMA_OK) L.have |= 1u << tensor_id;
  if (rc == PRIMA_OK && is_streamed(c, layer) && matrix && (L.have & kMatrixMask) == kMatrixMask) {
    if (!L.host) {
      void* hp = nullptr;
      cudaError_t e = cudaHostAlloc(&hp, c->layer_bytes, cudaHostAllocDefault);
      if (e != cudaSuccess) return cuda_fail(c, e, "cudaHostAlloc(streamed layer)");
      c->pinned.push_back(hp);
      L.host = static_cast<uint8_t*>(hp);
    }
    cudaError_t e = cudaMemcpyAsync(L.host, c->slots[0].dev, c->layer_bytes, cudaMemcpyDeviceToHost, c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "moving a streamed layer to pinned host memory");
    c->loading_layer = -1;
    point_layer_at(c, L, nullptr);
  }
  return rc;
}

// One step over layers [layer_begin, layer_end).  seq == nullptr: n_tok tokens of sequence 0 at positions
// pos0 .. pos0 + n_tok - 1, causal among themselves.  Otherwise token t belongs to sequence seq[t] and sits at
// position pos[t] of that sequence's own cache: the products run over all tokens together, attention per token.
static int forward_window_launch(prima_ctx* c, int layer_begin, int layer_end, const float* hidden_in, float* hidden_out, int pos0,
                                 int n_tok, const int32_t* seq, const int32_t* pos);

// Attention reads little and leaves HBM idle, and so does the O product (its matrix is short: the kernel is bound by
// its start-up, not by the stream).  In a step of one token their CTAs ask for the head of the gate/up matrix, the
// long HBM-bound stream that follows, into L2: attention for the first l2_ahead_bytes, the O product for the next
// l2_ahead_o_bytes; by default a sixteenth of the matrix each (measured: larger requests slow attention down by
// more than they save; steps of several tokens are not bound by the stream and gain nothing).
static int64_t ahead_share(const Layer& L, int64_t option) {
  const int64_t all = static_cast<int64_t>(L.gu.bytes());
  return std::min(all, option >= 0 ? option : all / 16 / 16384 * 16384);
}
static L2Ahead attn_ahead(const prima_ctx* c, const Layer& L, int n_tok) {
  L2Ahead a;
  if (n_tok != 1) return a;
  a.ptr[0] = L.gu.data;
  a.bytes[0] = static_cast<unsigned long long>(ahead_share(L, c->l2_ahead_bytes));
  return a;
}
static L2Ahead o_ahead(const prima_ctx* c, const Layer& L, int n_tok) {
  L2Ahead a;
  if (n_tok != 1) return a;
  const int64_t first = ahead_share(L, c->l2_ahead_bytes);
  a.ptr[0] = L.gu.data + first;
  a.bytes[0] = static_cast<unsigned long long>(std::min(static_cast<int64_t>(L.gu.bytes()) - first, ahead_share(L, c->l2_ahead_o_bytes)));
  return a;
}

static int forward_window_impl(prima_ctx* c, int layer_begin, int layer_end, const float* hidden_in, float* hidden_out, int pos0,
                               int n_tok, const int32_t* seq, const int32_t* pos) {
  DeviceGuard guard(c->cfg.device);
  // Everything that can fail without a launch comes first: the caches of the window's (layer, sequence)
  // pairs are allocated here, so that an allocation failure means that nothing was queued.
  if (seq) {
    for (int l = layer_begin; l < layer_end; ++l)
      for (int t = 0; t < n_tok; ++t) {
        __half *k = nullptr, *v = nullptr;
        const int rc = ensure_kv_seq(c, l, seq[t], &k, &v);
        if (rc != PRIMA_OK) return rc;
      }
  }
  const int64_t before = c->launches;
  const int rc = forward_window_launch(c, layer_begin, layer_end, hidden_in, hidden_out, pos0, n_tok, seq, pos);
  // A launch that failed after earlier kernels of the window were queued leaves accumulators that are
  // not zero: clear them behind the queued work, so that the next call starts from the usual state.
  if (rc != PRIMA_OK && c->launches != before) queue_reset(c);
  return rc;
}

static int forward_window_launch(prima_ctx* c, int layer_begin, int layer_end, const float* hidden_in, float* hidden_out, int pos0,
                                 int n_tok, const int32_t* seq, const int32_t* pos) {
  const prima_model_config& g = c->cfg;
  cudaStream_t st = c->stream;
  const int64_t e_ = g.hidden;
  const int H = g.n_q_heads, G = g.n_kv_heads;

  if (layer_begin == layer_end) {
    if (hidden_out != hidden_in) {
      cudaError_t e = cudaMemcpyAsync(hidden_out, hidden_in, static_cast<size_t>(n_tok) * e_ * 4, cudaMemcpyDeviceToDevice, st);
      if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemcpyAsync(hidden_out)");
    }
    return PRIMA_OK;
  }
  if (!seq) {
    LAUNCH(c, launch_rope_table(c->rope_tab, pos0, n_tok, g.rope_theta, st), "rope_table");
  } else {
    for (int t = 0; t < n_tok; ++t)
      LAUNCH(c, launch_rope_table(c->rope_tab + t * (kHeadDim / 2), pos[t], 1, g.rope_theta, st), "rope_table");
  }
  const int64_t mpad_e = (e_ + 7) / 8 * 8;
  // The residual stream entering a layer is h_in plus the value of the previous down projection's
  // accumulators (nothing for the first layer of the call); each product's CTAs finish what they
  // need of their producer's output while staging their activations.  Every accumulator array is
  // cleared by the kernel that follows its last reader: gate/up's by the next QKV product (or the
  // closing kernel), QKV's and down's by the O product, O's by the down product.
  const float* h_in = hidden_in;
  const acc_t* acc_prev = nullptr;
  int first_pos = pos0;
  if (seq)
    for (int t = 0; t < n_tok; ++t) first_pos = t == 0 ? pos[t] : std::min(first_pos, pos[t]);
  const int stable_below = std::min(first_pos, c->unsynced_min_pos);
  c->unsynced_min_pos = stable_below;      // this call appends at first_pos and above
  for (int l = layer_begin; l < layer_end; ++l) {
    Layer& L = c->layers[l];
    int slot = -1;
    if (is_streamed(c, l)) {
      const int rc = acquire_layer(c, l, &slot);
      if (rc != PRIMA_OK) return rc;
    }
    GemvIn in;                                   // QKV: residual (+ down projection of layer l-1) -> h_b
    in.kind = kResidual; in.h_in = h_in; in.h_out = c->h_b; in.acc_in = acc_prev; in.mpad_in = mpad_e;
    in.gain = L.g_attn; in.ssq_out = c->ssq_attn; in.status = c->status; in.first_wait_polls = c->first_wait_polls;
    in.zero0 = c->acc_gu; in.zero0_n = static_cast<int64_t>(n_tok) * L.gu.mpad();
    in.stamp = next_stamp(c, PRIMA_PROF_GEMV, q4k_bytes(L.qkv), 1, PRIMA_PROF_GEMV_QKV);
    LAUNCH_P(c, PRIMA_PROF_GEMV, q4k_bytes(L.qkv), launch_gemv_partials(L.qkv, in, n_tok, c->acc_qkv, c->sm_count, st), "gemv(qkv)");
    c->ssq_attn = in.ssq_out;
    c->ssq_attn.eps = g.rms_eps;
    c->attn.ahead = attn_ahead(c, L, n_tok);
    if (!seq) {
      c->attn.stamp = next_stamp(c, PRIMA_PROF_ATTENTION, static_cast<int64_t>(2) * G * kHeadDim * 2 * (pos0 + n_tok), 2);
      LAUNCH_P(c, PRIMA_PROF_ATTENTION, static_cast<int64_t>(2) * G * kHeadDim * 2 * (pos0 + n_tok),
               launch_attention(c->acc_qkv, L.qkv.mpad(), c->ssq_attn, c->rope_tab, g.rope_mode, L.k, L.v, g.kv_capacity, H, G, pos0, stable_below,
                                n_tok, c->attn, c->obuf, c->sm_count, st), "attention");
    } else {
      AttnSeqs as;                               // one request per token: its own cache, its own position
      as.n = n_tok;
      int64_t kv_bytes = 0;
      for (int t = 0; t < n_tok; ++t) {
        const int rc = ensure_kv_seq(c, l, seq[t], &as.k[t], &as.v[t]);
        if (rc != PRIMA_OK) return rc;
        as.pos[t] = pos[t];
        kv_bytes += static_cast<int64_t>(2) * G * kHeadDim * 2 * (pos[t] + 1);
      }
      c->attn.stamp = next_stamp(c, PRIMA_PROF_ATTENTION, kv_bytes, 2);
      LAUNCH_P(c, PRIMA_PROF_ATTENTION, kv_bytes,
               launch_attention_seqs(c->acc_qkv, L.qkv.mpad(), c->ssq_attn, c->rope_tab, g.rope_mode, as, stable_below, g.kv_capacity, H, G, c->attn,
                                     c->obuf, c->sm_count, st), "attention");
    }
    // Attention leaves HBM idle: its CTAs ask for the O matrix and the head of the gate/up matrix into L2, and the O
    // product, which then finds its weights there, asks for the next stretch of gate/up.
    GemvIn in_o;                                 // O: plain attention output
    in_o.kind = kPlain; in_o.x = c->obuf; in_o.status = c->status; in_o.first_wait_polls = c->first_wait_polls;
    in_o.zero0 = c->acc_qkv; in_o.zero0_n = static_cast<int64_t>(n_tok) * L.qkv.mpad();
    in_o.zero1 = c->acc_down; in_o.zero1_n = static_cast<int64_t>(n_tok) * mpad_e;
    in_o.out_order = kOrderResidual;
    in_o.ahead = o_ahead(c, L, n_tok);
    in_o.stamp = next_stamp(c, PRIMA_PROF_GEMV, q4k_bytes(L.o), 1, PRIMA_PROF_GEMV_O);
    LAUNCH_P(c, PRIMA_PROF_GEMV, q4k_bytes(L.o), launch_gemv_partials(L.o, in_o, n_tok, c->acc_o, c->sm_count, st), "gemv(o)");
    GemvIn in_f;                                 // gate/up: h_b + O projection -> h_a
    in_f.kind = kResidual; in_f.h_in = c->h_b; in_f.h_out = c->h_a; in_f.acc_in = c->acc_o; in_f.mpad_in = L.o.mpad();
    in_f.gain = L.g_ffn; in_f.ssq_out = c->ssq_ffn; in_f.status = c->status; in_f.out_order = kOrderSwiglu; in_f.first_wait_polls = c->first_wait_polls;
    in_f.stamp = next_stamp(c, PRIMA_PROF_GEMV, q4k_bytes(L.gu), 1, PRIMA_PROF_GEMV_GATE_UP);
    LAUNCH_P(c, PRIMA_PROF_GEMV, q4k_bytes(L.gu), launch_gemv_partials(L.gu, in_f, n_tok, c->acc_gu, c->sm_count, st), "gemv(gate/up)");
    c->ssq_ffn = in_f.ssq_out;
    c->ssq_ffn.eps = g.rms_eps;
    GemvIn in_d;                                 // down: SwiGLU of the gate/up product
    in_d.kind = kSwiglu; in_d.acc_in = c->acc_gu; in_d.mpad_in = L.gu.mpad();
    in_d.ssq_in = c->ssq_ffn; in_d.status = c->status; in_d.out_order = kOrderResidual; in_d.first_wait_polls = c->first_wait_polls;
    in_d.zero0 = c->acc_o; in_d.zero0_n = static_cast<int64_t>(n_tok) * L.o.mpad();
    in_d.stamp = next_stamp(c, PRIMA_PROF_GEMV, q4k_bytes(L.down), 1, PRIMA_PROF_GEMV_DOWN);
    LAUNCH_P(c, PRIMA_PROF_GEMV, q4k_bytes(L.down), launch_gemv_partials(L.down, in_d, n_tok, c->acc_down, c->sm_count, st), "gemv(down)");
    h_in = c->h_a;
    acc_prev = c->acc_down;
    if (slot >= 0) {
      const int rc = release_and_prefetch(c, l, slot);
      if (rc != PRIMA_OK) return rc;
    }
  }
  LAUNCH(c, launch_finish_residual(c->acc_down, mpad_e, e_, n_tok, c->h_a, hidden_out, c->acc_gu,
                                   static_cast<int64_t>(n_tok) * c->layers[layer_end - 1].gu.mpad(), st), "finish_residual");
  return PRIMA_OK;
}

static int window_args_ok(prima_ctx* c, const char* who, int layer_begin, int layer_end, const float* hidden_in, float* hidden_out, int n_tok) {
  const prima_model_config& g = c->cfg;
  if (!hidden_in || !hidden_out) return fail(c, PRIMA_ERR_ARG, std::string(who) + ": null hidden pointer");
  if (layer_begin < 0 || layer_end > g.n_layers || layer_begin > layer_end) return fail(c, PRIMA_ERR_ARG, "bad layer range");
  if (n_tok < 1 || n_tok > g.max_n_tok) return fail(c, PRIMA_ERR_ARG, "n_tok outside 1..max_n_tok");
  for (int l = layer_begin; l < layer_end; ++l)
    if ((c->layers[l].have & kLayerMask) != kLayerMask || l == c->loading_layer)
      return fail(c, PRIMA_ERR_STATE, "a layer of the window is not fully loaded");
  return PRIMA_OK;
}

int prima_forward_window(prima_ctx* c, int layer_begin, int layer_end, const float* hidden_in, float* hidden_out, int pos,
                         int n_tok) {
  if (!c) return fail(nullptr, PRIMA_ERR_ARG, "prima_forward_window: null context");
  int rc = window_args_ok(c, "prima_forward_window", layer_begin, layer_end, hidden_in, hidden_out, n_tok);
  if (rc != PRIMA_OK) return rc;
  if (n_tok > PRIMA_MAX_N_TOK) return fail(c, PRIMA_ERR_ARG, "a step of one sequence takes at most 8 tokens");
  if (pos < 0 || static_cast<int64_t>(pos) + n_tok > c->cfg.kv_capacity) return fail(c, PRIMA_ERR_ARG, "pos + n_tok exceeds kv_capacity");
  return forward_window_impl(c, layer_begin, layer_end, hidden_in, hidden_out, pos, n_tok, nullptr, nullptr);
}

int prima_forward_window_seqs(prima_ctx* c, int layer_begin, int layer_end, const float* hidden_in, float* hidden_out,
                              const int32_t* seq, const int32_t* pos, int n_seq) {
  if (!c) return fail(nullptr, PRIMA_ERR_ARG, "prima_forward_window_seqs: null context");
  int rc = window_args_ok(c, "prima_forward_window_seqs", layer_begin, layer_end, hidden_in, hidden_out, n_seq);
  if (rc != PRIMA_OK) return rc;
  if (!seq || !pos) return fail(c, PRIMA_ERR_ARG, "prima_forward_window_seqs: null seq or pos");
  for (int t = 0; t < n_seq; ++t) {
    if (seq[t] < 0 || seq[t] >= kMaxSeqs) return fail(c, PRIMA_ERR_ARG, "sequence id outside 0..63");
    if (pos[t] < 0 || pos[t] >= c->cfg.kv_capacity) return fail(c, PRIMA_ERR_ARG, "position outside the cache");
    for (int u = 0; u < t; ++u)
      if (seq[u] == seq[t]) return fail(c, PRIMA_ERR_ARG, "a sequence may appear once per step");
  }
  return forward_window_impl(c, layer_begin, layer_end, hidden_in, hidden_out, 0, n_seq, seq, pos);
}

int prima_logits(prima_ctx* c, const float* hidden, int n_tok, float* logits) {
  if (!c) return fail(nullptr, PRIMA_ERR_ARG, "prima_logits: null context");
  if (!hidden || !logits) return fail(c, PRIMA_ERR_ARG, "prima_logits: null pointer");
  if (n_tok < 1 || n_tok > c->cfg.max_n_tok) return fail(c, PRIMA_ERR_ARG, "n_tok outside 1..max_n_tok");
  if (!c->have_out_norm || !c->have_head) return fail(c, PRIMA_ERR_STATE, "output norm or head not loaded");
  DeviceGuard guard(c->cfg.device);
  cudaStream_t st = c->stream;
  GemvIn in;        // the head stages hidden itself (no partial sums to add) and leaves its sums of squares
  in.kind = kResidual; in.h_in = hidden; in.h_out = c->h_b; in.acc_in = nullptr;
  in.mpad_in = (c->cfg.hidden + 7) / 8 * 8; in.gain = c->g_out; in.ssq_out = c->ssq_out; in.status = c->status; in.first_wait_polls = c->first_wait_polls;
  in.stamp = next_stamp(c, PRIMA_PROF_GEMV, q4k_bytes(c->head), 1, PRIMA_PROF_GEMV_HEAD);
  LAUNCH_P(c, PRIMA_PROF_GEMV, q4k_bytes(c->head), launch_gemv_partials(c->head, in, n_tok, c->acc_qkv, c->sm_count, st), "gemv(head)");
  c->ssq_out = in.ssq_out;
  c->ssq_out.eps = c->cfg.rms_eps;
  LAUNCH(c, launch_finish_acc(c->acc_qkv, c->head.mpad(), c->cfg.vocab, n_tok, logits, c->ssq_out, st), "finish_acc");
  return PRIMA_OK;
}

int prima_embed(prima_ctx* c, const int32_t* tokens, int n_tok, float* hidden_out) {
  if (!c) return fail(nullptr, PRIMA_ERR_ARG, "prima_embed: null context");
  if (!tokens || !hidden_out) return fail(c, PRIMA_ERR_ARG, "prima_embed: null pointer");
  if (n_tok < 1 || n_tok > c->cfg.max_n_tok) return fail(c, PRIMA_ERR_ARG, "n_tok outside 1..max_n_tok");
  if (!c->have_embd) return fail(c, PRIMA_ERR_STATE, "embedding table not loaded");
  for (int t = 0; t < n_tok; ++t)
    if (tokens[t] < 0 || tokens[t] >= c->cfg.vocab) return fail(c, PRIMA_ERR_ARG, "token id out of range");
  DeviceGuard guard(c->cfg.device);
  cudaError_t e = cudaMemcpyAsync(c->d_tokens, tokens, static_cast<size_t>(n_tok) * 4, cudaMemcpyHostToDevice, c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemcpyAsync(tokens)");
  LAUNCH(c, launch_embed(c->embd, c->cfg.hidden / 256, c->d_tokens, n_tok, hidden_out, c->stream), "embed");
  return PRIMA_OK;
}

int prima_argmax(prima_ctx* c, const float* logits, int n_tok, int32_t* tokens_out) {
  if (!c) return fail(nullptr, PRIMA_ERR_ARG, "prima_argmax: null context");
  if (!logits || !tokens_out) return fail(c, PRIMA_ERR_ARG, "prima_argmax: null pointer");
  if (n_tok < 1 || n_tok > c->cfg.max_n_tok) return fail(c, PRIMA_ERR_ARG, "n_tok outside 1..max_n_tok");
  DeviceGuard guard(c->cfg.device);
  LAUNCH(c, launch_argmax(logits, c->cfg.vocab, n_tok, c->am_val, c->am_idx, c->am_out, c->stream), "argmax");
  cudaError_t e = cudaMemcpyAsync(tokens_out, c->am_out, static_cast<size_t>(n_tok) * 4, cudaMemcpyDeviceToHost, c->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "argmax readback");
  c->unsynced_min_pos = 0x7fffffff;
  return PRIMA_OK;
}

static int kv_args_ok(prima_ctx* c, int layer, int pos_begin, int n_pos, const void* k, const void* v) {
  if (!k || !v) return fail(c, PRIMA_ERR_ARG, "null k or v");
  if (layer < 0 || layer >= c->cfg.n_layers) return fail(c, PRIMA_ERR_ARG, "layer out of range");
  if (pos_begin < 0 || n_pos < 0 || static_cast<int64_t>(pos_begin) + n_pos > c->cfg.kv_capacity)
    return fail(c, PRIMA_ERR_ARG, "position range outside the cache");
  return PRIMA_OK;
}

// Host layout [n_pos][G][128]; device layout [G][capacity][128]: one strided 2-D copy per KV head.
int prima_kv_load(prima_ctx* c, int layer, int pos_begin, int n_pos, const uint16_t* k, const uint16_t* v) {
  return prima_kv_load_seq(c, 0, layer, pos_begin, n_pos, k, v);
}

int prima_kv_read(prima_ctx* c, int layer, int pos_begin, int n_pos, uint16_t* k, uint16_t* v) {
  return prima_kv_read_seq(c, 0, layer, pos_begin, n_pos, k, v);
}

int prima_kv_load_seq(prima_ctx* c, int seq, int layer, int pos_begin, int n_pos, const uint16_t* k, const uint16_t* v) {
  if (!c) return fail(nullptr, PRIMA_ERR_ARG, "prima_kv_load: null context");
  int rc = kv_args_ok(c, layer, pos_begin, n_pos, k, v);
  if (rc != PRIMA_OK) return rc;
  if (seq < 0 || seq >= kMaxSeqs) return fail(c, PRIMA_ERR_ARG, "sequence id outside 0..63");
  DeviceGuard guard(c->cfg.device);
  struct { __half* k; __half* v; } L;
  rc = ensure_kv_seq(c, layer, seq, &L.k, &L.v);
  if (rc != PRIMA_OK) return rc;
  if (n_pos == 0) return PRIMA_OK;
  const int G = c->cfg.n_kv_heads;
  const size_t row = kHeadDim * 2;
  for (int gk = 0; gk < G; ++gk) {
    cudaError_t e = cudaMemcpy2DAsync(L.k + (static_cast<size_t>(gk) * c->cfg.kv_capacity + pos_begin) * kHeadDim, row,
                                      k + static_cast<size_t>(gk) * kHeadDim, row * G, row, n_pos, cudaMemcpyHostToDevice, c->stream);
    if (e == cudaSuccess)
      e = cudaMemcpy2DAsync(L.v + (static_cast<size_t>(gk) * c->cfg.kv_capacity + pos_begin) * kHeadDim, row,
                            v + static_cast<size_t>(gk) * kHeadDim, row * G, row, n_pos, cudaMemcpyHostToDevice, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemcpy2DAsync(kv_load)");
  }
  cudaError_t e = cudaStreamSynchronize(c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "kv_load sync");
  c->unsynced_min_pos = 0x7fffffff;
  return PRIMA_OK;
}

int prima_kv_read_seq(prima_ctx* c, int seq, int layer, int pos_begin, int n_pos, uint16_t* k, uint16_t* v) {
  if (!c) return fail(nullptr, PRIMA_ERR_ARG, "prima_kv_read: null context");
  int rc = kv_args_ok(c, layer, pos_begin, n_pos, k, v);
  if (rc != PRIMA_OK) return rc;
  if (seq < 0 || seq >= kMaxSeqs) return fail(c, PRIMA_ERR_ARG, "sequence id outside 0..63");
  DeviceGuard guard(c->cfg.device);
  struct { __half* k; __half* v; } L;
  rc = ensure_kv_seq(c, layer, seq, &L.k, &L.v);
  if (rc != PRIMA_OK) return rc;
  if (n_pos == 0) return PRIMA_OK;
  const int G = c->cfg.n_kv_heads;
  const size_t row = kHeadDim * 2;
  for (int gk = 0; gk < G; ++gk) {
    cudaError_t e = cudaMemcpy2DAsync(k + static_cast<size_t>(gk) * kHeadDim, row * G,
                                      L.k + (static_cast<size_t>(gk) * c->cfg.kv_capacity + pos_begin) * kHeadDim, row, row, n_pos,
                                      cudaMemcpyDeviceToHost, c->stream);
    if (e == cudaSuccess)
      e = cudaMemcpy2DAsync(v + static_cast<size_t>(gk) * kHeadDim, row * G,
                            L.v + (static_cast<size_t>(gk) * c->cfg.kv_capacity + pos_begin) * kHeadDim, row, row, n_pos,
                            cudaMemcpyDeviceToHost, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "cudaMemcpy2DAsync(kv_read)");
  }
  cudaError_t e = cudaStreamSynchronize(c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "kv_read sync");
  c->unsynced_min_pos = 0x7fffffff;
  return PRIMA_OK;
}

int prima_sync(prima_ctx* c) {
  if (!c) return fail(nullptr, PRIMA_ERR_ARG, "prima_sync: null context");
  DeviceGuard guard(c->cfg.device);
  int status = 0;
  cudaError_t e = cudaMemcpyAsync(&status, c->status, sizeof(int), cudaMemcpyDeviceToHost, c->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "prima_sync");
  c->unsynced_min_pos = 0x7fffffff;
  if (status != 0) {      // reported once; whatever the failed step left in the accumulators is cleared, so the context stays usable
    queue_reset(c);
    e = cudaStreamSynchronize(c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "prima_sync(reset)");
  }
  if (status != 0)
    return fail(c, PRIMA_ERR_DEVICE, (status & 4) ? "an index was outside its array (range-checked build); results of this step are invalid (status " + std::to_string(status) + ")"
                                     : !(status & 1) ? "a partial sum was outside the accumulator range (+-2^27); results of this step are invalid"
                                                 : "a bounded wait inside a kernel gave up (status " + std::to_string(status) + ")");
  return PRIMA_OK;
}

int prima_ctx_set_option(prima_ctx* c, int option, int64_t value) {
  if (!c) return fail(nullptr, PRIMA_ERR_ARG, "prima_ctx_set_option: null context");
  switch (option) {
    case PRIMA_OPT_FIRST_WAIT_POLLS:
      if (value < -1 || value > (int64_t(1) << 30)) return fail(c, PRIMA_ERR_ARG, "PRIMA_OPT_FIRST_WAIT_POLLS: value outside -1 .. 2^30");
      c->first_wait_polls = value < 0 ? 0u : static_cast<uint32_t>(value) + 1u;
      return PRIMA_OK;
    case PRIMA_OPT_RESIDENT_LAYERS:
    case PRIMA_OPT_STREAM_SLOTS: {
      for (const Layer& L : c->layers)
        if (L.have & kMatrixMask) return fail(c, PRIMA_ERR_STATE, "residency options must be set before any layer matrix is loaded");
      if (option == PRIMA_OPT_RESIDENT_LAYERS) {
        if (value < -1 || value > c->cfg.n_layers) return fail(c, PRIMA_ERR_ARG, "PRIMA_OPT_RESIDENT_LAYERS: value outside -1 .. n_layers");
        c->n_resident = value == c->cfg.n_layers ? -1 : static_cast<int>(value);
      } else {
        if (value < 2 || value > 16) return fail(c, PRIMA_ERR_ARG, "PRIMA_OPT_STREAM_SLOTS: value outside 2 .. 16");
        if (!c->slots.empty()) return fail(c, PRIMA_ERR_STATE, "the slots exist already");
        c->n_slots = static_cast<int>(value);
      }
      return PRIMA_OK;
    }
    case PRIMA_OPT_L2_AHEAD_BYTES:
    case PRIMA_OPT_L2_AHEAD_O_BYTES:
      if (value < -1 || value > (int64_t(1) << 30) || (value > 0 && value % 16 != 0)) return fail(c, PRIMA_ERR_ARG, "PRIMA_OPT_L2_AHEAD_*: -1 or a multiple of 16 in 0 .. 2^30");
      (option == PRIMA_OPT_L2_AHEAD_BYTES ? c->l2_ahead_bytes : c->l2_ahead_o_bytes) = value;
      return PRIMA_OK;
    case PRIMA_OPT_FAIL_AFTER_LAUNCHES:
      if (value < -1) return fail(c, PRIMA_ERR_ARG, "PRIMA_OPT_FAIL_AFTER_LAUNCHES: value below -1");
      c->fail_after = value;
      return PRIMA_OK;
    default:
      return fail(c, PRIMA_ERR_ARG, "prima_ctx_set_option: unknown option");
  }
}

int prima_stream_stats(prima_ctx* c, int64_t* bytes_copied, double* copy_ms) {
  if (!c || !bytes_copied || !copy_ms) return fail(c, PRIMA_ERR_ARG, "prima_stream_stats: null argument");
  DeviceGuard guard(c->cfg.device);
  if (c->copy_stream) {
    cudaError_t e = cudaStreamSynchronize(c->copy_stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "prima_stream_stats");
    harvest_copy_times(c, true);
  }
  *bytes_copied = c->streamed_bytes;
  *copy_ms = c->copy_ms;
  return PRIMA_OK;
}

int prima_profile_enable(prima_ctx* c, int mode) {
  if (!c) return fail(nullptr, PRIMA_ERR_ARG, "prima_profile_enable: null context");
  if (mode < 0 || mode > 2) return fail(c, PRIMA_ERR_ARG, "prima_profile_enable: mode must be 0, 1 or 2");
  DeviceGuard guard(c->cfg.device);
  cudaStreamSynchronize(c->stream);
  for (auto& sp : c->spans) {
    cudaEventDestroy(sp.a);
    cudaEventDestroy(sp.b);
  }
  c->spans.clear();
  c->stamp_info.clear();
  c->profiling = mode == 1;
  c->stamping = false;
  if (mode == 2) {
    if (!c->stamp_t0) {
      int rc = dev_alloc(c, &c->stamp_t0, kMaxStamps);
      if (rc == PRIMA_OK) rc = dev_alloc(c, &c->stamp_t1, kMaxStamps);
      if (rc != PRIMA_OK) return rc;
    }
    cudaError_t e = cudaMemsetAsync(c->stamp_t0, 0xff, kMaxStamps * sizeof(unsigned long long), c->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->stamp_t1, 0, kMaxStamps * sizeof(unsigned long long), c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e, "prima_profile_enable");
    c->stamping = true;
  }
  c->attn.stamp = Stamp();
  return PRIMA_OK;
}

int prima_profile_read(prima_ctx* c, int klass, double* ms_total, int64_t* launches, int64_t* algo_bytes) {
  if (!c || !ms_total || !launches || !algo_bytes) return fail(c, PRIMA_ERR_ARG, "prima_profile_read: null argument");
  DeviceGuard guard(c->cfg.device);
  cudaError_t e = cudaStreamSynchronize(c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e, "prima_profile_read");
  double ms = 0;
  int64_t n = 0, bytes = 0;
  for (auto& sp : c->spans) {
    if (sp.klass != klass) continue;
    float t = 0.f;
    e = cudaEventElapsedTime(&t, sp.a, sp.b);
    if (e != cudaSuccess) return cuda_fail(c, e, "cudaEventElapsedTime");
    ms += t;
    n += sp.launches;
    bytes += sp.bytes;
  }
  if (!c->stamp_info.empty()) {
    const size_t k = c->stamp_info.size();
    std::vector<unsigned long long> t0(k), t1(k);
    e = cudaMemcpy(t0.data(), c->stamp_t0, k * sizeof(unsigned long long), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess) e = cudaMemcpy(t1.data(), c->stamp_t1, k * sizeof(unsigned long long), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(c, e, "prima_profile_read(stamps)");
    for (size_t i = 0; i < k; ++i) {
      const bool match = c->stamp_info[i].klass == klass || (c->stamp_info[i].klass == PRIMA_PROF_GEMV && c->stamp_info[i].sub == klass);
      if (!match || t1[i] <= t0[i]) continue;
      ms += static_cast<double>(t1[i] - t0[i]) * 1e-6;
      n += c->stamp_info[i].launches;
      bytes += c->stamp_info[i].bytes;
    }
  }
  *ms_total = ms;
  *launches = n;
  *algo_bytes = bytes;
  return PRIMA_OK;
}

const char* prima_last_error(prima_ctx* c) { return c ? c->err.c_str() : g_tls_error.c_str(); }

int64_t prima_launch_count(prima_ctx* c) { return c ? c->launches : 0; }

// ---- context-free primitives ------------------------------------------------------------------
int prima_dequant_q4k(const void* dev_blocks, int64_t n_superblocks, float* dev_out, void* stream) {
  if (n_superblocks == 0) return PRIMA_OK;
  if (!dev_blocks || !dev_out || n_superblocks < 0) return fail(nullptr, PRIMA_ERR_ARG, "prima_dequant_q4k: bad argument");
  int k = launch_dequant_std(static_cast<const uint8_t*>(dev_blocks), n_superblocks, dev_out, static_cast<cudaStream_t>(stream));
  if (k < 0) return cuda_fail(nullptr, static_cast<cudaError_t>(-k), "dequant kernel");
  return PRIMA_OK;
}

int prima_gemv_plan_create(const void* dev_w, int64_t rows, int64_t cols, int max_n_cols, prima_gemv_plan** out) {
  if (out) *out = nullptr;
  if (!dev_w || !out || rows < 1 || cols < 256 || cols % 256 || max_n_cols < 1 || max_n_cols > PRIMA_MAX_N_SEQ)
    return fail(nullptr, PRIMA_ERR_ARG, "prima_gemv_plan_create: bad argument");
  prima_gemv_plan* p = new (std::nothrow) prima_gemv_plan();
  if (!p) return fail(nullptr, PRIMA_ERR_NOMEM, "out of host memory");
  cudaGetDevice(&p->device);
  cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device);
  p->max_n_cols = max_n_cols;
  p->w = shape_tiled(rows, cols);
  cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&p->w.data), p->w.bytes());
  if (e == cudaSuccess) e = cudaMemset(p->w.data, 0, p->w.bytes());
  const size_t acc_bytes = static_cast<size_t>(max_n_cols) * p->w.mpad() * sizeof(acc_t);
  if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&p->acc), acc_bytes);
  if (e == cudaSuccess) e = cudaMemset(p->acc, 0, acc_bytes);
  if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&p->status), sizeof(int));
  if (e == cudaSuccess) e = cudaMemset(p->status, 0, sizeof(int));
  if (e == cudaSuccess) {
    int k = launch_retile(static_cast<const uint8_t*>(dev_w), rows, p->w.n_sb, p->w, 0, 1, nullptr);
    if (k < 0) e = static_cast<cudaError_t>(-k);
  }
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    prima_gemv_plan_destroy(p);
    return cuda_fail(nullptr, e, "prima_gemv_plan_create");
  }
  *out = p;
  return PRIMA_OK;
}

int prima_gemv_plan_run(prima_gemv_plan* p, const float* dev_x, int n_cols, float* dev_y, void* stream) {
  if (!p || !dev_x || !dev_y || n_cols < 1 || n_cols > p->max_n_cols) return fail(nullptr, PRIMA_ERR_ARG, "prima_gemv_plan_run: bad argument");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  GemvIn in;
  in.kind = kPlain; in.x = dev_x; in.status = p->status;
  int k = launch_gemv_partials(p->w, in, n_cols, p->acc, p->sm_count, st);
  if (k < 0) return cuda_fail(nullptr, static_cast<cudaError_t>(-k), "gemv kernel");
  k = launch_finish_acc(p->acc, p->w.mpad(), p->w.rows, n_cols, dev_y, SumSq(), st);
  if (k < 0) return cuda_fail(nullptr, static_cast<cudaError_t>(-k), "finish kernel");
  return PRIMA_OK;
}

int prima_gemv_plan_destroy(prima_gemv_plan* p) {
  if (!p) return PRIMA_OK;
  cudaFree(p->w.data);
  cudaFree(p->acc);
  cudaFree(p->status);
  delete p;
  return PRIMA_OK;
}

int prima_gemv_q4k(const void* dev_w, int64_t rows, int64_t cols, const float* dev_x, int n_cols, float* dev_y, void* stream) {
  if (!dev_x || !dev_y || n_cols < 1 || n_cols > PRIMA_MAX_N_SEQ) return fail(nullptr, PRIMA_ERR_ARG, "prima_gemv_q4k: bad argument");
  prima_gemv_plan* p = nullptr;
  int rc = prima_gemv_plan_create(dev_w, rows, cols, n_cols, &p);
  if (rc != PRIMA_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  rc = prima_gemv_plan_run(p, dev_x, n_cols, dev_y, st);
  cudaError_t e = cudaStreamSynchronize(st);
  int status = 0;
  if (e == cudaSuccess) e = cudaMemcpy(&status, p->status, sizeof(int), cudaMemcpyDeviceToHost);
  prima_gemv_plan_destroy(p);
  if (rc != PRIMA_OK) return rc;
  if (e != cudaSuccess) return cuda_fail(nullptr, e, "prima_gemv_q4k");
  if (status != 0)
    return fail(nullptr, PRIMA_ERR_DEVICE, !(status & 1) ? "prima_gemv_q4k: a partial sum is outside the accumulator range (+-2^27)"
                                                       : "prima_gemv_q4k: a bounded wait inside the kernel gave up");
  return PRIMA_OK;
}

}  // extern "C"
