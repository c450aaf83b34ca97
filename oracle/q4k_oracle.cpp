// CPU oracle for the Q4_K layer-window forward pass.  TEST INFRASTRUCTURE ONLY.
//
// This file is a plain, slow, fp64 restatement of what the GPU library computes.  It exists so
// that tests, the smoke check and the benchmark's CPU-baseline leg have something independent to
// compare against and to time.  It shares no code, header, table or helper with the CUDA path,
// and the product never calls it.
//
// What it follows.  The paper fixes the *shape* of the computation: a model is cut into
// contiguous layer windows (Section 3.1; Appendix A.12, "Mmap- and prefetch-based PRP"); what
// crosses a window boundary is the hidden state, e fp32 values per token (Appendix A.3,
// communication latency); every layer owns an fp16 KV cache that grows by 2(h_k e_k + h_v e_v)
// bytes per token (Appendix A.3, KV cache copy time); the input layer is a lookup table and the
// output layer produces logits on the head device (Appendix A.3, computation latency); draft
// tokens are verified by the target model in one batch (Section "Run Prima.cpp with Speculative
// Decoding"; Appendix A.12).  The paper names the weight format (Q4K) but does not print its bit
// layout or the layer arithmetic; the reading adopted here is the 144-byte super-block
// (fp16 d, fp16 dmin, 12 bytes of 6-bit scales/mins, 128 bytes of nibbles) with
// w = d*sc*q - dmin*m, and a Llama-style layer (RMSNorm, rotary embedding, grouped-query
// attention, SwiGLU).  Both PRP and speculative verification leave outputs unchanged, so the
// oracle is the plain definition: dequantise, then dense math in double precision.
//
// Storage roundings that are part of the definition (everything else is fp64):
//   * hidden state -> fp32 after each residual addition,
//   * K and V      -> fp16 (round to nearest even) when appended to the cache; attention reads
//                     the rounded values, including the current token's,
//   * logits       -> fp32.
//
// Pins (tests/test_oracle_*.py): hand-built super-blocks with known values, bit-toggle test of
// the 12 scale bytes, brute-force dense dot products written in numpy, fp16 conversion against
// numpy's float16 over all 65536 patterns, RMSNorm / RoPE / softmax closed forms and invariants,
// the window-split invariant, n-token step == n single-token steps.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <functional>
#include <limits>
#include <string>
#include <thread>
#include <vector>

namespace {

constexpr int kSuperBlock = 256;      // weights per super-block
constexpr int kBlockBytes = 144;      // bytes per super-block

// ---------------------------------------------------------------------------------------------
// IEEE binary16 <-> double, written from the format definition (1 sign, 5 exponent, 10 fraction).
// ---------------------------------------------------------------------------------------------
double half_bits_to_double(uint16_t bits) {
  const int sign = bits >> 15;
  const int expo = (bits >> 10) & 0x1f;
  const int frac = bits & 0x3ff;
  double v;
  if (expo == 0) {
    v = std::ldexp(static_cast<double>(frac), -24);            // subnormal: frac * 2^-24
  } else if (expo == 31) {
    v = frac ? std::numeric_limits<double>::quiet_NaN() : std::numeric_limits<double>::infinity();
  } else {
    v = std::ldexp(1.0 + static_cast<double>(frac) / 1024.0, expo - 15);
  }
  return sign ? -v : v;
}

// Round a double to the nearest binary16 value, ties to even.  Works on the exact value: scale so
// that one unit equals the spacing of binary16 numbers around |v|, round to an integer with
// ties-to-even, rebuild.
uint16_t double_to_half_bits(double v) {
  const uint16_t sign = std::signbit(v) ? 0x8000 : 0;
  if (std::isnan(v)) return sign | 0x7e00;
  double a = std::fabs(v);
  if (std::isinf(a)) return sign | 0x7c00;
  if (a == 0.0) return sign;
  int e;
  std::frexp(a, &e);                 // a = f * 2^e, f in [0.5, 1)  ->  a in [2^(e-1), 2^e)
  int unit_exp = (e - 1) - 10;       // spacing of binary16 in this binade is 2^(e-1-10)
  if (unit_exp < -24) unit_exp = -24;  // subnormal spacing
  const double scaled = std::ldexp(a, -unit_exp);   // exact (power-of-two scaling)
  double r = std::nearbyint(scaled);                // default rounding mode: nearest even
  // r is in [0, 2048]; rebuild the value and re-derive the fields.
  const double rounded = std::ldexp(r, unit_exp);
  if (rounded >= 65520.0) return sign | 0x7c00;     // beyond the largest finite value + half ulp
  if (rounded == 0.0) return sign;
  int e2;
  std::frexp(rounded, &e2);
  const int biased = (e2 - 1) + 15;
  if (biased <= 0) {                                // subnormal result
    const int frac = static_cast<int>(std::ldexp(rounded, 24));
    return sign | static_cast<uint16_t>(frac);
  }
  const int frac = static_cast<int>(std::ldexp(rounded, 10 - (e2 - 1))) - 1024;
  return sign | static_cast<uint16_t>((biased << 10) | frac);
}

// ---------------------------------------------------------------------------------------------
// Q4_K super-block fields.
//   byte 0..1   d     (binary16, little endian)
//   byte 2..3   dmin  (binary16, little endian)
//   byte 4..15  s[0..11]: eight 6-bit scales sc_j and eight 6-bit mins m_j
//   byte 16..143 qs[0..127]: for p = 0..3 and i = 0..31, byte qs[32p+i] holds weight 64p+i in
//               its low nibble (sub-block 2p) and weight 64p+32+i in its high nibble (2p+1)
// ---------------------------------------------------------------------------------------------
struct Fields {
  double d, dmin;
  int sc[8], m[8];
};

Fields read_fields(const uint8_t* sb) {
  Fields f;
  f.d = half_bits_to_double(static_cast<uint16_t>(sb[0] | (sb[1] << 8)));
  f.dmin = half_bits_to_double(static_cast<uint16_t>(sb[2] | (sb[3] << 8)));
  const uint8_t* s = sb + 4;
  for (int j = 0; j < 8; ++j) {
    if (j < 4) {
      f.sc[j] = s[j] & 63;
      f.m[j] = s[j + 4] & 63;
    } else {
      f.sc[j] = (s[j + 4] & 15) | ((s[j - 4] >> 6) << 4);
      f.m[j] = (s[j + 4] >> 4) | ((s[j] >> 6) << 4);
    }
  }
  return f;
}

// Dequantise one super-block: w_k = d*sc_j*q_k - dmin*m_j with j = k / 32.  Both products are
// exact in double (at most 21 significant bits each), so the only rounding is the subtraction's,
// and that is exact too whenever the result fits 53 bits, which it always does here.
void block_values(const uint8_t* sb, double* out256) {
  const Fields f = read_fields(sb);
  const uint8_t* qs = sb + 16;
  for (int p = 0; p < 4; ++p) {
    const int jlo = 2 * p, jhi = 2 * p + 1;
    const double slo = f.d * static_cast<double>(f.sc[jlo]), olo = f.dmin * static_cast<double>(f.m[jlo]);
    const double shi = f.d * static_cast<double>(f.sc[jhi]), ohi = f.dmin * static_cast<double>(f.m[jhi]);
    for (int i = 0; i < 32; ++i) {
      const uint8_t byte = qs[32 * p + i];
      out256[64 * p + i] = slo * static_cast<double>(byte & 15) - olo;
      out256[64 * p + 32 + i] = shi * static_cast<double>(byte >> 4) - ohi;
    }
  }
}

void parallel_for(int64_t n, int n_threads, const std::function<void(int64_t, int64_t)>& body) {
  if (n_threads <= 1 || n < 2) {
    body(0, n);
    return;
  }
  const int64_t t = std::min<int64_t>(n_threads, n);
  std::vector<std::thread> pool;
  for (int64_t i = 0; i < t; ++i) {
    const int64_t lo = n * i / t, hi = n * (i + 1) / t;
    pool.emplace_back([=, &body] { body(lo, hi); });
  }
  for (auto& th : pool) th.join();
}

// y[c][r] = sum_k w[r][k] * x[c][k], in index order, fp64.  s_abs (optional) gets sum |w*x|.
void gemv_rows(const uint8_t* w, int64_t rows, int64_t cols, const double* x, int n_cols,
               double* y, double* s_abs, int n_threads) {
  const int64_t n_sb = cols / kSuperBlock;
  parallel_for(rows, n_threads, [&](int64_t lo, int64_t hi) {
    std::vector<double> wrow(static_cast<size_t>(cols));
    for (int64_t r = lo; r < hi; ++r) {
      const uint8_t* row = w + r * n_sb * kBlockBytes;
      for (int64_t b = 0; b < n_sb; ++b) {
        const uint8_t* sb = row + b * kBlockBytes;
        block_values(sb, &wrow[b * kSuperBlock]);
      }
      for (int c = 0; c < n_cols; ++c) {
        const double* xc = x + static_cast<int64_t>(c) * cols;
        double acc = 0.0, abs_acc = 0.0;
        for (int64_t k = 0; k < cols; ++k) {
          const double t = wrow[k] * xc[k];
          acc += t;
          abs_acc += std::fabs(t);
        }
        y[static_cast<int64_t>(c) * rows + r] = acc;
        if (s_abs) s_abs[static_cast<int64_t>(c) * rows + r] = abs_acc;
      }
    }
  });
}

void rmsnorm(const double* h, const float* g, int64_t n, double eps, double* out) {
  double ss = 0.0;
  for (int64_t i = 0; i < n; ++i) ss += h[i] * h[i];
  const double inv = 1.0 / std::sqrt(ss / static_cast<double>(n) + eps);
  for (int64_t i = 0; i < n; ++i) out[i] = h[i] * inv * static_cast<double>(g[i]);
}

// Rotary embedding of one head vector of length D at position pos.
// mode 0: pairs (i, i + D/2); mode 1: pairs (2i, 2i+1).  Angle = pos * theta^(-2i/D).
void rope_head(double* v, int D, int64_t pos, double theta, int mode) {
  const int half = D / 2;
  for (int i = 0; i < half; ++i) {
    const double phi = static_cast<double>(pos) * std::pow(theta, -2.0 * i / static_cast<double>(D));
    const double c = std::cos(phi), s = std::sin(phi);
    const int a = mode == 0 ? i : 2 * i;
    const int b = mode == 0 ? i + half : 2 * i + 1;
    const double xa = v[a], xb = v[b];
    v[a] = xa * c - xb * s;
    v[b] = xb * c + xa * s;
  }
}

// One query head against n_ctx cached positions of one KV head (fp16 bit patterns, position-major
// with `stride` halves between consecutive positions).  Naive softmax with max subtraction.
void attend_one(const double* q, const uint16_t* kc, const uint16_t* vc, int64_t n_ctx,
                int64_t stride, int D, double* out) {
  std::vector<double> s(static_cast<size_t>(n_ctx));
  const double scale = 1.0 / std::sqrt(static_cast<double>(D));
  double mx = -std::numeric_limits<double>::infinity();
  for (int64_t j = 0; j < n_ctx; ++j) {
    double dot = 0.0;
    for (int i = 0; i < D; ++i) dot += q[i] * half_bits_to_double(kc[j * stride + i]);
    s[j] = dot * scale;
    mx = std::max(mx, s[j]);
  }
  double denom = 0.0;
  for (int64_t j = 0; j < n_ctx; ++j) {
    s[j] = std::exp(s[j] - mx);
    denom += s[j];
  }
  for (int i = 0; i < D; ++i) {
    double acc = 0.0;
    for (int64_t j = 0; j < n_ctx; ++j) acc += s[j] * half_bits_to_double(vc[j * stride + i]);
    out[i] = acc / denom;
  }
}

inline double silu(double z) { return z / (1.0 + std::exp(-z)); }

// ---------------------------------------------------------------------------------------------
// Model context
// ---------------------------------------------------------------------------------------------
enum TensorId {
  T_ATTN_NORM = 0, T_WQ, T_WK, T_WV, T_WO, T_FFN_NORM, T_W_GATE, T_W_UP, T_W_DOWN,
  T_OUT_NORM, T_W_HEAD, T_TOK_EMBD, T_COUNT
};

struct Tensor {
  std::vector<uint8_t> own;
  const uint8_t* data = nullptr;
  int64_t rows = 0, cols = 0;
  bool loaded() const { return data != nullptr; }
};

struct Config {
  int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab;
  int32_t kv_capacity, max_n_tok;
  float rms_eps, rope_theta;
  int32_t rope_mode;
};

struct Ctx {
  Config cfg;
  std::vector<std::vector<Tensor>> layer;   // [n_layers][9]
  Tensor out_norm, w_head, tok_embd;
  // KV cache per layer: [kv_capacity][n_kv_heads][head_dim] fp16 bit patterns
  std::vector<std::vector<uint16_t>> kcache, vcache;
  std::string err;
};

bool layer_ready(const Ctx& c, int l) {
  for (int t = T_ATTN_NORM; t <= T_W_DOWN; ++t)
    if (!c.layer[l][t].loaded()) return false;
  return true;
}

void project(const Tensor& w, const std::vector<double>& x, int n_tok, std::vector<double>& y,
             int n_threads) {
  y.assign(static_cast<size_t>(n_tok) * w.rows, 0.0);
  gemv_rows(w.data, w.rows, w.cols, x.data(), n_tok, y.data(), nullptr, n_threads);
}

// One transformer layer for n_tok tokens at positions pos..pos+n_tok-1.  h is [n_tok][hidden],
// fp32 on entry and on exit.
void layer_forward(Ctx& c, int l, std::vector<float>& h, int64_t pos, int n_tok, int n_threads) {
  const Config& g = c.cfg;
  const int e = g.hidden, H = g.n_q_heads, G = g.n_kv_heads, D = g.head_dim, F = g.ffn;
  const int group = H / G;
  auto& L = c.layer[l];
  const float* g_attn = reinterpret_cast<const float*>(L[T_ATTN_NORM].data);
  const float* g_ffn = reinterpret_cast<const float*>(L[T_FFN_NORM].data);

  std::vector<double> hd(h.begin(), h.end());
  std::vector<double> a(static_cast<size_t>(n_tok) * e);
  for (int t = 0; t < n_tok; ++t) rmsnorm(&hd[static_cast<size_t>(t) * e], g_attn, e, g.rms_eps, &a[static_cast<size_t>(t) * e]);

  std::vector<double> q, k, v;
  project(L[T_WQ], a, n_tok, q, n_threads);     // [n_tok][H*D]
  project(L[T_WK], a, n_tok, k, n_threads);     // [n_tok][G*D]
  project(L[T_WV], a, n_tok, v, n_threads);

  // Rotate q and k, append rounded k and v at positions pos+t.
  for (int t = 0; t < n_tok; ++t) {
    const int64_t p = pos + t;
    for (int hh = 0; hh < H; ++hh) rope_head(&q[(static_cast<size_t>(t) * H + hh) * D], D, p, g.rope_theta, g.rope_mode);
    for (int gg = 0; gg < G; ++gg) rope_head(&k[(static_cast<size_t>(t) * G + gg) * D], D, p, g.rope_theta, g.rope_mode);
    uint16_t* kd = &c.kcache[l][static_cast<size_t>(p) * G * D];
    uint16_t* vd = &c.vcache[l][static_cast<size_t>(p) * G * D];
    for (int i = 0; i < G * D; ++i) {
      kd[i] = double_to_half_bits(k[static_cast<size_t>(t) * G * D + i]);
      vd[i] = double_to_half_bits(v[static_cast<size_t>(t) * G * D + i]);
    }
  }

  // Attention: token t sees cache positions 0..pos+t.
  std::vector<double> o(static_cast<size_t>(n_tok) * H * D);
  parallel_for(static_cast<int64_t>(n_tok) * H, n_threads, [&](int64_t lo, int64_t hi) {
    for (int64_t idx = lo; idx < hi; ++idx) {
      const int t = static_cast<int>(idx / H), hh = static_cast<int>(idx % H);
      const int gg = hh / group;
      attend_one(&q[(static_cast<size_t>(t) * H + hh) * D], &c.kcache[l][static_cast<size_t>(gg) * D],
                 &c.vcache[l][static_cast<size_t>(gg) * D], pos + t + 1, static_cast<int64_t>(G) * D, D,
                 &o[(static_cast<size_t>(t) * H + hh) * D]);
    }
  });

  std::vector<double> proj;
  project(L[T_WO], o, n_tok, proj, n_threads);  // [n_tok][e]
  for (size_t i = 0; i < h.size(); ++i) h[i] = static_cast<float>(hd[i] + proj[i]);

  // Feed-forward
  for (size_t i = 0; i < h.size(); ++i) hd[i] = h[i];
  for (int t = 0; t < n_tok; ++t) rmsnorm(&hd[static_cast<size_t>(t) * e], g_ffn, e, g.rms_eps, &a[static_cast<size_t>(t) * e]);
  std::vector<double> gate, up, act(static_cast<size_t>(n_tok) * F), down;
  project(L[T_W_GATE], a, n_tok, gate, n_threads);
  project(L[T_W_UP], a, n_tok, up, n_threads);
  for (size_t i = 0; i < act.size(); ++i) act[i] = silu(gate[i]) * up[i];
  project(L[T_W_DOWN], act, n_tok, down, n_threads);
  for (size_t i = 0; i < h.size(); ++i) h[i] = static_cast<float>(hd[i] + down[i]);
}

}  // namespace

// =============================================================================================
// C interface (host memory only)
// =============================================================================================
extern "C" {

double orc_half_to_double(uint16_t bits) { return half_bits_to_double(bits); }
uint16_t orc_double_to_half(double v) { return double_to_half_bits(v); }

// Decode the header of one super-block: d, dmin and the sixteen 6-bit fields.
void orc_q4k_fields(const uint8_t* sb, double* d, double* dmin, int32_t* sc8, int32_t* m8) {
  const Fields f = read_fields(sb);
  *d = f.d;
  *dmin = f.dmin;
  for (int j = 0; j < 8; ++j) {
    sc8[j] = f.sc[j];
    m8[j] = f.m[j];
  }
}

// Build one super-block from its fields (inverse of the decode above).
void orc_q4k_pack(uint16_t d_bits, uint16_t dmin_bits, const int32_t* sc8, const int32_t* m8,
                  const uint8_t* q256, uint8_t* out144) {
  std::memset(out144, 0, kBlockBytes);
  out144[0] = d_bits & 0xff;
  out144[1] = d_bits >> 8;
  out144[2] = dmin_bits & 0xff;
  out144[3] = dmin_bits >> 8;
  uint8_t* s = out144 + 4;
  for (int j = 0; j < 4; ++j) {
    s[j] = static_cast<uint8_t>((sc8[j] & 63) | ((sc8[j + 4] >> 4) << 6));
    s[j + 4] = static_cast<uint8_t>((m8[j] & 63) | ((m8[j + 4] >> 4) << 6));
    s[j + 8] = static_cast<uint8_t>((sc8[j + 4] & 15) | ((m8[j + 4] & 15) << 4));
  }
  for (int p = 0; p < 4; ++p)
    for (int i = 0; i < 32; ++i)
      out144[16 + 32 * p + i] = static_cast<uint8_t>((q256[64 * p + i] & 15) | ((q256[64 * p + 32 + i] & 15) << 4));
}

void orc_q4k_dequant_f64(const uint8_t* blocks, int64_t n_sb, double* out) {
  for (int64_t b = 0; b < n_sb; ++b) {
    block_values(blocks + b * kBlockBytes, out + b * kSuperBlock);
  }
}

// fp32 view of the weights: the exact value rounded once to binary32.
void orc_q4k_dequant_f32(const uint8_t* blocks, int64_t n_sb, float* out) {
  for (int64_t b = 0; b < n_sb; ++b) {
    double w[kSuperBlock];
    block_values(blocks + b * kBlockBytes, w);
    for (int k = 0; k < kSuperBlock; ++k) out[b * kSuperBlock + k] = static_cast<float>(w[k]);
  }
}

// y[c][r] = sum_k W[r][k] x[c][k]; x is [n_cols][cols] fp32, y and s_abs are [n_cols][rows] fp64.
int orc_gemv_q4k(const uint8_t* w, int64_t rows, int64_t cols, const float* x, int n_cols,
                 double* y, double* s_abs, int n_threads) {
  if (cols % kSuperBlock != 0 || rows < 0 || n_cols < 1) return -1;
  std::vector<double> xd(static_cast<size_t>(n_cols) * cols);
  for (size_t i = 0; i < xd.size(); ++i) xd[i] = x[i];
  gemv_rows(w, rows, cols, xd.data(), n_cols, y, s_abs, n_threads);
  return 0;
}

void orc_rmsnorm(const double* h, const float* g, int64_t n, double eps, double* out) { rmsnorm(h, g, n, eps, out); }

void orc_rope(double* heads, int n_heads, int D, int64_t pos, double theta, int mode) {
  for (int h = 0; h < n_heads; ++h) rope_head(heads + static_cast<int64_t>(h) * D, D, pos, theta, mode);
}

void orc_attend(const double* q, const uint16_t* kc, const uint16_t* vc, int64_t n_ctx, int64_t stride,
                int D, double* out) {
  attend_one(q, kc, vc, n_ctx, stride, D, out);
}

double orc_silu(double z) { return silu(z); }

// ---- model context --------------------------------------------------------------------------
void* orc_ctx_create(const int32_t* cfg_ints /*9*/, float rms_eps, float rope_theta, int rope_mode) {
  Ctx* c = new Ctx();
  c->cfg.n_layers = cfg_ints[0];
  c->cfg.hidden = cfg_ints[1];
  c->cfg.n_q_heads = cfg_ints[2];
  c->cfg.n_kv_heads = cfg_ints[3];
  c->cfg.head_dim = cfg_ints[4];
  c->cfg.ffn = cfg_ints[5];
  c->cfg.vocab = cfg_ints[6];
  c->cfg.kv_capacity = cfg_ints[7];
  c->cfg.max_n_tok = cfg_ints[8];
  c->cfg.rms_eps = rms_eps;
  c->cfg.rope_theta = rope_theta;
  c->cfg.rope_mode = rope_mode;
  c->layer.resize(c->cfg.n_layers);
  for (auto& l : c->layer) l.resize(T_OUT_NORM);
  c->kcache.resize(c->cfg.n_layers);
  c->vcache.resize(c->cfg.n_layers);
  return c;
}

void orc_ctx_destroy(void* p) { delete static_cast<Ctx*>(p); }

// copy != 0: the oracle keeps its own copy; copy == 0: it borrows `data` (caller keeps it alive).
int orc_load_tensor(void* p, int layer, int tensor_id, const void* data, int64_t rows, int64_t cols,
                    int64_t nbytes, int copy) {
  Ctx* c = static_cast<Ctx*>(p);
  if (tensor_id < 0 || tensor_id >= T_COUNT) return -1;
  const bool is_norm = tensor_id == T_ATTN_NORM || tensor_id == T_FFN_NORM || tensor_id == T_OUT_NORM;
  const int64_t expect = is_norm ? cols * 4 : rows * (cols / kSuperBlock) * kBlockBytes;
  if (!is_norm && cols % kSuperBlock != 0) return -1;
  if (nbytes != expect) return -1;
  Tensor* t;
  if (tensor_id >= T_OUT_NORM) {
    if (layer != -1) return -1;
    t = tensor_id == T_OUT_NORM ? &c->out_norm : tensor_id == T_W_HEAD ? &c->w_head : &c->tok_embd;
  } else {
    if (layer < 0 || layer >= c->cfg.n_layers) return -1;
    t = &c->layer[layer][tensor_id];
  }
  t->rows = rows;
  t->cols = cols;
  if (copy) {
    t->own.assign(static_cast<const uint8_t*>(data), static_cast<const uint8_t*>(data) + nbytes);
    t->data = t->own.data();
  } else {
    t->own.clear();
    t->data = static_cast<const uint8_t*>(data);
  }
  return 0;
}

static void ensure_kv(Ctx* c, int layer) {
  const size_t n = static_cast<size_t>(c->cfg.kv_capacity) * c->cfg.n_kv_heads * c->cfg.head_dim;
  if (c->kcache[layer].size() != n) {
    c->kcache[layer].assign(n, 0);
    c->vcache[layer].assign(n, 0);
  }
}

// k, v: [n_pos][n_kv_heads][head_dim] fp16 bit patterns.
int orc_kv_load(void* p, int layer, int pos_begin, int n_pos, const uint16_t* k, const uint16_t* v) {
  Ctx* c = static_cast<Ctx*>(p);
  if (layer < 0 || layer >= c->cfg.n_layers || pos_begin < 0 || pos_begin + n_pos > c->cfg.kv_capacity) return -1;
  ensure_kv(c, layer);
  const size_t row = static_cast<size_t>(c->cfg.n_kv_heads) * c->cfg.head_dim;
  std::memcpy(&c->kcache[layer][pos_begin * row], k, n_pos * row * 2);
  std::memcpy(&c->vcache[layer][pos_begin * row], v, n_pos * row * 2);
  return 0;
}

int orc_kv_read(void* p, int layer, int pos_begin, int n_pos, uint16_t* k, uint16_t* v) {
  Ctx* c = static_cast<Ctx*>(p);
  if (layer < 0 || layer >= c->cfg.n_layers || pos_begin < 0 || pos_begin + n_pos > c->cfg.kv_capacity) return -1;
  ensure_kv(c, layer);
  const size_t row = static_cast<size_t>(c->cfg.n_kv_heads) * c->cfg.head_dim;
  std::memcpy(k, &c->kcache[layer][pos_begin * row], n_pos * row * 2);
  std::memcpy(v, &c->vcache[layer][pos_begin * row], n_pos * row * 2);
  return 0;
}

// Layers [layer_begin, layer_end) for n_tok tokens at positions pos.. ; hidden is [n_tok][hidden].
int orc_forward_window(void* p, int layer_begin, int layer_end, const float* hidden_in, float* hidden_out,
                       int pos, int n_tok, int n_threads) {
  Ctx* c = static_cast<Ctx*>(p);
  if (layer_begin < 0 || layer_end > c->cfg.n_layers || layer_begin > layer_end) return -1;
  if (n_tok < 1 || pos < 0 || pos + n_tok > c->cfg.kv_capacity) return -1;
  for (int l = layer_begin; l < layer_end; ++l)
    if (!layer_ready(*c, l)) return -2;
  std::vector<float> h(hidden_in, hidden_in + static_cast<size_t>(n_tok) * c->cfg.hidden);
  for (int l = layer_begin; l < layer_end; ++l) {
    ensure_kv(c, l);
    layer_forward(*c, l, h, pos, n_tok, n_threads);
  }
  std::memcpy(hidden_out, h.data(), h.size() * sizeof(float));
  return 0;
}

// logits[t][v] = fp32( W_head . RMSNorm(h_t; g_out) )
int orc_logits(void* p, const float* hidden, int n_tok, float* logits, int n_threads) {
  Ctx* c = static_cast<Ctx*>(p);
  if (!c->out_norm.loaded() || !c->w_head.loaded()) return -2;
  const int e = c->cfg.hidden;
  std::vector<double> hd(hidden, hidden + static_cast<size_t>(n_tok) * e), a(hd.size()), y;
  const float* g = reinterpret_cast<const float*>(c->out_norm.data);
  for (int t = 0; t < n_tok; ++t) rmsnorm(&hd[static_cast<size_t>(t) * e], g, e, c->cfg.rms_eps, &a[static_cast<size_t>(t) * e]);
  project(c->w_head, a, n_tok, y, n_threads);
  for (size_t i = 0; i < y.size(); ++i) logits[i] = static_cast<float>(y[i]);
  return 0;
}

// hidden[t] = fp32(dequantised row tokens[t] of the embedding table)
int orc_embed(void* p, const int32_t* tokens, int n_tok, float* hidden_out) {
  Ctx* c = static_cast<Ctx*>(p);
  if (!c->tok_embd.loaded()) return -2;
  const int64_t n_sb = c->tok_embd.cols / kSuperBlock;
  for (int t = 0; t < n_tok; ++t) {
    if (tokens[t] < 0 || tokens[t] >= c->tok_embd.rows) return -1;
    orc_q4k_dequant_f32(c->tok_embd.data + static_cast<int64_t>(tokens[t]) * n_sb * kBlockBytes, n_sb,
                        hidden_out + static_cast<int64_t>(t) * c->tok_embd.cols);
  }
  return 0;
}

// Greedy choice: the lowest index among the largest logits; also reports the gap to the runner-up.
int orc_argmax(const float* logits, int64_t n, float* margin) {
  int64_t best = 0;
  for (int64_t i = 1; i < n; ++i)
    if (logits[i] > logits[best]) best = i;
  if (margin) {
    float second = -std::numeric_limits<float>::infinity();
    for (int64_t i = 0; i < n; ++i)
      if (i != best && logits[i] > second) second = logits[i];
    *margin = logits[best] - second;
  }
  return static_cast<int>(best);
}

}  // extern "C"
