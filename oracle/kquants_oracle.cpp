// CPU oracle for the other weight formats of the paper's set Q (Appendix A.3, computation latency:
// Q = {Q4_K, Q5_K, Q6_K, Q8_0, FP16, FP32}): Q6_K, Q8_0 and FP16 matrices, dequantisation and the
// matrix-vector product in double precision.  TEST INFRASTRUCTURE ONLY: tests, the smoke check and the
// benchmark's CPU legs may use it; it shares nothing with the CUDA path and the product never calls it.
//
// The paper names these formats and prints none of their bit layouts.  The layouts adopted here are the
// public ones of the file format the paper's system reads:
//
//   Q8_0   a block covers 32 consecutive weights of a row and is 34 bytes:
//            bytes 0-1  d, IEEE binary16, little endian;  bytes 2-33  q[0..31], signed bytes
//            weight k = d * q[k]
//   Q6_K   a super-block covers 256 consecutive weights of a row and is 210 bytes:
//            bytes   0-127  ql: the low four bits of the 6-bit values
//            bytes 128-191  qh: their high two bits
//            bytes 192-207  sc[0..15]: signed byte scales, one per 16 weights
//            bytes 208-209  d, IEEE binary16, little endian
//          weight k = d * sc[k / 16] * (v_k - 32), v_k in 0..63.  With k = 128 n + 32 i + l
//          (n = 0, 1; i = 0..3; l = 0..31):
//            low bits of v_k : byte ql[64 n + 32 (i & 1) + l], its low nibble for i < 2, its high nibble for i >= 2
//            high bits of v_k: bits 2i, 2i+1 of byte qh[32 n + l]
//   FP16   binary16 values, row-major.
//
// The dequantised value is exact in binary32 for both block formats (11 significant bits of d times at
// most 13 bits of integer), so "the fp32 value" is well defined without any rounding.
//
// Pins (tests/test_oracle_kquants.py): hand-built blocks whose values were worked out by hand
// (tests/golden/kquants_handbuilt.txt), one-bit toggles of every header and payload field, dense numpy
// products from fields that were chosen rather than decoded, and, where it is installed, the decoder of the
// gguf Python package on random blocks.
#include <cmath>
#include <cstdint>
#include <cstring>
#include <functional>
#include <limits>
#include <thread>
#include <vector>

namespace {

double half_bits_to_double(uint16_t bits) {
  const int sign = bits >> 15;
  const int expo = (bits >> 10) & 0x1f;
  const int frac = bits & 0x3ff;
  double v;
  if (expo == 0) v = std::ldexp(static_cast<double>(frac), -24);
  else if (expo == 31) v = frac ? std::numeric_limits<double>::quiet_NaN() : std::numeric_limits<double>::infinity();
  else v = std::ldexp(1.0 + static_cast<double>(frac) / 1024.0, expo - 15);
  return sign ? -v : v;
}

constexpr int kFmtQ6K = 1, kFmtQ80 = 2, kFmtF16 = 3;

int64_t block_weights(int fmt) { return fmt == kFmtQ6K ? 256 : fmt == kFmtQ80 ? 32 : 1; }
int64_t block_bytes(int fmt) { return fmt == kFmtQ6K ? 210 : fmt == kFmtQ80 ? 34 : 2; }

void q8_0_values(const uint8_t* b, double* out32) {
  const double d = half_bits_to_double(static_cast<uint16_t>(b[0] | (b[1] << 8)));
  for (int k = 0; k < 32; ++k) out32[k] = d * static_cast<double>(static_cast<int8_t>(b[2 + k]));
}

void q6k_values(const uint8_t* b, double* out256) {
  const uint8_t* ql = b;
  const uint8_t* qh = b + 128;
  const int8_t* sc = reinterpret_cast<const int8_t*>(b + 192);
  const double d = half_bits_to_double(static_cast<uint16_t>(b[208] | (b[209] << 8)));
  for (int k = 0; k < 256; ++k) {
    const int n = k / 128, i = (k % 128) / 32, l = k % 32;
    const uint8_t lo_byte = ql[64 * n + 32 * (i & 1) + l];
    const int lo = i < 2 ? (lo_byte & 15) : (lo_byte >> 4);
    const int hi = (qh[32 * n + l] >> (2 * i)) & 3;
    const int v = lo | (hi << 4);
    out256[k] = d * static_cast<double>(sc[k / 16]) * static_cast<double>(v - 32);
  }
}

void block_values(int fmt, const uint8_t* b, double* out) {
  if (fmt == kFmtQ6K) q6k_values(b, out);
  else if (fmt == kFmtQ80) q8_0_values(b, out);
  else out[0] = half_bits_to_double(static_cast<uint16_t>(b[0] | (b[1] << 8)));
}

void parallel_rows(int64_t rows, int n_threads, const std::function<void(int64_t, int64_t)>& fn) {
  if (n_threads < 1) n_threads = 1;
  if (n_threads > rows) n_threads = static_cast<int>(rows > 0 ? rows : 1);
  std::vector<std::thread> th;
  for (int t = 0; t < n_threads; ++t) {
    const int64_t r0 = rows * t / n_threads, r1 = rows * (t + 1) / n_threads;
    th.emplace_back([=, &fn] { fn(r0, r1); });
  }
  for (auto& t : th) t.join();
}

}  // namespace

extern "C" {

int orc_fmt_block_weights(int fmt) { return static_cast<int>(block_weights(fmt)); }
int orc_fmt_block_bytes(int fmt) { return static_cast<int>(block_bytes(fmt)); }

// n_blocks blocks -> doubles / floats (exact in both).
int orc_fmt_dequant_f64(int fmt, const uint8_t* blocks, int64_t n_blocks, double* out) {
  if (fmt < kFmtQ6K || fmt > kFmtF16) return -1;
  const int64_t bw = block_weights(fmt), bb = block_bytes(fmt);
  for (int64_t i = 0; i < n_blocks; ++i) block_values(fmt, blocks + i * bb, out + i * bw);
  return 0;
}

int orc_fmt_dequant_f32(int fmt, const uint8_t* blocks, int64_t n_blocks, float* out) {
  if (fmt < kFmtQ6K || fmt > kFmtF16) return -1;
  const int64_t bw = block_weights(fmt), bb = block_bytes(fmt);
  std::vector<double> tmp(static_cast<size_t>(bw));
  for (int64_t i = 0; i < n_blocks; ++i) {
    block_values(fmt, blocks + i * bb, tmp.data());
    for (int64_t k = 0; k < bw; ++k) out[i * bw + k] = static_cast<float>(tmp[static_cast<size_t>(k)]);
  }
  return 0;
}

// y[c][r] = sum_k W[r][k] x[c][k] in index order, fp64; s_abs[c][r] = sum_k |W[r][k] x[c][k]|.
// W: rows x cols, row-major blocks; cols a multiple of the block's weights.
int orc_fmt_gemv(int fmt, const uint8_t* w, int64_t rows, int64_t cols, const float* x, int n_cols, double* y, double* s_abs,
                 int n_threads) {
  if (fmt < kFmtQ6K || fmt > kFmtF16 || rows < 0 || cols < 1 || n_cols < 1) return -1;
  const int64_t bw = block_weights(fmt), bb = block_bytes(fmt);
  if (cols % bw != 0) return -1;
  const int64_t n_blk = cols / bw;
  parallel_rows(rows, n_threads, [&](int64_t r0, int64_t r1) {
    std::vector<double> vals(static_cast<size_t>(bw));
    std::vector<double> acc(static_cast<size_t>(n_cols)), mag(static_cast<size_t>(n_cols));
    for (int64_t r = r0; r < r1; ++r) {
      for (int c = 0; c < n_cols; ++c) acc[c] = mag[c] = 0.0;
      for (int64_t b = 0; b < n_blk; ++b) {
        block_values(fmt, w + (r * n_blk + b) * bb, vals.data());
        for (int c = 0; c < n_cols; ++c) {
          const float* xc = x + static_cast<int64_t>(c) * cols + b * bw;
          for (int64_t k = 0; k < bw; ++k) {
            const double p = vals[static_cast<size_t>(k)] * static_cast<double>(xc[k]);
            acc[c] += p;
            mag[c] += std::fabs(p);
          }
        }
      }
      for (int c = 0; c < n_cols; ++c) {
        y[static_cast<int64_t>(c) * rows + r] = acc[c];
        s_abs[static_cast<int64_t>(c) * rows + r] = mag[c];
      }
    }
  });
  return 0;
}

}  // extern "C"
