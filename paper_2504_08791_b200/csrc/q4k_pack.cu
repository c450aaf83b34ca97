// Q4_K format kernels: reference-layout dequantisation and the one-time re-tiling of a matrix
// into the streaming layout described in common.cuh.
#include "common.cuh"

namespace prima {
namespace {

// The sixteen 6-bit fields of a standard header (bytes 4..15 of a super-block).
struct Fields6 {
  uint32_t sc[8], m[8];
};

__device__ __forceinline__ Fields6 decode_fields(const uint8_t* s) {
  Fields6 f;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    f.sc[j] = s[j] & 63u;
    f.m[j] = s[j + 4] & 63u;
    f.sc[j + 4] = (s[j + 8] & 15u) | ((s[j] >> 6) << 4);
    f.m[j + 4] = (s[j + 8] >> 4) | ((s[j + 4] >> 6) << 4);
  }
  return f;
}

// One thread per (super-block, byte of qs): two weights.  w = d*sc*q - dmin*m: the three products
// are exact in binary32 (at most 21 significant bits), so the fused multiply-subtract rounds the
// exact value once.
__global__ void dequant_std_kernel(const uint8_t* __restrict__ blocks, int64_t n_sb, float* __restrict__ out) {
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t b = idx >> 7;
  if (b >= n_sb) return;
  const int byte = static_cast<int>(idx & 127);
  const uint8_t* sb = blocks + b * kBlockBytes;
  const float d = __half2float(__ushort_as_half(static_cast<unsigned short>(sb[0] | (sb[1] << 8))));
  const float dmin = __half2float(__ushort_as_half(static_cast<unsigned short>(sb[2] | (sb[3] << 8))));
  const Fields6 f = decode_fields(sb + 4);
  const int p = byte >> 5, i = byte & 31;
  const uint32_t v = sb[16 + byte];
  const float q_lo = static_cast<float>(v & 15u), q_hi = static_cast<float>(v >> 4);
  const float a_lo = d * static_cast<float>(f.sc[2 * p]), b_lo = dmin * static_cast<float>(f.m[2 * p]);
  const float a_hi = d * static_cast<float>(f.sc[2 * p + 1]), b_hi = dmin * static_cast<float>(f.m[2 * p + 1]);
  out[b * 256 + 64 * p + i] = fmaf(a_lo, q_lo, -b_lo);
  out[b * 256 + 64 * p + 32 + i] = fmaf(a_hi, q_hi, -b_hi);
}

// Embedding lookup: one block of 128 threads per (token, super-block of the row); same arithmetic
// as the dequantisation above.
__global__ void embed_kernel(const uint8_t* __restrict__ table, int64_t n_sb_row, const int32_t* __restrict__ tokens,
                             float* __restrict__ out) {
  const int tok = blockIdx.y;
  const int64_t s = blockIdx.x;
  const int byte = threadIdx.x;
  const uint8_t* sb = table + (static_cast<int64_t>(tokens[tok]) * n_sb_row + s) * kBlockBytes;
  const float d = __half2float(__ushort_as_half(static_cast<unsigned short>(sb[0] | (sb[1] << 8))));
  const float dmin = __half2float(__ushort_as_half(static_cast<unsigned short>(sb[2] | (sb[3] << 8))));
  const Fields6 f = decode_fields(sb + 4);
  const int p = byte >> 5, i = byte & 31;
  const uint32_t v = sb[16 + byte];
  float* dst = out + (static_cast<int64_t>(tok) * n_sb_row + s) * 256;
  dst[64 * p + i] = fmaf(d * static_cast<float>(f.sc[2 * p]), static_cast<float>(v & 15u), -(dmin * static_cast<float>(f.m[2 * p])));
  dst[64 * p + 32 + i] = fmaf(d * static_cast<float>(f.sc[2 * p + 1]), static_cast<float>(v >> 4), -(dmin * static_cast<float>(f.m[2 * p + 1])));
}

// One thread per (source row, super-block column): reads 144 bytes, writes its 16-byte header and
// its eight 16-byte nibble chunks into the unit (s, rt).
__global__ void retile_kernel(const uint8_t* __restrict__ src, int64_t rows_src, int64_t n_sb, uint8_t* __restrict__ dst,
                              int64_t n_rt, int64_t dst_row0, int64_t dst_row_stride) {
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= rows_src * n_sb) return;
  const int64_t r = idx / n_sb, s = idx % n_sb;
  const uint8_t* sb = src + idx * kBlockBytes;
  const int64_t row = dst_row0 + r * dst_row_stride;
  const int64_t rt = row >> 3;
  const int g = static_cast<int>(row & 7);
  uint8_t* unit = dst + (s * n_rt + rt) * kUnitBytes;

  const Fields6 f = decode_fields(sb + 4);
  uint32_t ft[4];
#pragma unroll
  for (int t = 0; t < 4; ++t) ft[t] = f.sc[t] | (f.sc[t + 4] << 6) | (f.m[t] << 12) | (f.m[t + 4] << 18);
  uint4 hdr;
  hdr.x = static_cast<uint32_t>(sb[0]) | (static_cast<uint32_t>(sb[1]) << 8) | (static_cast<uint32_t>(sb[2]) << 16) |
          (static_cast<uint32_t>(sb[3]) << 24);
  hdr.y = ft[0] | ((ft[3] & 0xffu) << 24);
  hdr.z = ft[1] | (((ft[3] >> 8) & 0xffu) << 24);
  hdr.w = ft[2] | ((ft[3] >> 16) << 24);
  *reinterpret_cast<uint4*>(unit + g * 16) = hdr;

  const uint8_t* qs = sb + 16;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int p = j >> 1, hi = j & 1;
    uint32_t words[4];
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      uint32_t word = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const uint32_t byte = qs[32 * p + 8 * w + i];
        word |= (hi ? (byte >> 4) : (byte & 15u)) << (4 * i);
      }
      words[w] = word;
    }
    const int half_idx = j >> 2, t = j & 3;
    uint8_t* chunk = unit + kUnitHdrBytes + half_idx * 512 + unit_piece_slot(g, t) * 16;
    *reinterpret_cast<uint4*>(chunk) = make_uint4(words[0], words[1], words[2], words[3]);
  }
}

}  // namespace

int launch_dequant_std(const uint8_t* blocks, int64_t n_sb, float* out, cudaStream_t st) {
  if (n_sb == 0) return 0;
  const int64_t threads = n_sb * 128;
  const int block = 256;
  const int64_t grid = (threads + block - 1) / block;
  dequant_std_kernel<<<static_cast<unsigned>(grid), block, 0, st>>>(blocks, n_sb, out);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 1 : cuda_rc(e);
}

int launch_retile(const uint8_t* src, int64_t rows_src, int64_t n_sb, TiledMat dst, int64_t dst_row0,
                  int64_t dst_row_stride, cudaStream_t st) {
  const int64_t n = rows_src * n_sb;
  if (n == 0) return 0;
  const int block = 128;
  const int64_t grid = (n + block - 1) / block;
  retile_kernel<<<static_cast<unsigned>(grid), block, 0, st>>>(src, rows_src, n_sb, dst.data, dst.n_rt, dst_row0, dst_row_stride);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 1 : cuda_rc(e);
}

int launch_embed(const uint8_t* table_std, int64_t n_sb_per_row, const int32_t* dev_tokens, int n_tok, float* out,
                 cudaStream_t st) {
  dim3 grid(static_cast<unsigned>(n_sb_per_row), n_tok);
  embed_kernel<<<grid, 128, 0, st>>>(table_std, n_sb_per_row, dev_tokens, out);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? 1 : cuda_rc(e);
}

}  // namespace prima
