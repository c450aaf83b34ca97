// The other weight formats of the paper's set Q (Appendix A.3, computation latency): Q6_K, Q8_0 and FP16 matrices
// in their standard row-major block layouts.  Bit-exact dequantisation and a streaming matrix-vector product.
//
// Layouts (the public ones of the file format the paper's system reads; the paper prints none):
//   Q8_0  34-byte block of 32 weights: binary16 d, then 32 signed bytes q;            w = d * q
//   Q6_K  210-byte super-block of 256 weights: ql[128] low nibbles, qh[64] high bit pairs, sc[16] signed byte
//         scales (one per 16 weights), binary16 d;                                     w = d * sc * (v - 32)
//         weight k = 128 n + 32 i + l: low nibble in byte ql[64 n + 32 (i & 1) + l] (low half for i < 2, high half
//         otherwise), high two bits in bits 2i, 2i+1 of byte qh[32 n + l]
//   FP16  binary16 values.
//
// The product.  One CTA works on one row at a time (persistent grid, rows dealt round-robin): the row's bytes are
// brought into shared memory with 16-byte asynchronous copies (the copy starts at the 16-byte boundary at or
// below the row's first byte, since rows of these formats need not start on one), the next row is requested
// before the current one is used, and the activations of all columns sit in shared memory as fp32 for the
// whole kernel.  FP16 weights are multiplied in fp32 (one CTA per row, double-buffered 16-byte copies).  For the two
// block formats the activations are held as in the Q4_K kernels: 16-bit integers x_q = round(x / s_b) with one fp32
// step s_b per block of 32, cut into a high and a low signed byte, so that the sum over a group of weights is an exact
// integer from 4-way byte dot products (Q8_0: q * x_q; Q6_K: v * x_q - 32 * sum(x_q), v the unsigned 6-bit value),
// scaled once per group by d * s_b (* sc for Q6_K) in fp32.  Every CTA quantises the activations once into shared
// memory; then every warp takes rows of its own and streams them in segments of 2048 weights through a ring of
// 16-byte asynchronous copies of its own (no barrier between warps), a lane working on 64 weights of a segment; the
// lanes' sums are added by shuffles, so the result is the same from run to run.
// Bound: HBM (0.82 / 1.06 / 2 bytes per weight).
#include <cstdio>

#include "../../include/prima.h"
#include "common.cuh"

namespace prima {
namespace {

constexpr int kThreads = 256;
constexpr float kMagic = 8388608.0f;      // 2^23: the integers 0..2^23-1 are the mantissas of [2^23, 2^24)

__device__ __forceinline__ float half_bits_to_float(uint32_t bits) { return __half2float(__ushort_as_half(static_cast<unsigned short>(bits))); }
__device__ __forceinline__ uint32_t lds_u16(const uint8_t* p) { return *reinterpret_cast<const uint16_t*>(p); }
// Byte `sel` (0..3) of w as an exact float, plus 2^23.
__device__ __forceinline__ float byte_plus_magic(uint32_t w, uint32_t sel) { return __uint_as_float(__byte_perm(w, 0x4B000000u, 0x7440u | sel)); }

// ---- dequantisation (the bit-exact definitions) ---------------------------------------------------------------
__global__ void dequant_q8_0_kernel(const uint8_t* __restrict__ blocks, int64_t n_blocks, float* __restrict__ out) {
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= n_blocks * 32) return;
  const uint8_t* b = blocks + (idx >> 5) * 34;
  const float d = half_bits_to_float(b[0] | (b[1] << 8));
  out[idx] = d * static_cast<float>(static_cast<int8_t>(b[2 + (idx & 31)]));      // 11 x 8 bits: exact
}

__global__ void dequant_q6k_kernel(const uint8_t* __restrict__ blocks, int64_t n_blocks, float* __restrict__ out) {
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= n_blocks * 256) return;
  const uint8_t* b = blocks + (idx >> 8) * 210;
  const int k = static_cast<int>(idx & 255);
  const int n = k >> 7, i = (k >> 5) & 3, l = k & 31;
  const uint32_t lo_byte = b[64 * n + 32 * (i & 1) + l];
  const int v = static_cast<int>((i < 2 ? (lo_byte & 15u) : (lo_byte >> 4)) | (((b[128 + 32 * n + l] >> (2 * i)) & 3u) << 4));
  const int sc = static_cast<int8_t>(b[192 + (k >> 4)]);
  const float d = half_bits_to_float(b[208] | (b[209] << 8));
  // 11 x 13 bits: exact; the factors are multiplied as floats so that a zero weight gets the sign of the product of
  // the three signs, as in d * sc * (v - 32) evaluated in any order
  out[idx] = d * (static_cast<float>(sc) * static_cast<float>(v - 32));
}

__global__ void dequant_f16_kernel(const uint8_t* __restrict__ blocks, int64_t n, float* __restrict__ out) {
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx < n) out[idx] = half_bits_to_float(blocks[2 * idx] | (blocks[2 * idx + 1] << 8));
}

// ---- the product ----------------------------------------------------------------------------------------------
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(__cvta_generic_to_global(src)) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Sum over a row's weights of w * x for NC columns: the thread's share.  `row` points at the row's first byte
// in shared memory (2-byte aligned), xs at the activations [NC][cols].
template <int FMT, int NC>
__device__ __forceinline__ void row_partial(const uint8_t* row, const float* xs, int64_t cols, float (&acc)[NC]) {
  const int t = threadIdx.x;
  if (FMT == PRIMA_FMT_Q8_0) {
    // eight threads per block of 32 weights, four consecutive weights each
    const int64_t n_blk = cols >> 5;
    const int j = t & 7;
    for (int64_t b = t >> 3; b < n_blk; b += kThreads / 8) {
      const uint8_t* blk = row + b * 34;
      const float d = half_bits_to_float(lds_u16(blk));
      const uint32_t q = (lds_u16(blk + 2 + 4 * j) | (lds_u16(blk + 4 + 4 * j) << 16)) ^ 0x80808080u;      // q + 128 as unsigned bytes
      float f[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) f[e] = byte_plus_magic(q, e) - (kMagic + 128.0f);
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        const float4 x = *reinterpret_cast<const float4*>(xs + c * cols + 32 * b + 4 * j);
        acc[c] = fmaf(d, fmaf(f[0], x.x, fmaf(f[1], x.y, fmaf(f[2], x.z, f[3] * x.w))), acc[c]);
      }
    }
  } else if (FMT == PRIMA_FMT_Q6_K) {
    // sixteen threads per super-block: thread u = (half n, four consecutive positions l0..l0+3), 16 weights each
    const int64_t n_sb = cols >> 8;
    const int u = t & 15, n = u >> 3, l0 = 4 * (u & 7);
    for (int64_t s = t >> 4; s < n_sb; s += kThreads / 16) {
      const uint8_t* sb = row + s * 210;
      const uint8_t* pa = sb + 64 * n + l0;
      const uint32_t ql_a = lds_u16(pa) | (lds_u16(pa + 2) << 16);
      const uint32_t ql_b = lds_u16(pa + 32) | (lds_u16(pa + 34) << 16);
      const uint8_t* ph = sb + 128 + 32 * n + l0;
      const uint32_t qh = lds_u16(ph) | (lds_u16(ph + 2) << 16);
      const float d = half_bits_to_float(lds_u16(sb + 208));
      const int8_t* scp = reinterpret_cast<const int8_t*>(sb + 192 + 8 * n + (l0 >> 4));
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t src = (i & 1) ? ql_b : ql_a;
        const uint32_t lo = i < 2 ? (src & 0x0f0f0f0fu) : ((src >> 4) & 0x0f0f0f0fu);
        const uint32_t v4 = lo | (((qh >> (2 * i)) & 0x03030303u) << 4);      // four values 0..63
        const float dsc = d * static_cast<float>(scp[2 * i]);
        float f[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) f[e] = byte_plus_magic(v4, e) - (kMagic + 32.0f);
#pragma unroll
        for (int c = 0; c < NC; ++c) {
          const float4 x = *reinterpret_cast<const float4*>(xs + c * cols + 256 * s + 128 * n + 32 * i + l0);
          acc[c] = fmaf(dsc, fmaf(f[0], x.x, fmaf(f[1], x.y, fmaf(f[2], x.z, f[3] * x.w))), acc[c]);
        }
      }
    }
  } else {      // FP16: two weights per 32-bit word
    for (int64_t k = 2 * static_cast<int64_t>(t); k < cols; k += 2 * kThreads) {
      const uint32_t w2 = lds_u16(row + 2 * k) | (lds_u16(row + 2 * k + 2) << 16);
      const float2 wf = __half22float2(*reinterpret_cast<const __half2*>(&w2));
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        const float2 x = *reinterpret_cast<const float2*>(xs + c * cols + k);
        acc[c] = fmaf(wf.x, x.x, fmaf(wf.y, x.y, acc[c]));
      }
    }
  }
}

template <int FMT, int NC>
__global__ void __launch_bounds__(kThreads) gemv_fmt_kernel(const uint8_t* __restrict__ w, int64_t rows, int64_t cols, int64_t row_bytes,
                                                             int64_t buf_bytes, const float* __restrict__ x, float* __restrict__ y) {
  extern __shared__ __align__(16) uint8_t smem[];
  float* xs = reinterpret_cast<float*>(smem);                                            // [NC][cols]
  uint8_t* bufs = smem + static_cast<size_t>(NC) * cols * sizeof(float);                 // two row buffers of buf_bytes
  __shared__ float s_part[kThreads / 32][NC];
  const int t = threadIdx.x;
  // The bytes of row r, from the 16-byte boundary at or below its first byte; every 16-byte piece that the row
  // touches lies inside the matrix's allocation rounded up to 16 bytes, which every CUDA allocation is.
  auto request = [&](int64_t r, int slot) {
    const uintptr_t first = reinterpret_cast<uintptr_t>(w) + static_cast<uintptr_t>(r * row_bytes);
    const uintptr_t a0 = first & ~static_cast<uintptr_t>(15), a1 = (first + row_bytes + 15) & ~static_cast<uintptr_t>(15);
    const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(bufs + static_cast<size_t>(slot) * buf_bytes));
    for (uintptr_t off = static_cast<uintptr_t>(t) * 16; off < a1 - a0; off += kThreads * 16) cp_async16(dst + static_cast<uint32_t>(off), reinterpret_cast<const void*>(a0 + off));
  };
  int64_t r = blockIdx.x;
  if (r < rows) request(r, 0);
  cp_async_commit();
  for (int64_t i = t; i < NC * cols / 4; i += kThreads) reinterpret_cast<float4*>(xs)[i] = __ldg(reinterpret_cast<const float4*>(x) + i);
  int slot = 0;
  for (; r < rows; r += gridDim.x, slot ^= 1) {
    const int64_t nxt = r + gridDim.x;
    if (nxt < rows) request(nxt, slot ^ 1);
    cp_async_commit();
    cp_async_wait<1>();      // the current row's copies of this thread; the barrier makes everybody's visible
    __syncthreads();
    const uintptr_t first = reinterpret_cast<uintptr_t>(w) + static_cast<uintptr_t>(r * row_bytes);
    const uint8_t* row = bufs + static_cast<size_t>(slot) * buf_bytes + (first & 15);
    float acc[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) acc[c] = 0.f;
    row_partial<FMT, NC>(row, xs, cols, acc);
#pragma unroll
    for (int c = 0; c < NC; ++c) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], o);
      if ((t & 31) == 0) s_part[t >> 5][c] = acc[c];
    }
    __syncthreads();      // also: everybody is done with this row's buffer before the request after next overwrites it
    if (t < NC) {
      float sum = 0.f;
#pragma unroll
      for (int wp = 0; wp < kThreads / 32; ++wp) sum += s_part[wp][t];
      y[static_cast<int64_t>(t) * rows + r] = sum;
    }
  }
  cp_async_wait<0>();
}

// ---- the block formats with 16-bit integer activations ---------------------------------------------------------
__device__ __forceinline__ int dp4a_ss(uint32_t a, uint32_t b, int c) { return __dp4a(static_cast<int>(a), static_cast<int>(b), c); }
__device__ __forceinline__ int dp4a_us(uint32_t a, uint32_t b, int c) {      // unsigned bytes of a times signed bytes of b
  int d;
  asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
// Loads from shared memory by 32-bit shared-space address (volatile: they stay behind the wait that precedes them).
__device__ __forceinline__ uint32_t sld32(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ uint32_t sld16(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ int sld8s(uint32_t a) {
  int v;
  asm volatile("ld.shared.s8 %0, [%1];" : "=r"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ uint4 sld128(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}
// N consecutive words starting at an even shared-memory address `a`: N + 1 aligned words, shifted by 0 or 16 bits.
template <int N>
__device__ __forceinline__ void lds_even(uint32_t a, uint32_t (&out)[N]) {
  const uint32_t base = a & ~3u, sh = (a & 2u) * 8u;
  uint32_t w[N + 1];
#pragma unroll
  for (int i = 0; i <= N; ++i) w[i] = sld32(base + 4 * i);
#pragma unroll
  for (int i = 0; i < N; ++i) out[i] = __funnelshift_r(w[i], w[i + 1], sh);
}

// A row is cut into segments of 2048 weights (8 Q6_K super-blocks, 1680 bytes; 64 Q8_0 blocks, 2176 bytes; the last
// segment of a row may be shorter).  The shared-memory image of one column of activations is cut into pieces of 16
// consecutive values: piece j has its 16 high bytes at 16 j, its low bytes at P + 16 j and two pairs (sum of eight
// x_q, step of their block of 32 as fp32 bits) at 2 P + 16 j; P = cols rounded up to 2048.  The pieces of a segment
// are ordered so that the 32 lanes of a warp read 512 consecutive bytes with every 16-byte load:
//   Q8_0: lane = block b of 32 within the half segment; piece (b, first / second 16 values) -> 64 (b / 32) + 32 half + b % 32
//   Q6_K: lane = (super-block s, half n, 16 positions h); piece of values 256 s + 128 n + 32 i + 16 h .. -> 32 i + 4 s + 2 n + h
template <int FMT>
__device__ __forceinline__ int piece_slot(int piece) {      // piece = index of 16 consecutive values within the row
  const int seg = piece >> 7, in = piece & 127;
  if (FMT == PRIMA_FMT_Q8_0) {
    const int b = in >> 1, half = in & 1;
    return 128 * seg + 64 * (b >> 5) + 32 * half + (b & 31);
  }
  const int s = in >> 4, n = (in >> 3) & 1, i = (in >> 1) & 3, h = in & 1;
  return 128 * seg + 32 * i + 4 * s + 2 * n + h;
}

constexpr int kSegWeights = 2048;
template <int FMT>
struct SegShape {
  static constexpr int kBytes = FMT == PRIMA_FMT_Q8_0 ? 64 * 34 : 8 * 210;      // a full segment
  static constexpr int kBuf = kBytes + 32;                                      // + the bytes around an unaligned start and end
  static constexpr int kUnit = FMT == PRIMA_FMT_Q8_0 ? 272 : 210;               // bytes of 256 weights
};

// One segment of one row, staged at shared-memory address `seg` (its first byte): this lane's share of sum w x.
// `ximg` is the address of the activations' image of column 0 at this segment (+ 16 * lane).
template <int FMT, int NC>
__device__ __forceinline__ void segment_partial(uint32_t seg, int n_units, uint32_t ximg, uint32_t col_bytes, uint32_t padded, int lane, float (&acc)[NC]) {
  if (FMT == PRIMA_FMT_Q8_0) {
    // lane = block within a half segment of 32 blocks (8 units of 256 weights = 64 blocks)
#pragma unroll
    for (int hs = 0; hs < 2; ++hs) {
      const int b = 32 * hs + lane;
      if (b < 8 * n_units) {
        const uint32_t blk = seg + 34 * b;
        const float d = half_bits_to_float(sld16(blk));
        uint32_t q[8];
        lds_even<8>(blk + 2, q);
#pragma unroll
        for (int c = 0; c < NC; ++c) {
          const uint32_t xc = ximg + c * col_bytes + 1024 * hs;
          const uint4 h0 = sld128(xc), h1 = sld128(xc + 512);
          const uint4 l0 = sld128(xc + padded), l1 = sld128(xc + padded + 512);
          const float step = __uint_as_float(sld32(xc + 2 * padded + 4));
          int h = dp4a_ss(q[3], h0.w, dp4a_ss(q[2], h0.z, dp4a_ss(q[1], h0.y, dp4a_ss(q[0], h0.x, 0))));
          h = dp4a_ss(q[7], h1.w, dp4a_ss(q[6], h1.z, dp4a_ss(q[5], h1.y, dp4a_ss(q[4], h1.x, h))));
          int l = dp4a_ss(q[3], l0.w, dp4a_ss(q[2], l0.z, dp4a_ss(q[1], l0.y, dp4a_ss(q[0], l0.x, 0))));
          l = dp4a_ss(q[7], l1.w, dp4a_ss(q[6], l1.z, dp4a_ss(q[5], l1.y, dp4a_ss(q[4], l1.x, l))));
          acc[c] = fmaf(static_cast<float>(h * 256 + l), d * step, acc[c]);
        }
      }
    }
  } else {
    // lane = (super-block s of the segment, half n, 16 positions 16 h ..): 64 weights
    const int s = lane >> 2, n = (lane >> 1) & 1, h16 = lane & 1;
    if (s < n_units) {
      const uint32_t sb = seg + 210 * s;
      uint32_t qa[4], qb[4], qh[4];
      lds_even<4>(sb + 64 * n + 16 * h16, qa);
      lds_even<4>(sb + 64 * n + 32 + 16 * h16, qb);
      lds_even<4>(sb + 128 + 32 * n + 16 * h16, qh);
      const float d = half_bits_to_float(sld16(sb + 208));
      const uint32_t scp = sb + 192 + 8 * n + h16;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        uint32_t v[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint32_t src = (i & 1) ? qb[k] : qa[k];
          const uint32_t hi2 = (i < 2 ? (qh[k] << (4 - 2 * i)) : (qh[k] >> (2 * i - 4))) & 0x30303030u;
          v[k] = ((i < 2 ? src : (src >> 4)) & 0x0f0f0f0fu) | hi2;
        }
        const float dsc = d * static_cast<float>(sld8s(scp + 2 * i));
#pragma unroll
        for (int c = 0; c < NC; ++c) {
          const uint32_t xc = ximg + c * col_bytes + 512 * i;
          const uint4 xh = sld128(xc);
          const uint4 xl = sld128(xc + padded);
          const uint4 ss = sld128(xc + 2 * padded);      // (sum, step, sum, step): one block of 32, one step
          const int hh = dp4a_us(v[3], xh.w, dp4a_us(v[2], xh.z, dp4a_us(v[1], xh.y, dp4a_us(v[0], xh.x, 0))));
          const int ll = dp4a_us(v[3], xl.w, dp4a_us(v[2], xl.z, dp4a_us(v[1], xl.y, dp4a_us(v[0], xl.x, 0))));
          acc[c] = fmaf(static_cast<float>(hh * 256 + ll - 32 * (static_cast<int>(ss.x) + static_cast<int>(ss.z))), dsc * __uint_as_float(ss.y), acc[c]);
        }
      }
    }
  }
}

constexpr int kMaxQThreads = 512;

// Every warp takes rows of its own (global warp number, then every total-warps-th row) and streams their segments
// through a ring of `depth` buffers of its own in shared memory: no barrier between warps after the prologue.
template <int FMT, int NC>
__global__ void __launch_bounds__(kMaxQThreads) gemv_fmtq_kernel(const uint8_t* __restrict__ w, int64_t rows, int cols, int row_bytes, int depth,
                                                                  const float* __restrict__ x, float* __restrict__ y) {
  using Seg = SegShape<FMT>;
  extern __shared__ __align__(16) uint8_t smem[];
  const int padded = (cols + kSegWeights - 1) / kSegWeights * kSegWeights, col_bytes = 3 * padded;
  const int t = threadIdx.x, nthr = blockDim.x, lane = t & 31, warp = t >> 5, n_warps = nthr >> 5;
  const int ring = NC * col_bytes + warp * depth * Seg::kBuf;      // offset of this warp's ring
  const uint32_t ring_u32 = static_cast<uint32_t>(__cvta_generic_to_shared(smem + ring));
  const uint32_t img_u32 = static_cast<uint32_t>(__cvta_generic_to_shared(smem)) + 16 * lane;      // this lane's piece of a segment's image
  const int segs_per_row = (cols + kSegWeights - 1) / kSegWeights;
  const int64_t gw = static_cast<int64_t>(blockIdx.x) * n_warps + warp, total_warps = static_cast<int64_t>(gridDim.x) * n_warps;
  const int64_t my_rows = gw < rows ? (rows - 1 - gw) / total_warps + 1 : 0;
  const int64_t n_flat = my_rows * segs_per_row;      // this warp's segments, row after row
  // running description of the next segment to request: its first byte, its number within the row, its ring slot
  const uintptr_t row_step = static_cast<uintptr_t>(total_warps) * row_bytes - static_cast<uintptr_t>(segs_per_row - 1) * Seg::kBytes;
  uintptr_t rq_first = reinterpret_cast<uintptr_t>(w) + static_cast<uintptr_t>(gw) * row_bytes;
  int rq_seg = 0, rq_slot = 0;
  int64_t rq_left = n_flat;
  const int tail_units = (cols >> 8) - 8 * (segs_per_row - 1);      // units of a row's last segment (1..8)
  auto request = [&]() {
    if (rq_left > 0) {
      const bool last = rq_seg == segs_per_row - 1;
      const int units = last ? tail_units : 8;
      const uint32_t lead = static_cast<uint32_t>(rq_first) & 15u;
      const uint8_t* src = reinterpret_cast<const uint8_t*>(rq_first - lead) + 16 * lane;
      const int n16 = static_cast<int>((lead + units * Seg::kUnit + 15) >> 4);
      const uint32_t dst = ring_u32 + rq_slot * Seg::kBuf + 16 * lane;
      for (int k = lane; k < n16; k += 32) cp_async16(dst + 16 * (k - lane), src + 16 * (k - lane));
      rq_first += last ? row_step : static_cast<uintptr_t>(Seg::kBytes);
      rq_seg = last ? 0 : rq_seg + 1;
      --rq_left;
    }
    rq_slot = rq_slot + 1 == depth ? 0 : rq_slot + 1;
    cp_async_commit();
  };
  for (int j = 0; j < depth - 1; ++j) request();
  // quantise the activations: one thread per chunk of eight values, four neighbouring lanes per block of 32
  // (the number of chunks is a multiple of 32 and so is the stride: a warp is in a pass as a whole)
  const int n_chunks = cols >> 3;
  const bool x_vec = (reinterpret_cast<uintptr_t>(x) & 15) == 0;
  for (int task = t; task < NC * n_chunks; task += nthr) {
    const int c = task / n_chunks, kc = task - c * n_chunks;
    const float* xp = x + static_cast<int64_t>(c) * cols + 8 * kc;
    float v[8];
    if (x_vec) {
      const float4 a = __ldg(reinterpret_cast<const float4*>(xp)), b = __ldg(reinterpret_cast<const float4*>(xp) + 1);
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = __ldg(xp + e);
    }
    float amax = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) amax = fmaxf(amax, fabsf(v[e]));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
    const bool ok = amax > 0.f && amax < 3.0e38f;
    const float inv = ok ? __fdividef(32639.0f, amax) : 0.f;
    uint32_t hi[2] = {0u, 0u}, lo[2] = {0u, 0u};
    int sum = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int q = max(-32639, min(32639, __float2int_rn(v[e] * inv)));
      const int l = ((q + 128) & 255) - 128, h = (q - l) >> 8;
      sum += q;
      hi[e >> 2] |= static_cast<uint32_t>(h & 255) << (8 * (e & 3));
      lo[e >> 2] |= static_cast<uint32_t>(l & 255) << (8 * (e & 3));
    }
    uint8_t* xc = smem + c * col_bytes + 16 * piece_slot<FMT>(kc >> 1) + 8 * (kc & 1);
    *reinterpret_cast<uint2*>(xc) = make_uint2(hi[0], hi[1]);
    *reinterpret_cast<uint2*>(xc + padded) = make_uint2(lo[0], lo[1]);
    *reinterpret_cast<int2*>(xc + 2 * padded) = make_int2(sum, __float_as_int(ok ? amax * (1.0f / 32639.0f) : 0.f));
  }
  __syncthreads();      // the image is complete; from here on the warps go their own ways

  float acc[NC];
#pragma unroll
  for (int c = 0; c < NC; ++c) acc[c] = 0.f;
  int64_t row = gw;
  int seg = 0, slot = 0;
  uintptr_t first = reinterpret_cast<uintptr_t>(w) + static_cast<uintptr_t>(gw) * row_bytes;
  for (int64_t q = 0; q < n_flat; ++q) {
    // this segment's copies of this lane (all but the depth-1 newest groups), then everybody's
    switch (depth) {
      case 2: cp_async_wait<0>(); break;
      case 3: cp_async_wait<1>(); break;
      case 4: cp_async_wait<2>(); break;
      case 5: cp_async_wait<3>(); break;
      default: cp_async_wait<4>(); break;
    }
    __syncwarp();      // also: every lane is done with the buffer of segment q - 1, which the next request overwrites
    request();
    const bool last = seg == segs_per_row - 1;
    const uint32_t at = ring_u32 + slot * Seg::kBuf + (static_cast<uint32_t>(first) & 15u);
    segment_partial<FMT, NC>(at, last ? tail_units : 8, img_u32 + 2048 * seg, col_bytes, padded, lane, acc);
    slot = slot + 1 == depth ? 0 : slot + 1;
    if (last) {
#pragma unroll
      for (int c = 0; c < NC; ++c) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], o);
        if (lane == 0) y[static_cast<int64_t>(c) * rows + row] = acc[c];
        acc[c] = 0.f;
      }
      seg = 0;
      row += total_warps;
      first += row_step;
    } else {
      ++seg;
      first += Seg::kBytes;
    }
  }
  cp_async_wait<0>();
}

template <int FMT>
int launch_gemv_fmt(const uint8_t* w, int64_t rows, int64_t cols, int64_t row_bytes, const float* x, int n_cols, float* y, int sm_count,
                    cudaStream_t st) {
  if (FMT == PRIMA_FMT_F16) {
    const int64_t buf_bytes = ((row_bytes + 15) / 16 + 1) * 16;
    const size_t smem = static_cast<size_t>(n_cols) * cols * sizeof(float) + 2 * static_cast<size_t>(buf_bytes);
    if (smem > 200 * 1024) return cuda_rc(cudaErrorInvalidValue);
    void (*kern)(const uint8_t*, int64_t, int64_t, int64_t, int64_t, const float*, float*) = nullptr;
    switch (n_cols) {
      case 1: kern = gemv_fmt_kernel<PRIMA_FMT_F16, 1>; break;
      case 2: kern = gemv_fmt_kernel<PRIMA_FMT_F16, 2>; break;
      case 3: kern = gemv_fmt_kernel<PRIMA_FMT_F16, 3>; break;
      default: kern = gemv_fmt_kernel<PRIMA_FMT_F16, 4>; break;
    }
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return cuda_rc(e);
    const int per_sm = static_cast<int>(std::max<size_t>(1, std::min<size_t>(8, (220 * 1024) / (smem + 1024))));
    const int64_t grid = std::min<int64_t>(rows, static_cast<int64_t>(sm_count) * per_sm);
    kern<<<static_cast<unsigned>(grid), kThreads, smem, st>>>(w, rows, cols, row_bytes, buf_bytes, x, y);
    e = cudaGetLastError();
    return e == cudaSuccess ? 1 : cuda_rc(e);
  }
  constexpr int F = FMT == PRIMA_FMT_F16 ? PRIMA_FMT_Q8_0 : FMT;      // (the block formats only; keeps the F16 instantiation out)
  // one CTA per SM: the activations' image once, the rest of shared memory for the warps' rings (2..6 buffers each);
  // 16 warps, or 8 when the image leaves too little room
  const size_t x_bytes = static_cast<size_t>(n_cols) * 3 * static_cast<size_t>((cols + kSegWeights - 1) / kSegWeights * kSegWeights);
  const size_t room = 215 * 1024;
  // 8..16 warps a CTA: as many as leave every warp a ring of three buffers (two at least), and among those the count
  // that wastes the fewest warp-rows in the last round (8192 rows on 148 SMs: 14 warps, 98.8 % against 86.5 % with 16)
  int warps = 0;
  double best = -1.0;
  for (int cand = kMaxQThreads / 32; cand >= 8; --cand) {
    if (x_bytes + static_cast<size_t>(cand) * (cand > 8 ? 3 : 2) * SegShape<F>::kBuf > room) continue;
    const int64_t all = static_cast<int64_t>(sm_count) * cand;
    const double eff = static_cast<double>(rows) / static_cast<double>((rows + all - 1) / all * all);
    if (eff > best + 0.02) {
      best = eff;
      warps = cand;
    }
  }
  if (warps == 0) return cuda_rc(cudaErrorInvalidValue);
  const int depth = static_cast<int>(std::min<size_t>(6, (room - x_bytes) / (static_cast<size_t>(warps) * SegShape<F>::kBuf)));
  const size_t smem = x_bytes + static_cast<size_t>(warps) * depth * SegShape<F>::kBuf;
  void (*kern)(const uint8_t*, int64_t, int, int, int, const float*, float*) = nullptr;
  switch (n_cols) {
    case 1: kern = gemv_fmtq_kernel<F, 1>; break;
    case 2: kern = gemv_fmtq_kernel<F, 2>; break;
    case 3: kern = gemv_fmtq_kernel<F, 3>; break;
    default: kern = gemv_fmtq_kernel<F, 4>; break;
  }
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return cuda_rc(e);
  const int64_t grid = std::min<int64_t>((rows + warps - 1) / warps, sm_count);
  kern<<<static_cast<unsigned>(grid), warps * 32, smem, st>>>(w, rows, static_cast<int>(cols), static_cast<int>(row_bytes), depth, x, y);
  e = cudaGetLastError();
  return e == cudaSuccess ? 1 : cuda_rc(e);
}

thread_local char g_fmt_error[200] = "";
int fmt_fail(const char* msg) {
  snprintf(g_fmt_error, sizeof(g_fmt_error), "%s", msg);
  return PRIMA_ERR_ARG;
}

}  // namespace
}  // namespace prima

using namespace prima;

extern "C" {

int prima_fmt_block_weights(int fmt) { return fmt == PRIMA_FMT_Q4_K || fmt == PRIMA_FMT_Q6_K ? 256 : fmt == PRIMA_FMT_Q8_0 ? 32 : fmt == PRIMA_FMT_F16 ? 1 : 0; }
int prima_fmt_block_bytes(int fmt) { return fmt == PRIMA_FMT_Q4_K ? 144 : fmt == PRIMA_FMT_Q6_K ? 210 : fmt == PRIMA_FMT_Q8_0 ? 34 : fmt == PRIMA_FMT_F16 ? 2 : 0; }
const char* prima_fmt_last_error(void) { return g_fmt_error; }

int prima_dequant_fmt(int fmt, const void* dev_blocks, int64_t n_blocks, float* dev_out, void* stream) {
  if (fmt == PRIMA_FMT_Q4_K) return prima_dequant_q4k(dev_blocks, n_blocks, dev_out, stream);
  if (prima_fmt_block_weights(fmt) == 0) return fmt_fail("prima_dequant_fmt: unknown format");
  if (n_blocks == 0) return PRIMA_OK;
  if (!dev_blocks || !dev_out || n_blocks < 0) return fmt_fail("prima_dequant_fmt: bad argument");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t n = n_blocks * prima_fmt_block_weights(fmt);
  const unsigned grid = static_cast<unsigned>((n + 255) / 256);
  const uint8_t* b = static_cast<const uint8_t*>(dev_blocks);
  if (fmt == PRIMA_FMT_Q8_0) dequant_q8_0_kernel<<<grid, 256, 0, st>>>(b, n_blocks, dev_out);
  else if (fmt == PRIMA_FMT_Q6_K) dequant_q6k_kernel<<<grid, 256, 0, st>>>(b, n_blocks, dev_out);
  else dequant_f16_kernel<<<grid, 256, 0, st>>>(b, n, dev_out);
  if (cudaGetLastError() != cudaSuccess) {
    snprintf(g_fmt_error, sizeof(g_fmt_error), "prima_dequant_fmt: launch failed");
    return PRIMA_ERR_CUDA;
  }
  return PRIMA_OK;
}

int prima_gemv_fmt(int fmt, const void* dev_w, int64_t rows, int64_t cols, const float* dev_x, int n_cols, float* dev_y, void* stream) {
  if (fmt == PRIMA_FMT_Q4_K) return prima_gemv_q4k(dev_w, rows, cols, dev_x, n_cols, dev_y, stream);
  if (prima_fmt_block_weights(fmt) == 0) return fmt_fail("prima_gemv_fmt: unknown format");
  if (!dev_w || !dev_x || !dev_y || rows < 1 || cols < 256 || cols % 256 != 0 || n_cols < 1 || n_cols > 4)
    return fmt_fail("prima_gemv_fmt: rows >= 1, cols a positive multiple of 256 and 1 <= n_cols <= 4 are required");
  if (reinterpret_cast<uintptr_t>(dev_w) & 1) return fmt_fail("prima_gemv_fmt: dev_w must be at an even address");
  const int64_t row_bytes = cols / prima_fmt_block_weights(fmt) * prima_fmt_block_bytes(fmt);
  const int64_t x_bytes = fmt == PRIMA_FMT_F16 ? cols * 4 : 3 * ((cols + 2047) / 2048 * 2048);
  if (static_cast<int64_t>(n_cols) * x_bytes + (fmt == PRIMA_FMT_F16 ? 2 * (row_bytes + 32) : 8 * 2 * 2208) > 200 * 1024)
    return fmt_fail("prima_gemv_fmt: the activations of all columns and the copy buffers must fit 200 KiB of shared memory");
  int dev = 0, sm_count = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const uint8_t* w = static_cast<const uint8_t*>(dev_w);
  int k;
  if (fmt == PRIMA_FMT_Q8_0) k = launch_gemv_fmt<PRIMA_FMT_Q8_0>(w, rows, cols, row_bytes, dev_x, n_cols, dev_y, sm_count, st);
  else if (fmt == PRIMA_FMT_Q6_K) k = launch_gemv_fmt<PRIMA_FMT_Q6_K>(w, rows, cols, row_bytes, dev_x, n_cols, dev_y, sm_count, st);
  else k = launch_gemv_fmt<PRIMA_FMT_F16>(w, rows, cols, row_bytes, dev_x, n_cols, dev_y, sm_count, st);
  if (k < 0) {
    snprintf(g_fmt_error, sizeof(g_fmt_error), "prima_gemv_fmt: launch failed: %s", cudaGetErrorString(static_cast<cudaError_t>(-k)));
    return PRIMA_ERR_CUDA;
  }
  return PRIMA_OK;
}

}  // extern "C"
