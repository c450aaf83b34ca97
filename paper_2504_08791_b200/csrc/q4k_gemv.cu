// Dequantise-fused Q4_K matrix-vector product, streaming formulation.
//
// Work decomposition.  The matrix is a grid of units (row tile of 8 rows  x  super-block column of
// 256 weights, 1152 bytes each, see common.cuh) stored column-major, so unit index u = s*n_rt + rt
// is also its position in memory.  The grid is persistent (a fixed number of CTAs per SM); the
// U units are cut into one contiguous range per warp, so every warp streams one contiguous slice
// of HBM, and all warps get the same number of units to within one.  A warp therefore stays at
// one column s for (almost) its whole range and keeps that column's 256 activations in registers.
//
// Arithmetic.  Lane (g, t) = (lane / 4, lane % 4) owns row g of the tile and sub-blocks t and
// 4 + t of the super-block: two 16-byte nibble chunks plus the 16-byte header of its row.
// The activations of a sub-block are held as 16-bit integers x_q = round(x / s_j), with one fp32
// step s_j = max|x| / 32767 per sub-block, split into a signed high byte and an unsigned low byte.
// Nibbles are masked in place into unsigned bytes and multiplied with the 4-way byte dot product
// (dp4a): I_j = sum q * x_q is an exact integer below 2^24, so the only rounding errors are the
// 16-bit step of x (about 2e-5 of a typical activation) and a handful of fp32 operations per
// sub-block:  partial = d * sum_j sc_j * s_j * I_j  -  dmin * sum_j m_j * s_j * sum(x_q).
// With RMSNorm fused, x is multiplied by the gain before quantisation and the scalar
// rsqrt(mean(x^2) + eps) is applied to the fp32 partial.
//
// Output.  Each unit yields 8 row partials per token; they are written to
//   part[(s * n_tok + t) * mpad + row]
// and summed over s in ascending order by the finisher kernels (finish.cu), which makes the
// result independent of how the units were split over warps.
#include "common.cuh"

namespace prima {
namespace {

constexpr int kWarpsPerCta = 8;
constexpr int kPipe = 4;   // units in flight per warp

struct UnitRegs {
  uint4 h, q0, q1;
};

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 v;
  asm("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// 4-way byte dot products: unsigned nibble bytes times signed / unsigned activation bytes.
__device__ __forceinline__ int dp4a_us(uint32_t a, uint32_t b, int c) {
  int d;
  asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ uint32_t dp4a_uu(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("dp4a.u32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// The 32 activations of one sub-block as bytes: hi[2w + p] / lo[2w + p] hold the high / low bytes of
// x_q for weights 8w + p, 8w + p + 2, 8w + p + 4, 8w + p + 6 (p = 0 even nibbles, 1 odd nibbles).
struct SubX {
  uint32_t hi[8], lo[8];
  float step;       // s_j
  float step_sum;   // s_j * sum(x_q)
};

// sum over the 32 weights of q * x_q (exact)
__device__ __forceinline__ int chunk_dot(const uint4& q, const SubX& x) {
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
  int he = 0, ho = 0;
  uint32_t le = 0, lo = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint32_t e = w[i] & 0x0f0f0f0fu, o = (w[i] >> 4) & 0x0f0f0f0fu;
    he = dp4a_us(e, x.hi[2 * i], he);
    ho = dp4a_us(o, x.hi[2 * i + 1], ho);
    le = dp4a_uu(e, x.lo[2 * i], le);
    lo = dp4a_uu(o, x.lo[2 * i + 1], lo);
  }
  return (he + ho) * 256 + static_cast<int>(le + lo);
}

// Quantise 32 consecutive activations (times gain, if any) into a SubX.
__device__ __forceinline__ void load_sub(const float* __restrict__ xp, const float* __restrict__ gp, SubX& out) {
  float v[32];
  float amax = 0.f;
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    float4 a = *reinterpret_cast<const float4*>(xp + 4 * c);
    if (gp) {
      const float4 gv = *reinterpret_cast<const float4*>(gp + 4 * c);
      a.x *= gv.x; a.y *= gv.y; a.z *= gv.z; a.w *= gv.w;
    }
    v[4 * c] = a.x; v[4 * c + 1] = a.y; v[4 * c + 2] = a.z; v[4 * c + 3] = a.w;
    amax = fmaxf(amax, fmaxf(fmaxf(fabsf(a.x), fabsf(a.y)), fmaxf(fabsf(a.z), fabsf(a.w))));
  }
  const bool ok = amax > 0.f && amax < 3.0e38f;
  const float inv_step = ok ? 32767.0f / amax : 0.f;
  int sum = 0;
#pragma unroll
  for (int w = 0; w < 4; ++w) {
#pragma unroll
    for (int p = 0; p < 2; ++p) {
      uint32_t hi = 0, lo = 0;
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        int xq = __float2int_rn(v[8 * w + 2 * b + p] * inv_step);
        xq = max(-32767, min(32767, xq));
        sum += xq;
        hi |= (static_cast<uint32_t>(xq >> 8) & 0xffu) << (8 * b);
        lo |= (static_cast<uint32_t>(xq) & 0xffu) << (8 * b);
      }
      out.hi[2 * w + p] = hi;
      out.lo[2 * w + p] = lo;
    }
  }
  out.step = ok ? amax / 32767.0f : 0.f;
  out.step_sum = out.step * static_cast<float>(sum);
}

// rsqrt(mean(x^2) + eps) of one token from the statistics blocks, reduced the same way in every warp.
__device__ __forceinline__ float token_inv_rms(const float2* __restrict__ stats, int n_blocks, int tok, int64_t cols, float eps) {
  const int lane = threadIdx.x & 31;
  float ss = 0.f;
  for (int b = lane; b < n_blocks; b += 32) ss += stats[tok * kMaxStatBlocks + b].x;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  return 1.0f / sqrtf(ss / static_cast<float>(cols) + eps);
}

template <int NTOK>
__global__ void __launch_bounds__(kWarpsPerCta * 32, (NTOK == 1 ? 2 : 1))
gemv_partials_kernel(const uint8_t* __restrict__ w, int64_t n_rt, int64_t n_sb, int64_t cols, const float* __restrict__ x,
                     const float* __restrict__ gain, float eps, const float2* __restrict__ stats, int n_stat_blocks, int tok0,
                     int n_tok_total, float* __restrict__ part, int64_t mpad) {
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int64_t wg = static_cast<int64_t>(blockIdx.x) * kWarpsPerCta + warp;
  const int64_t n_warps = static_cast<int64_t>(gridDim.x) * kWarpsPerCta;
  const int64_t n_units = n_rt * n_sb;
  const int64_t u0 = n_units * wg / n_warps, u1 = n_units * (wg + 1) / n_warps;
  if (u0 >= u1) return;

  const uint8_t* lane_h = w + g * 16;
  const uint8_t* lane_q = w + kUnitHdrBytes + lane * 16;

  UnitRegs buf[kPipe];
#pragma unroll
  for (int i = 0; i < kPipe; ++i) {
    if (u0 + i < u1) {
      const int64_t off = (u0 + i) * kUnitBytes;
      buf[i].h = ldg_stream(lane_h + off);
      buf[i].q0 = ldg_stream(lane_q + off);
      buf[i].q1 = ldg_stream(lane_q + off + 512);
    }
  }

  float post[NTOK];
#pragma unroll
  for (int k = 0; k < NTOK; ++k) post[k] = gain ? token_inv_rms(stats, n_stat_blocks, tok0 + k, cols, eps) : 1.0f;

  // lane-constant byte selectors that pull this lane's 24-bit field group out of header words 1..3
  const uint32_t sel_a = t == 1 ? 0x7654u : (t == 3 ? 0x0073u : 0x3210u);
  const uint32_t sel_b = t == 2 ? 0x7654u : (t == 3 ? 0x0710u : 0x3210u);

  SubX xa[NTOK], xb[NTOK];   // sub-blocks t and 4 + t of the current column
  int64_t cur_s = -1;

  for (int64_t ub = u0; ub < u1; ub += kPipe) {
#pragma unroll
    for (int i = 0; i < kPipe; ++i) {
      const int64_t u = ub + i;
      if (u < u1) {
        const UnitRegs r = buf[i];
        if (u + kPipe < u1) {
          const int64_t off = (u + kPipe) * kUnitBytes;
          buf[i].h = ldg_stream(lane_h + off);
          buf[i].q0 = ldg_stream(lane_q + off);
          buf[i].q1 = ldg_stream(lane_q + off + 512);
        }
        const int64_t s = u / n_rt, rt = u - s * n_rt;
        if (s != cur_s) {
          cur_s = s;
#pragma unroll
          for (int k = 0; k < NTOK; ++k) {
            const float* xp = x + static_cast<int64_t>(tok0 + k) * cols + s * 256 + 32 * t;
            const float* gp = gain ? gain + s * 256 + 32 * t : nullptr;
            load_sub(xp, gp, xa[k]);
            load_sub(xp + 128, gp ? gp + 128 : nullptr, xb[k]);
          }
        }
        const float d = __half2float(__ushort_as_half(static_cast<unsigned short>(r.h.x & 0xffffu)));
        const float dmin = __half2float(__ushort_as_half(static_cast<unsigned short>(r.h.x >> 16)));
        const uint32_t f = __byte_perm(__byte_perm(r.h.y, r.h.z, sel_a), r.h.w, sel_b);
        const float sc_lo = static_cast<float>(f & 63u), sc_hi = static_cast<float>((f >> 6) & 63u);
        const float m_lo = static_cast<float>((f >> 12) & 63u), m_hi = static_cast<float>((f >> 18) & 63u);
#pragma unroll
        for (int k = 0; k < NTOK; ++k) {
          const float i0 = static_cast<float>(chunk_dot(r.q0, xa[k]));
          const float i1 = static_cast<float>(chunk_dot(r.q1, xb[k]));
          const float t1 = sc_lo * (xa[k].step * i0) + sc_hi * (xb[k].step * i1);
          const float t2 = m_lo * xa[k].step_sum + m_hi * xb[k].step_sum;
          float acc = d * t1 - dmin * t2;
          acc += __shfl_xor_sync(0xffffffffu, acc, 1);
          acc += __shfl_xor_sync(0xffffffffu, acc, 2);
          if (t == 0) part[(s * n_tok_total + tok0 + k) * mpad + rt * kRowsPerTile + g] = acc * post[k];
        }
      }
    }
  }
}

}  // namespace

int launch_gemv_partials(const TiledMat& w, const GemvIn& in, int n_tok, float* part, int sm_count, cudaStream_t st) {
  if (w.n_rt == 0 || w.n_sb == 0) return 0;
  const int64_t n_units = w.n_rt * w.n_sb;
  int launches = 0;
  const int block = kWarpsPerCta * 32;
  int tok = 0;
  while (tok < n_tok) {
    const int chunk = (n_tok - tok >= 2) ? 2 : 1;
    const int ctas_per_sm = chunk == 1 ? 2 : 1;
    int64_t grid = static_cast<int64_t>(sm_count) * ctas_per_sm;
    const int64_t max_useful = (n_units + kWarpsPerCta - 1) / kWarpsPerCta;
    if (grid > max_useful) grid = max_useful;
    if (chunk == 1)
      gemv_partials_kernel<1><<<static_cast<unsigned>(grid), block, 0, st>>>(
          w.data, w.n_rt, w.n_sb, w.cols, in.x, in.gain, in.eps, in.stats.data, in.stats.n_blocks, tok, n_tok, part, w.mpad());
    else
      gemv_partials_kernel<2><<<static_cast<unsigned>(grid), block, 0, st>>>(
          w.data, w.n_rt, w.n_sb, w.cols, in.x, in.gain, in.eps, in.stats.data, in.stats.n_blocks, tok, n_tok, part, w.mpad());
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_rc(e);
    ++launches;
    tok += chunk;
  }
  return launches;
}

}  // namespace prima
