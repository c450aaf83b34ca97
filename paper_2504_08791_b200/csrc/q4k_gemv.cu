// Dequantise-fused Q4_K matrix-vector product, streaming formulation.
//
// Work decomposition.  The matrix is a grid of units (row tile of 8 rows  x  super-block column of
// 256 weights, 1152 bytes each, see common.cuh) stored column-major, so unit index u = s*n_rt + rt
// is also its position in memory.  The grid is persistent (a fixed number of CTAs per SM); the
// U units are cut into one contiguous range per warp, so every warp streams one contiguous slice
// of HBM, and all warps get the same number of units to within one.  A warp therefore stays at
// one column s for (almost) its whole range and keeps that column's 256 activations in registers
// as binary16 pairs.
//
// Arithmetic.  Lane (g, t) = (lane / 4, lane % 4) owns row g of the tile and sub-blocks t and
// 4 + t of the super-block: two 16-byte nibble chunks plus the 16-byte header of its row.
// Nibbles are never converted: masked in place they are binary16 subnormals q * 2^-24 (or
// q * 2^-20 for the odd pairs), which HFMA2 multiplies exactly by the binary16 activations.
// Each sub-block is accumulated in two binary16x2 chains of 8 products, promoted to fp32, scaled
// by d*sc, and the -dmin*m term uses the per-sub-block activation sums held in fp32.  Activations
// are pre-scaled by a power of two chosen from the vector's max |x| so that the largest lies in
// [2^14, 2^15): products and chain sums stay well inside binary16's range and the scale is undone
// exactly on the fp32 result.
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

__device__ __forceinline__ __half2 as_h2(uint32_t v) { return *reinterpret_cast<__half2*>(&v); }

// Eight weights of one 32-bit word against four activation pairs; lo collects the pairs whose
// nibbles sit at mantissa bits 0..3 (q * 2^-24), hi those at bits 4..7 (q * 2^-20).
__device__ __forceinline__ void word_fma(uint32_t w, const __half2* x, __half2& lo, __half2& hi) {
  const uint32_t w8 = w >> 8;
  lo = __hfma2(as_h2(w & 0x000f000fu), x[0], lo);
  hi = __hfma2(as_h2(w & 0x00f000f0u), x[1], hi);
  lo = __hfma2(as_h2(w8 & 0x000f000fu), x[2], lo);
  hi = __hfma2(as_h2(w8 & 0x00f000f0u), x[3], hi);
}

// sum over 32 weights of q * xs, in units of 2^-24
__device__ __forceinline__ float chunk_dot(const uint4& q, const __half2* x) {
  __half2 lo = __float2half2_rn(0.f), hi = __float2half2_rn(0.f);
  word_fma(q.x, x + 0, lo, hi);
  word_fma(q.y, x + 4, lo, hi);
  word_fma(q.z, x + 8, lo, hi);
  word_fma(q.w, x + 12, lo, hi);
  const float2 l = __half22float2(lo), h = __half22float2(hi);
  return (l.x + l.y) + (h.x + h.y) * 0.0625f;
}

// Reduce the statistics blocks of one token the same way in every warp.
__device__ __forceinline__ void token_scale(const float2* __restrict__ stats, int n_blocks, int tok, int64_t cols,
                                            bool has_norm, float eps, float gain_max, float& mul, float& post) {
  const int lane = threadIdx.x & 31;
  float ss = 0.f, am = 0.f;
  for (int b = lane; b < n_blocks; b += 32) {
    const float2 v = stats[tok * kMaxStatBlocks + b];
    ss += v.x;
    am = fmaxf(am, v.y);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    ss += __shfl_xor_sync(0xffffffffu, ss, o);
    am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, o));
  }
  const float inv = has_norm ? 1.0f / sqrtf(ss / static_cast<float>(cols) + eps) : 1.0f;
  const float amax = am * gain_max * inv;
  int k = 0;
  if (amax > 0.f && amax < 3.0e38f) {
    int e;
    frexpf(amax, &e);        // amax < 2^e
    k = 15 - e;              // largest scaled activation < 2^15
    k = max(-100, min(100, k));
  }
  mul = ldexpf(inv, k);
  post = ldexpf(1.0f, -k);
}

template <int NTOK>
__global__ void __launch_bounds__(kWarpsPerCta * 32, (NTOK == 1 ? 2 : 1))
gemv_partials_kernel(const uint8_t* __restrict__ w, int64_t n_rt, int64_t n_sb, int64_t cols, const float* __restrict__ x,
                     const float* __restrict__ gain, float gain_max, float eps, const float2* __restrict__ stats,
                     int n_stat_blocks, int tok0, int n_tok_total, float* __restrict__ part, int64_t mpad) {
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

  float mul[NTOK], post[NTOK];
#pragma unroll
  for (int k = 0; k < NTOK; ++k)
    token_scale(stats, n_stat_blocks, tok0 + k, cols, gain != nullptr, eps, gain_max, mul[k], post[k]);

  // lane-constant byte selectors that pull this lane's 24-bit field group out of header words 1..3
  const uint32_t sel_a = t == 1 ? 0x7654u : (t == 3 ? 0x0073u : 0x3210u);
  const uint32_t sel_b = t == 2 ? 0x7654u : (t == 3 ? 0x0710u : 0x3210u);

  __half2 xr[NTOK][32];
  float x_lo[NTOK], x_hi[NTOK];
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
            float sum_lo = 0.f, sum_hi = 0.f;
#pragma unroll
            for (int hlf = 0; hlf < 2; ++hlf) {
#pragma unroll
              for (int c = 0; c < 8; ++c) {
                float4 v = *reinterpret_cast<const float4*>(xp + 128 * hlf + 4 * c);
                if (gp) {
                  const float4 gv = *reinterpret_cast<const float4*>(gp + 128 * hlf + 4 * c);
                  v.x *= gv.x; v.y *= gv.y; v.z *= gv.z; v.w *= gv.w;
                }
                const __half2 a = __floats2half2_rn(v.x * mul[k], v.y * mul[k]);
                const __half2 b = __floats2half2_rn(v.z * mul[k], v.w * mul[k]);
                xr[k][16 * hlf + 2 * c] = a;
                xr[k][16 * hlf + 2 * c + 1] = b;
                const float2 af = __half22float2(a), bf = __half22float2(b);
                if (hlf == 0) sum_lo += (af.x + af.y) + (bf.x + bf.y);
                else sum_hi += (af.x + af.y) + (bf.x + bf.y);
              }
            }
            x_lo[k] = sum_lo;
            x_hi[k] = sum_hi;
          }
        }
        const float d = __half2float(__ushort_as_half(static_cast<unsigned short>(r.h.x & 0xffffu)));
        const float dmin = __half2float(__ushort_as_half(static_cast<unsigned short>(r.h.x >> 16)));
        const uint32_t f = __byte_perm(__byte_perm(r.h.y, r.h.z, sel_a), r.h.w, sel_b);
        const float sc_lo = static_cast<float>(f & 63u), sc_hi = static_cast<float>((f >> 6) & 63u);
        const float m_lo = static_cast<float>((f >> 12) & 63u), m_hi = static_cast<float>((f >> 18) & 63u);
        const float d24 = d * 16777216.0f;
#pragma unroll
        for (int k = 0; k < NTOK; ++k) {
          const float a0 = chunk_dot(r.q0, &xr[k][0]);
          const float a1 = chunk_dot(r.q1, &xr[k][16]);
          const float t1 = sc_lo * a0 + sc_hi * a1;
          const float t2 = m_lo * x_lo[k] + m_hi * x_hi[k];
          float acc = d24 * t1 - dmin * t2;
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
          w.data, w.n_rt, w.n_sb, w.cols, in.x, in.gain, in.gain_max, in.eps, in.stats.data, in.stats.n_blocks, tok,
          n_tok, part, w.mpad());
    else
      gemv_partials_kernel<2><<<static_cast<unsigned>(grid), block, 0, st>>>(
          w.data, w.n_rt, w.n_sb, w.cols, in.x, in.gain, in.gain_max, in.eps, in.stats.data, in.stats.n_blocks, tok,
          n_tok, part, w.mpad());
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_rc(e);
    ++launches;
    tok += chunk;
  }
  return launches;
}

}  // namespace prima
