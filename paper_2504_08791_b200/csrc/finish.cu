// Finishers that are separate kernels (logits, the residual stream leaving a window, the sum over
// per-column partial sums used by the entry point that allocates nothing), the rotary table and the
// greedy argmax.
#include "common.cuh"

namespace prima {
namespace {

constexpr int kBlock = 256;

__device__ __forceinline__ float column_sum(const float* __restrict__ part, int64_t n_sb, int64_t stride, int64_t idx) {
  float sum = 0.f;
#pragma unroll 8
  for (int64_t s = 0; s < n_sb; ++s) sum += part[s * stride + idx];
  return sum;
}

// y[t][r] = scale_t * sum of the partial sums; scale_t = RMSNorm factor from ssq, or 1.
__global__ void finish_plain_kernel(const float* __restrict__ part, int64_t n_parts, int64_t mpad, int64_t rows, int n_tok,
                                    float* __restrict__ y, const float* __restrict__ ssq, int n_groups, float inv_width, float eps) {
  pdl_trigger();
  pdl_wait();
  const int tok = blockIdx.y;
  const int64_t stride = static_cast<int64_t>(n_tok) * mpad;
  float scale = 1.0f;
  if (ssq) {
    float ss = 0.f;
    for (int gi = 0; gi < n_groups; ++gi) ss += ssq[tok * kMaxStatBlocks + gi];
    scale = 1.0f / sqrtf(ss * inv_width + eps);
  }
  for (int64_t r = static_cast<int64_t>(blockIdx.x) * kBlock + threadIdx.x; r < rows; r += static_cast<int64_t>(gridDim.x) * kBlock)
    y[tok * rows + r] = scale * column_sum(part, n_parts, stride, tok * mpad + r);
}

// y[t][r] = scale_t * value(acc[t * mpad + r]); the accumulator is cleared behind the read.
__global__ void finish_acc_kernel(acc_t* __restrict__ acc, int64_t mpad, int64_t rows, int n_tok, float* __restrict__ y,
                                  const float* __restrict__ ssq, int n_groups, float inv_width, float eps) {
  pdl_trigger();
  pdl_wait();
  const int tok = blockIdx.y;
  float scale = 1.0f;
  if (ssq) {
    float ss = 0.f;
    for (int gi = 0; gi < n_groups; ++gi) ss += ssq[tok * kMaxStatBlocks + gi];
    scale = 1.0f / sqrtf(ss * inv_width + eps);
  }
  for (int64_t r = static_cast<int64_t>(blockIdx.x) * kBlock + threadIdx.x; r < mpad; r += static_cast<int64_t>(gridDim.x) * kBlock) {
    const acc_t a = __ldcg(acc + tok * mpad + r);
    acc[tok * mpad + r] = 0;
    if (r < rows) y[tok * rows + r] = scale * acc_value(a);
  }
}

// out[t][r] = h[t][r] + value(acc[t * mpad + r]) (same expression as the staging step of the GEMV,
// so a window boundary changes no bits); clears the accumulator behind the read, and zero0.
__global__ void finish_residual_kernel(acc_t* __restrict__ acc, int64_t mpad, int64_t rows, int n_tok, const float* __restrict__ h,
                                       float* __restrict__ out, acc_t* __restrict__ zero0, int64_t zero0_n) {
  pdl_trigger();
  pdl_wait();
  const int tok = blockIdx.y;
  for (int64_t r = static_cast<int64_t>(blockIdx.x) * kBlock + threadIdx.x; r < mpad; r += static_cast<int64_t>(gridDim.x) * kBlock) {
    const int64_t at = tok * mpad + acc_position(kOrderResidual, r);
    const acc_t a = __ldcg(acc + at);
    acc[at] = 0;
    if (r < rows) out[tok * rows + r] = h[tok * rows + r] + acc_value(a);
  }
  const int64_t stride = static_cast<int64_t>(gridDim.x) * gridDim.y * kBlock;
  for (int64_t i = (static_cast<int64_t>(blockIdx.y) * gridDim.x + blockIdx.x) * kBlock + threadIdx.x; i < zero0_n; i += stride) zero0[i] = 0;
}

__global__ void rope_table_kernel(float2* __restrict__ tab, int pos, int n_tok, double theta) {
  pdl_trigger();
  pdl_wait();
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_tok * (kHeadDim / 2)) return;
  const int tok = idx / (kHeadDim / 2), i = idx % (kHeadDim / 2);
  const double freq = pow(theta, -2.0 * static_cast<double>(i) / static_cast<double>(kHeadDim));
  double s, c;
  sincos(static_cast<double>(pos + tok) * freq, &s, &c);
  tab[idx] = make_float2(static_cast<float>(c), static_cast<float>(s));
}

// ---- argmax -------------------------------------------------------------------------------------
__device__ __forceinline__ void better(float& v, int& i, float ov, int oi) {
  if (ov > v || (ov == v && oi < i)) {
    v = ov;
    i = oi;
  }
}

__device__ __forceinline__ void block_argmax(float v, int i, float* out_v, int32_t* out_i) {
  __shared__ float s_v[kBlock / 32];
  __shared__ int s_i[kBlock / 32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, v, o);
    const int oi = __shfl_xor_sync(0xffffffffu, i, o);
    better(v, i, ov, oi);
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) {
    s_v[warp] = v;
    s_i[warp] = i;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int k = 1; k < static_cast<int>(blockDim.x >> 5); ++k) better(v, i, s_v[k], s_i[k]);
    *out_v = v;
    *out_i = i;
  }
}

__global__ void argmax_stage1_kernel(const float* __restrict__ logits, int64_t vocab, float* __restrict__ val,
                                     int32_t* __restrict__ idx) {
  pdl_trigger();
  pdl_wait();
  const int tok = blockIdx.y;
  float v = -INFINITY;
  int i = 0x7fffffff;
  for (int64_t r = static_cast<int64_t>(blockIdx.x) * kBlock + threadIdx.x; r < vocab; r += static_cast<int64_t>(gridDim.x) * kBlock)
    better(v, i, logits[tok * vocab + r], static_cast<int>(r));
  block_argmax(v, i, &val[tok * kArgmaxBlocks + blockIdx.x], &idx[tok * kArgmaxBlocks + blockIdx.x]);
}

__global__ void argmax_stage2_kernel(const float* __restrict__ val, const int32_t* __restrict__ idx, int n_blocks,
                                     int32_t* __restrict__ out) {
  pdl_trigger();
  pdl_wait();
  const int tok = blockIdx.x;
  float v = -INFINITY;
  int i = 0x7fffffff;
  for (int k = threadIdx.x; k < n_blocks; k += kBlock) better(v, i, val[tok * kArgmaxBlocks + k], idx[tok * kArgmaxBlocks + k]);
  __shared__ int32_t bi;
  __shared__ float sink;
  block_argmax(v, i, &sink, &bi);
  __syncthreads();
  if (threadIdx.x == 0) out[tok] = bi;
}

inline int done(int launches) {
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? launches : cuda_rc(e);
}

}  // namespace

int launch_finish_plain(const float* part, int64_t n_parts, int64_t mpad, int64_t rows, int n_tok, float* y, const SumSq& ssq,
                        cudaStream_t st) {
  dim3 grid(static_cast<unsigned>(std::min<int64_t>(1024, (rows + kBlock - 1) / kBlock)), n_tok);
  launch_pdl(finish_plain_kernel, grid, dim3(kBlock), 0, st, part, n_parts, mpad, rows, n_tok, y, static_cast<const float*>(ssq.data),
             ssq.n_groups, ssq.width > 0 ? 1.0f / static_cast<float>(ssq.width) : 0.f, ssq.eps);
  return done(1);
}

int launch_finish_acc(acc_t* acc, int64_t mpad, int64_t rows, int n_tok, float* y, const SumSq& ssq, cudaStream_t st) {
  dim3 grid(static_cast<unsigned>(std::min<int64_t>(1024, (mpad + kBlock - 1) / kBlock)), n_tok);
  launch_pdl(finish_acc_kernel, grid, dim3(kBlock), 0, st, acc, mpad, rows, n_tok, y, static_cast<const float*>(ssq.data), ssq.n_groups,
             ssq.width > 0 ? 1.0f / static_cast<float>(ssq.width) : 0.f, ssq.eps);
  return done(1);
}

int launch_finish_residual(acc_t* acc, int64_t mpad, int64_t rows, int n_tok, const float* h, float* out, acc_t* zero0, int64_t zero0_n,
                           cudaStream_t st) {
  dim3 grid(static_cast<unsigned>(std::min<int64_t>(1024, (mpad + kBlock - 1) / kBlock)), n_tok);
  launch_pdl(finish_residual_kernel, grid, dim3(kBlock), 0, st, acc, mpad, rows, n_tok, h, out, zero0, zero0_n);
  return done(1);
}

int launch_rope_table(float2* tab, int pos, int n_tok, float theta, cudaStream_t st) {
  const int n = n_tok * (kHeadDim / 2);
  launch_pdl(rope_table_kernel, dim3((n + 127) / 128), dim3(128), 0, st, tab, pos, n_tok, static_cast<double>(theta));
  return done(1);
}

int launch_argmax(const float* logits, int64_t vocab, int n_tok, float* scratch_val, int32_t* scratch_idx, int32_t* dev_out,
                  cudaStream_t st) {
  int nb = static_cast<int>((vocab + kBlock - 1) / kBlock);
  if (nb > kArgmaxBlocks) nb = kArgmaxBlocks;
  dim3 grid(nb, n_tok);
  launch_pdl(argmax_stage1_kernel, dim3(grid), dim3(kBlock), 0, st, logits, vocab, scratch_val, scratch_idx);
  launch_pdl(argmax_stage2_kernel, dim3(n_tok), dim3(kBlock), 0, st, scratch_val, scratch_idx, nb, dev_out);
  return done(2);
}

}  // namespace prima
