// Finishers of the streaming GEMV (sum of per-column partials in ascending order + the fused
// element-wise step that follows the projection), activation statistics, rotary table, argmax.
#include "common.cuh"

namespace prima {
namespace {

constexpr int kBlock = 256;

// Deterministic block reduction of (sum, max): shuffle tree inside each warp, then thread 0 adds
// the warp results in warp order.
__device__ __forceinline__ void block_stats(float ss, float am, float2* out) {
  __shared__ float s_ss[kBlock / 32], s_am[kBlock / 32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    ss += __shfl_xor_sync(0xffffffffu, ss, o);
    am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, o));
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) {
    s_ss[warp] = ss;
    s_am[warp] = am;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    float a = 0.f, b = 0.f;
    for (int i = 0; i < static_cast<int>(blockDim.x >> 5); ++i) {
      a += s_ss[i];
      b = fmaxf(b, s_am[i]);
    }
    *out = make_float2(a, b);
  }
}

__device__ __forceinline__ float column_sum(const float* __restrict__ part, int64_t n_sb, int64_t stride, int64_t idx) {
  float sum = 0.f;
#pragma unroll 8
  for (int64_t s = 0; s < n_sb; ++s) sum += part[s * stride + idx];
  return sum;
}

__global__ void finish_plain_kernel(const float* __restrict__ part, int64_t n_sb, int64_t mpad, int64_t rows, int n_tok,
                                    float* __restrict__ y) {
  pdl_trigger();
  pdl_wait();
  const int tok = blockIdx.y;
  const int64_t stride = static_cast<int64_t>(n_tok) * mpad;
  for (int64_t r = static_cast<int64_t>(blockIdx.x) * kBlock + threadIdx.x; r < rows; r += static_cast<int64_t>(gridDim.x) * kBlock)
    y[tok * rows + r] = column_sum(part, n_sb, stride, tok * mpad + r);
}

__global__ void finish_residual_kernel(const float* __restrict__ part, int64_t n_sb, int64_t mpad, int64_t rows, int n_tok,
                                       float* __restrict__ h, float2* __restrict__ stats) {
  pdl_trigger();
  pdl_wait();
  const int tok = blockIdx.y;
  const int64_t stride = static_cast<int64_t>(n_tok) * mpad;
  float ss = 0.f, am = 0.f;
  for (int64_t r = static_cast<int64_t>(blockIdx.x) * kBlock + threadIdx.x; r < rows; r += static_cast<int64_t>(gridDim.x) * kBlock) {
    const float v = h[tok * rows + r] + column_sum(part, n_sb, stride, tok * mpad + r);
    h[tok * rows + r] = v;
    ss += v * v;
    am = fmaxf(am, fabsf(v));
  }
  block_stats(ss, am, &stats[tok * kMaxStatBlocks + blockIdx.x]);
}

__global__ void finish_swiglu_kernel(const float* __restrict__ part, int64_t n_sb, int64_t mpad, int64_t ffn, int n_tok,
                                     float* __restrict__ act, float2* __restrict__ stats) {
  pdl_trigger();
  pdl_wait();
  const int tok = blockIdx.y;
  const int64_t stride = static_cast<int64_t>(n_tok) * mpad;
  float ss = 0.f, am = 0.f;
  for (int64_t r = static_cast<int64_t>(blockIdx.x) * kBlock + threadIdx.x; r < ffn; r += static_cast<int64_t>(gridDim.x) * kBlock) {
    float gate = 0.f, up = 0.f;
#pragma unroll 8
    for (int64_t s = 0; s < n_sb; ++s) {
      const float2 v = *reinterpret_cast<const float2*>(part + s * stride + tok * mpad + 2 * r);
      gate += v.x;
      up += v.y;
    }
    const float v = gate / (1.0f + expf(-gate)) * up;
    act[tok * ffn + r] = v;
    ss += v * v;
    am = fmaxf(am, fabsf(v));
  }
  block_stats(ss, am, &stats[tok * kMaxStatBlocks + blockIdx.x]);
}

// One block of 64 threads per (head, token); thread i owns one rotation pair.
__global__ void finish_qkv_kernel(const float* __restrict__ part, int64_t n_sb, int64_t mpad, int n_q_heads, int n_kv_heads,
                                  int n_tok, const float2* __restrict__ rope_tab, int rope_mode, float* __restrict__ q_out,
                                  __half* __restrict__ k_cache, __half* __restrict__ v_cache, int kv_capacity, int pos) {
  pdl_trigger();
  pdl_wait();
  const int head = blockIdx.x, tok = blockIdx.y, i = threadIdx.x;
  const int64_t stride = static_cast<int64_t>(n_tok) * mpad;
  const int a = rope_mode == 0 ? i : 2 * i;
  const int b = rope_mode == 0 ? i + kHeadDim / 2 : 2 * i + 1;
  const int64_t row0 = static_cast<int64_t>(head) * kHeadDim;
  float va = column_sum(part, n_sb, stride, tok * mpad + row0 + a);
  float vb = column_sum(part, n_sb, stride, tok * mpad + row0 + b);
  if (head < n_q_heads + n_kv_heads) {
    const float2 cs = rope_tab[tok * (kHeadDim / 2) + i];
    const float ra = va * cs.x - vb * cs.y;
    const float rb = vb * cs.x + va * cs.y;
    va = ra;
    vb = rb;
  }
  if (head < n_q_heads) {
    float* q = q_out + (static_cast<int64_t>(tok) * n_q_heads + head) * kHeadDim;
    q[a] = va;
    q[b] = vb;
  } else {
    const bool is_k = head < n_q_heads + n_kv_heads;
    const int gk = is_k ? head - n_q_heads : head - n_q_heads - n_kv_heads;
    __half* dst = (is_k ? k_cache : v_cache) + (static_cast<int64_t>(gk) * kv_capacity + pos + tok) * kHeadDim;
    dst[a] = __float2half_rn(va);
    dst[b] = __float2half_rn(vb);
  }
}

__global__ void copy_stats_kernel(const float* __restrict__ src, float* __restrict__ dst, int64_t width,
                                  float2* __restrict__ stats) {
  pdl_trigger();
  pdl_wait();
  const int tok = blockIdx.y;
  float ss = 0.f, am = 0.f;
  for (int64_t r = static_cast<int64_t>(blockIdx.x) * kBlock + threadIdx.x; r < width; r += static_cast<int64_t>(gridDim.x) * kBlock) {
    const float v = src[tok * width + r];
    if (dst) dst[tok * width + r] = v;
    ss += v * v;
    am = fmaxf(am, fabsf(v));
  }
  block_stats(ss, am, &stats[tok * kMaxStatBlocks + blockIdx.x]);
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

int stat_blocks_for(int64_t width) {
  int64_t nb = (width + kBlock - 1) / kBlock;
  if (nb < 1) nb = 1;
  if (nb > kMaxStatBlocks) nb = kMaxStatBlocks;
  return static_cast<int>(nb);
}

inline int done(int launches) {
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? launches : cuda_rc(e);
}

}  // namespace

int launch_finish_plain(const float* part, int64_t n_sb, int64_t mpad, int64_t rows, int n_tok, float* y, cudaStream_t st) {
  dim3 grid(static_cast<unsigned>((rows + kBlock - 1) / kBlock > 1024 ? 1024 : (rows + kBlock - 1) / kBlock), n_tok);
  launch_pdl(finish_plain_kernel, dim3(grid), dim3(kBlock), 0, st, part, n_sb, mpad, rows, n_tok, y);
  return done(1);
}

int launch_finish_residual(const float* part, int64_t n_sb, int64_t mpad, int64_t rows, int n_tok, float* h, VecStats* stats,
                           cudaStream_t st) {
  const int nb = stat_blocks_for(rows);
  dim3 grid(nb, n_tok);
  launch_pdl(finish_residual_kernel, dim3(grid), dim3(kBlock), 0, st, part, n_sb, mpad, rows, n_tok, h, stats->data);
  stats->n_blocks = nb;
  return done(1);
}

int launch_finish_swiglu(const float* part, int64_t n_sb, int64_t mpad, int64_t ffn, int n_tok, float* act, VecStats* stats,
                         cudaStream_t st) {
  const int nb = stat_blocks_for(ffn);
  dim3 grid(nb, n_tok);
  launch_pdl(finish_swiglu_kernel, dim3(grid), dim3(kBlock), 0, st, part, n_sb, mpad, ffn, n_tok, act, stats->data);
  stats->n_blocks = nb;
  return done(1);
}

int launch_finish_qkv(const float* part, int64_t n_sb, int64_t mpad, int n_q_heads, int n_kv_heads, int n_tok,
                      const float2* rope_tab, int rope_mode, float* q_out, __half* k_cache, __half* v_cache, int kv_capacity,
                      int pos, cudaStream_t st) {
  dim3 grid(n_q_heads + 2 * n_kv_heads, n_tok);
  launch_pdl(finish_qkv_kernel, dim3(grid), dim3(kHeadDim / 2), 0, st, part, n_sb, mpad, n_q_heads, n_kv_heads, n_tok, rope_tab, rope_mode, q_out,
                                                   k_cache, v_cache, kv_capacity, pos);
  return done(1);
}

int launch_copy_stats(const float* src, float* dst, int64_t width, int n_tok, VecStats* stats, cudaStream_t st) {
  const int nb = stat_blocks_for(width);
  dim3 grid(nb, n_tok);
  launch_pdl(copy_stats_kernel, dim3(grid), dim3(kBlock), 0, st, src, dst, width, stats->data);
  stats->n_blocks = nb;
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
