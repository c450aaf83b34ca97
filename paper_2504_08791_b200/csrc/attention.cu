// Grouped-query decode attention over the fp16 KV cache, split along the context.
//
// One CTA per (context chunk of 64 positions, KV head).  The CTA stages its 64 keys and 64 values
// (256 bytes each) in shared memory once and serves all query rows that share the KV head: the
// H/G query heads of every token of the step.  It produces, per query row, the chunk's running
// maximum m, the sum l of exp(s - m), and the un-normalised output sum exp(s - m) V.  A second
// kernel merges the chunks of a row in ascending order: M = max m_c,
// o = sum_c e^(m_c - M) o_c / sum_c e^(m_c - M) l_c.  Token t of the step attends positions
// 0 .. pos + t (causal inside the step); positions beyond that get weight zero.
#include "common.cuh"

namespace prima {
namespace {

constexpr int kChunk = 64;
constexpr int kThreads = 256;
constexpr int kRowHalves = kHeadDim + 8;   // padded row: conflict-free 16-byte reads down a column of rows

__global__ void __launch_bounds__(kThreads)
attn_partial_kernel(const float* __restrict__ q, const __half* __restrict__ k_cache, const __half* __restrict__ v_cache,
                    int kv_capacity, int n_q_heads, int n_kv_heads, int pos, int n_tok, int n_chunks,
                    float* __restrict__ o_part, float2* __restrict__ ml_part) {
  pdl_trigger();
  pdl_wait();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int group = n_q_heads / n_kv_heads;
  const int n_q = n_tok * group;                       // query rows served by this CTA
  __half* ks = reinterpret_cast<__half*>(smem_raw);    // [64][136]
  __half* vs = ks + kChunk * kRowHalves;               // [64][136]
  float* qs = reinterpret_cast<float*>(vs + kChunk * kRowHalves);  // [n_q][128]
  float* sc = qs + n_q * kHeadDim;                     // [n_q][64]

  const int chunk = blockIdx.x, g = blockIdx.y, tid = threadIdx.x;
  const int c0 = chunk * kChunk;
  const int n_ctx = pos + n_tok;
  const int valid = min(kChunk, n_ctx - c0);

  for (int idx = tid; idx < n_q * kHeadDim; idx += kThreads) {
    const int qi = idx >> 7, d = idx & 127;
    const int tok = qi / group, head = g * group + qi % group;
    qs[idx] = q[(static_cast<int64_t>(tok) * n_q_heads + head) * kHeadDim + d];
  }
  for (int idx = tid; idx < kChunk * 16; idx += kThreads) {
    const int row = idx >> 4, col = idx & 15;
    uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
    if (row < valid) {
      const int64_t off = (static_cast<int64_t>(g) * kv_capacity + c0 + row) * kHeadDim + col * 8;
      kv = *reinterpret_cast<const uint4*>(k_cache + off);
      vv = *reinterpret_cast<const uint4*>(v_cache + off);
    }
    *reinterpret_cast<uint4*>(ks + row * kRowHalves + col * 8) = kv;
    *reinterpret_cast<uint4*>(vs + row * kRowHalves + col * 8) = vv;
  }
  __syncthreads();

  // scores
  const float scale = 0.08838834764831845f;   // 1 / sqrt(128)
  for (int idx = tid; idx < n_q * kChunk; idx += kThreads) {
    const int qi = idx >> 6, j = idx & 63;
    const int tok = qi / group;
    float s = -INFINITY;
    if (j < valid && c0 + j <= pos + tok) {
      const __half* kr = ks + j * kRowHalves;
      const float* qr = qs + qi * kHeadDim;
      float acc = 0.f;
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        const uint4 kv = *reinterpret_cast<const uint4*>(kr + c * 8);
        const float4 q0 = *reinterpret_cast<const float4*>(qr + c * 8);
        const float4 q1 = *reinterpret_cast<const float4*>(qr + c * 8 + 4);
        const float2 k0 = __half22float2(*reinterpret_cast<const __half2*>(&kv.x));
        const float2 k1 = __half22float2(*reinterpret_cast<const __half2*>(&kv.y));
        const float2 k2 = __half22float2(*reinterpret_cast<const __half2*>(&kv.z));
        const float2 k3 = __half22float2(*reinterpret_cast<const __half2*>(&kv.w));
        acc = fmaf(q0.x, k0.x, acc); acc = fmaf(q0.y, k0.y, acc);
        acc = fmaf(q0.z, k1.x, acc); acc = fmaf(q0.w, k1.y, acc);
        acc = fmaf(q1.x, k2.x, acc); acc = fmaf(q1.y, k2.y, acc);
        acc = fmaf(q1.z, k3.x, acc); acc = fmaf(q1.w, k3.y, acc);
      }
      s = acc * scale;
    }
    sc[idx] = s;
  }
  __syncthreads();

  // per-row maximum, exponentials and their sum: one warp per query row
  const int warp = tid >> 5, lane = tid & 31;
  for (int qi = warp; qi < n_q; qi += kThreads / 32) {
    const float s0 = sc[qi * kChunk + lane], s1 = sc[qi * kChunk + lane + 32];
    float m = fmaxf(s0, s1);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float p0 = 0.f, p1 = 0.f;
    if (m > -INFINITY) {
      p0 = expf(s0 - m);
      p1 = expf(s1 - m);
    }
    float l = p0 + p1;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    sc[qi * kChunk + lane] = p0;
    sc[qi * kChunk + lane + 32] = p1;
    if (lane == 0) {
      const int tok = qi / group, head = g * group + qi % group;
      ml_part[(static_cast<int64_t>(tok) * n_q_heads + head) * n_chunks + chunk] = make_float2(m, l);
    }
  }
  __syncthreads();

  // weighted values: each thread owns two adjacent output lanes of one query row at a time
  for (int idx = tid; idx < n_q * (kHeadDim / 2); idx += kThreads) {
    const int qi = idx >> 6, d = (idx & 63) * 2;
    const float* pr = sc + qi * kChunk;
    float ax = 0.f, ay = 0.f;
    for (int j = 0; j < valid; ++j) {
      const float2 v = __half22float2(*reinterpret_cast<const __half2*>(vs + j * kRowHalves + d));
      const float p = pr[j];
      ax = fmaf(p, v.x, ax);
      ay = fmaf(p, v.y, ay);
    }
    const int tok = qi / group, head = g * group + qi % group;
    float* dst = o_part + ((static_cast<int64_t>(tok) * n_q_heads + head) * n_chunks + chunk) * kHeadDim + d;
    *reinterpret_cast<float2*>(dst) = make_float2(ax, ay);
  }
}

// One block of 128 threads per (token, head): merge the chunks in ascending order.
__global__ void attn_merge_kernel(const float* __restrict__ o_part, const float2* __restrict__ ml_part, int n_chunks,
                                  int n_q_heads, float* __restrict__ o, float2* __restrict__ stats) {
  pdl_trigger();
  pdl_wait();
  const int row = blockIdx.x;            // tok * H + head
  const int d = threadIdx.x;
  const float2* ml = ml_part + static_cast<int64_t>(row) * n_chunks;
  float big = -INFINITY;
  for (int c = 0; c < n_chunks; ++c) big = fmaxf(big, ml[c].x);
  float denom = 0.f, acc = 0.f;
  for (int c = 0; c < n_chunks; ++c) {
    const float2 v = ml[c];
    if (v.x > -INFINITY) {
      const float w = expf(v.x - big);
      denom += w * v.y;
      acc += w * o_part[(static_cast<int64_t>(row) * n_chunks + c) * kHeadDim + d];
    }
  }
  const float out = acc / denom;
  o[static_cast<int64_t>(row) * kHeadDim + d] = out;

  __shared__ float s_ss[4], s_am[4];
  float ss = out * out, am = fabsf(out);
#pragma unroll
  for (int of = 16; of > 0; of >>= 1) {
    ss += __shfl_xor_sync(0xffffffffu, ss, of);
    am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, of));
  }
  if ((d & 31) == 0) {
    s_ss[d >> 5] = ss;
    s_am[d >> 5] = am;
  }
  __syncthreads();
  if (d == 0) {
    const int tok = row / n_q_heads, head = row % n_q_heads;
    stats[tok * kMaxStatBlocks + head] =
        make_float2((s_ss[0] + s_ss[1]) + (s_ss[2] + s_ss[3]), fmaxf(fmaxf(s_am[0], s_am[1]), fmaxf(s_am[2], s_am[3])));
  }
}

}  // namespace

int attention_chunk_len() { return kChunk; }

int launch_attention(const float* q, const __half* k_cache, const __half* v_cache, int kv_capacity, int n_q_heads,
                     int n_kv_heads, int pos, int n_tok, const AttnScratch& scr, float* o, VecStats* stats, cudaStream_t st) {
  const int n_ctx = pos + n_tok;
  const int n_chunks = (n_ctx + kChunk - 1) / kChunk;
  if (n_chunks > scr.max_chunks) return cuda_rc(cudaErrorInvalidValue);
  const int group = n_q_heads / n_kv_heads;
  const int n_q = n_tok * group;
  const size_t smem = 2 * kChunk * kRowHalves * sizeof(__half) + static_cast<size_t>(n_q) * (kHeadDim + kChunk) * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(attn_partial_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
  if (e != cudaSuccess) return cuda_rc(e);
  dim3 grid(n_chunks, n_kv_heads);
  e = launch_pdl(attn_partial_kernel, grid, dim3(kThreads), smem, st, q, k_cache, v_cache, kv_capacity, n_q_heads, n_kv_heads, pos, n_tok,
                                                    n_chunks, scr.o_part, scr.ml_part);
  if (e != cudaSuccess) return cuda_rc(e);
  e = launch_pdl(attn_merge_kernel, dim3(n_tok * n_q_heads), dim3(kHeadDim), 0, st, scr.o_part, scr.ml_part, n_chunks, n_q_heads, o, stats->data);
  if (e != cudaSuccess) return cuda_rc(e);
  stats->n_blocks = n_q_heads;
  return 2;
}

}  // namespace prima
