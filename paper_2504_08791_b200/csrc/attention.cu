// Grouped-query decode attention over the fp16 KV cache, split along the context.
//
// One CTA of 8 warps per (context chunk of 128 positions, KV head); each warp owns 16 positions.
// The query rows that share the KV head -- the H/G heads of every token of the step, at most 64
// rows -- are processed 16 at a time (one m16n8k16 tile of rows).  Per tile a warp computes
//   S = Q K^T   with  A = Q (16 rows x 16 dims, fp16, pre-scaled by 1/sqrt(128)),  B = K,
//   P = exp(S - max),   O = P V   with  A = P (fp16),  B = V,
// all with fp32 accumulation on the tensor cores.  K and V go from global memory straight into
// the B-operand registers with fully used 16-byte loads: the instruction's k index is only a
// label, so each lane is given the head dimensions (for K) or positions (for V) that make its
// bytes contiguous in the cache, and Q / P are arranged to match.  The eight warps' (max, sum, O)
// are combined through shared memory, giving per query row and chunk the running maximum m, the
// sum l of exp(s - m) and the un-normalised output.  A second kernel merges the chunks of a row in
// ascending order:  M = max m_c,  o = sum_c e^(m_c - M) o_c / sum_c e^(m_c - M) l_c.
// Token t of the step attends positions 0 .. pos + t (causal inside the step).
//
// The kernel also finishes the fused QKV product that precedes it: every CTA forms the queries of
// its KV head from that product's partial sums (sum, RMSNorm factor, rotation), and the CTA whose
// chunk contains a new position forms that position's key and value, rounds them to binary16 and
// appends them to the cache before its warps read the chunk.
#include "common.cuh"

namespace prima {
namespace {

constexpr int kChunk = 128;
constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;

__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_h2(float a, float b) {
  const __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// Lane (g, t) = (lane / 4, lane % 4).
//  * S tile: instruction column n = g is position (block base + g); the lane's k slots of step ks are
//    head dims  32 (ks / 2) + 8 t + 4 (ks % 2) + {0, 1}  (first register) and  + {2, 3}  (second).
//  * O tile: instruction d of 16 has column n = g at head dim  64 (d / 8) + 8 g + (d % 8); the lane's
//    k slots are the positions  2t, 2t+1, 2t+8, 2t+9  of the warp's 16.
__global__ void __launch_bounds__(kThreads)
attn_partial_kernel(const float* __restrict__ part, int n_parts, int64_t mpad, const float* __restrict__ ssq, int n_groups,
                    float inv_width, float eps, const float2* __restrict__ rope_tab, int rope_mode, __half* __restrict__ k_cache,
                    __half* __restrict__ v_cache, int kv_capacity, int n_q_heads, int n_kv_heads, int pos, int n_tok, int n_chunks,
                    float* __restrict__ o_part, float2* __restrict__ ml_part) {
  pdl_trigger();
  extern __shared__ float dyn_smem[];
  float (*s_o)[16][kHeadDim] = reinterpret_cast<float (*)[16][kHeadDim]>(dyn_smem);   // [kWarps][16][128]
  float* q_s = dyn_smem + kWarps * 16 * kHeadDim;    // [n_rows][128] rotated queries of this KV head
  __shared__ float s_m[kWarps][16], s_l[kWarps][16];
  __shared__ float s_inv[kMaxTok];

  const int group = n_q_heads / n_kv_heads;
  const int n_rows = n_tok * group;                  // query rows served by this CTA
  const int chunk = blockIdx.x, kv = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int n_ctx = pos + n_tok;
  const int wbase = chunk * kChunk + warp * 16;      // first position of this warp

  // ---- K and V of the warp's 16 positions.  Entries below `pos` were written by earlier steps and do
  //      not change, so a warp whose positions are all old loads them before waiting for the
  //      predecessor kernel; the others load after the new entries have been appended below.
  const bool old_only = wbase + 16 <= pos;
  uint4 kreg[2][4];      // [position block of 8][32-dim slice]
  uint4 vreg[4][2];      // [k-slot position][64-dim half]
  const __half* kbase = k_cache + static_cast<int64_t>(kv) * kv_capacity * kHeadDim;
  const __half* vbase = v_cache + static_cast<int64_t>(kv) * kv_capacity * kHeadDim;
  auto load_kv = [&]() {
#pragma unroll
    for (int pb = 0; pb < 2; ++pb) {
      const int p = wbase + 8 * pb + g;
#pragma unroll
      for (int j = 0; j < 4; ++j)
        kreg[pb][j] = p < n_ctx ? __ldcg(reinterpret_cast<const uint4*>(kbase + static_cast<int64_t>(p) * kHeadDim + 32 * j + 8 * t)) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int pi = 0; pi < 4; ++pi) {
      const int p = wbase + 2 * t + (pi & 1) + 8 * (pi >> 1);
#pragma unroll
      for (int hf = 0; hf < 2; ++hf)
        vreg[pi][hf] = p < n_ctx ? __ldcg(reinterpret_cast<const uint4*>(vbase + static_cast<int64_t>(p) * kHeadDim + 64 * hf + 8 * g)) : make_uint4(0, 0, 0, 0);
    }
  };
  if (old_only) load_kv();
  pdl_wait();

  // ---- finish the QKV product for this KV head: one thread per rotation pair
  const int64_t pstride = static_cast<int64_t>(n_tok) * mpad;
  auto pair_sum = [&](int tok, int64_t row_a, int64_t row_b, float& va, float& vb) {
    va = vb = 0.f;
    int p = 0;
    for (; p + 4 <= n_parts; p += 4) {      // four loads in flight per row, additions in ascending order
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        a[i] = part[(p + i) * pstride + tok * mpad + row_a];
        b[i] = part[(p + i) * pstride + tok * mpad + row_b];
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        va += a[i];
        vb += b[i];
      }
    }
    for (; p < n_parts; ++p) {
      va += part[p * pstride + tok * mpad + row_a];
      vb += part[p * pstride + tok * mpad + row_b];
    }
  };
  if (threadIdx.x < n_tok) {
    float ss = 0.f;
    for (int gi = 0; gi < n_groups; ++gi) ss += ssq[threadIdx.x * kMaxStatBlocks + gi];
    s_inv[threadIdx.x] = 1.0f / sqrtf(ss * inv_width + eps);
  }
  __syncthreads();
  const int chunk0 = chunk * kChunk;
  for (int idx = threadIdx.x; idx < n_tok * (kHeadDim / 2); idx += kThreads) {   // new keys and values
    const int tok = idx / (kHeadDim / 2), i = idx % (kHeadDim / 2);
    const int p = pos + tok;
    if (p < chunk0 || p >= chunk0 + kChunk) continue;
    const int a = rope_mode == 0 ? i : 2 * i, b = rope_mode == 0 ? i + kHeadDim / 2 : 2 * i + 1;
    const float inv = s_inv[tok];
    float ka, kb, va, vb;
    pair_sum(tok, static_cast<int64_t>(n_q_heads + kv) * kHeadDim + a, static_cast<int64_t>(n_q_heads + kv) * kHeadDim + b, ka, kb);
    pair_sum(tok, static_cast<int64_t>(n_q_heads + n_kv_heads + kv) * kHeadDim + a,
             static_cast<int64_t>(n_q_heads + n_kv_heads + kv) * kHeadDim + b, va, vb);
    ka *= inv; kb *= inv; va *= inv; vb *= inv;
    const float2 cs = rope_tab[tok * (kHeadDim / 2) + i];
    __half* kd = k_cache + (static_cast<int64_t>(kv) * kv_capacity + p) * kHeadDim;
    __half* vd = v_cache + (static_cast<int64_t>(kv) * kv_capacity + p) * kHeadDim;
    kd[a] = __float2half_rn(ka * cs.x - kb * cs.y);
    kd[b] = __float2half_rn(kb * cs.x + ka * cs.y);
    vd[a] = __float2half_rn(va);
    vd[b] = __float2half_rn(vb);
  }
  // queries: four rotation pairs per thread and trip, their loads issued together
  const int n_pairs = n_rows * (kHeadDim / 2);
  for (int base = threadIdx.x; base < n_pairs; base += 4 * kThreads) {
    float qa_[4], qb_[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int idx = base + u * kThreads;
      qa_[u] = qb_[u] = 0.f;
      if (idx < n_pairs) {
        const int r = idx / (kHeadDim / 2), i = idx % (kHeadDim / 2);
        const int tok = r / group, head = kv * group + r % group;
        const int a = rope_mode == 0 ? i : 2 * i, b = rope_mode == 0 ? i + kHeadDim / 2 : 2 * i + 1;
        pair_sum(tok, static_cast<int64_t>(head) * kHeadDim + a, static_cast<int64_t>(head) * kHeadDim + b, qa_[u], qb_[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int idx = base + u * kThreads;
      if (idx < n_pairs) {
        const int r = idx / (kHeadDim / 2), i = idx % (kHeadDim / 2);
        const int tok = r / group;
        const int a = rope_mode == 0 ? i : 2 * i, b = rope_mode == 0 ? i + kHeadDim / 2 : 2 * i + 1;
        const float inv = s_inv[tok];
        const float x = qa_[u] * inv, y = qb_[u] * inv;
        const float2 cs = rope_tab[tok * (kHeadDim / 2) + i];
        q_s[r * kHeadDim + a] = x * cs.x - y * cs.y;
        q_s[r * kHeadDim + b] = y * cs.x + x * cs.y;
      }
    }
  }
  __syncthreads();
  if (!old_only) load_kv();

  const float scale = 0.08838834764831845f;   // 1 / sqrt(128)
  for (int tile = 0; tile * 16 < n_rows; ++tile) {
    // ---- Q fragments of rows (tile*16 + g) and (+ 8)
    uint32_t qa[8][4];
    int row_tok[2];
#pragma unroll
    for (int hr = 0; hr < 2; ++hr) {
      const int r = tile * 16 + g + 8 * hr;
      const bool live = r < n_rows;
      row_tok[hr] = live ? r / group : -1;
      const float* qr = q_s + (live ? r : 0) * kHeadDim;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
        if (live) {
          a = *reinterpret_cast<const float4*>(qr + 32 * j + 8 * t);
          b = *reinterpret_cast<const float4*>(qr + 32 * j + 8 * t + 4);
        }
        qa[2 * j][hr] = pack_h2(a.x * scale, a.y * scale);
        qa[2 * j][2 + hr] = pack_h2(a.z * scale, a.w * scale);
        qa[2 * j + 1][hr] = pack_h2(b.x * scale, b.y * scale);
        qa[2 * j + 1][2 + hr] = pack_h2(b.z * scale, b.w * scale);
      }
    }
    // ---- scores of the 16 positions: two blocks of 8
    float sc[2][4];
#pragma unroll
    for (int pb = 0; pb < 2; ++pb) {
      sc[pb][0] = sc[pb][1] = sc[pb][2] = sc[pb][3] = 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        mma_f16(sc[pb], qa[2 * j][0], qa[2 * j][1], qa[2 * j][2], qa[2 * j][3], kreg[pb][j].x, kreg[pb][j].y);
        mma_f16(sc[pb], qa[2 * j + 1][0], qa[2 * j + 1][1], qa[2 * j + 1][2], qa[2 * j + 1][3], kreg[pb][j].z, kreg[pb][j].w);
      }
    }
    // ---- mask, row maxima, exponentials
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int pb = 0; pb < 2; ++pb)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int hr = e >> 1;
        const int p = wbase + 8 * pb + 2 * t + (e & 1);
        const bool ok = row_tok[hr] >= 0 && p <= pos + row_tok[hr];
        sc[pb][e] = ok ? sc[pb][e] : -INFINITY;
        mx[hr] = fmaxf(mx[hr], sc[pb][e]);
      }
    float lsum[2];
#pragma unroll
    for (int hr = 0; hr < 2; ++hr) {
      mx[hr] = fmaxf(mx[hr], __shfl_xor_sync(0xffffffffu, mx[hr], 1));
      mx[hr] = fmaxf(mx[hr], __shfl_xor_sync(0xffffffffu, mx[hr], 2));
      lsum[hr] = 0.f;
    }
    uint32_t pa[4];
#pragma unroll
    for (int pb = 0; pb < 2; ++pb) {
      float pv[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int hr = e >> 1;
        pv[e] = mx[hr] > -INFINITY ? expf(sc[pb][e] - mx[hr]) : 0.f;
        lsum[hr] += pv[e];
      }
      pa[2 * pb] = pack_h2(pv[0], pv[1]);        // row g,   k slots of this block
      pa[2 * pb + 1] = pack_h2(pv[2], pv[3]);    // row g+8
    }
#pragma unroll
    for (int hr = 0; hr < 2; ++hr) {
      lsum[hr] += __shfl_xor_sync(0xffffffffu, lsum[hr], 1);
      lsum[hr] += __shfl_xor_sync(0xffffffffu, lsum[hr], 2);
    }
    // ---- O = P V, 16 instructions of 8 head dims each
#pragma unroll
    for (int d = 0; d < 16; ++d) {
      const int hf = d >> 3, j = (d & 7) >> 1;
      const uint32_t sel = (d & 1) ? 0x7632u : 0x5410u;
      const uint32_t* v0 = reinterpret_cast<const uint32_t*>(&vreg[0][hf]);
      const uint32_t* v1 = reinterpret_cast<const uint32_t*>(&vreg[1][hf]);
      const uint32_t* v2 = reinterpret_cast<const uint32_t*>(&vreg[2][hf]);
      const uint32_t* v3 = reinterpret_cast<const uint32_t*>(&vreg[3][hf]);
      const uint32_t b0 = __byte_perm(v0[j], v1[j], sel);
      const uint32_t b1 = __byte_perm(v2[j], v3[j], sel);
      float oc[4] = {0.f, 0.f, 0.f, 0.f};
      mma_f16(oc, pa[0], pa[1], pa[2], pa[3], b0, b1);
      const int dim = 64 * hf + (d & 7);
      s_o[warp][g][dim + 16 * t] = oc[0];
      s_o[warp][g][dim + 16 * t + 8] = oc[1];
      s_o[warp][g + 8][dim + 16 * t] = oc[2];
      s_o[warp][g + 8][dim + 16 * t + 8] = oc[3];
    }
    if (t == 0) {
      s_m[warp][g] = mx[0];
      s_m[warp][g + 8] = mx[1];
      s_l[warp][g] = lsum[0];
      s_l[warp][g + 8] = lsum[1];
    }
    __syncthreads();
    // ---- combine the warps: each group of 128 threads takes every (kThreads/128)-th row of the
    //      tile, thread d of the group owning head dim d
    {
      const int d = threadIdx.x % kHeadDim;
      for (int r = threadIdx.x / kHeadDim; r < 16 && tile * 16 + r < n_rows; r += kThreads / kHeadDim) {
        float big = -INFINITY;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) big = fmaxf(big, s_m[w][r]);
        float l = 0.f, acc = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
          const float f = s_m[w][r] > -INFINITY ? expf(s_m[w][r] - big) : 0.f;
          l += f * s_l[w][r];
          acc += f * s_o[w][r][d];
        }
        const int rr = tile * 16 + r;
        const int tok = rr / group, head = kv * group + rr % group;
        const int64_t slot = (static_cast<int64_t>(tok) * n_q_heads + head) * n_chunks + chunk;
        o_part[slot * kHeadDim + d] = acc;
        if (d == 0) ml_part[slot] = make_float2(big, l);
      }
    }
    __syncthreads();
  }
}

// One block of 128 threads per (token, head): merge the chunks in ascending order.  The weights
// e^(m_c - M) / L of all chunks are prepared first, in parallel; then thread d sums its head dim.
__global__ void __launch_bounds__(kHeadDim)
attn_merge_kernel(const float* __restrict__ o_part, const float2* __restrict__ ml_part, int n_chunks, float* __restrict__ o) {
  pdl_trigger();
  pdl_wait();
  extern __shared__ float s_w[];         // [n_chunks]
  __shared__ float s_red[4];
  const int row = blockIdx.x;            // tok * H + head
  const int d = threadIdx.x;
  const float2* ml = ml_part + static_cast<int64_t>(row) * n_chunks;
  float big = -INFINITY;
  for (int c = d; c < n_chunks; c += kHeadDim) big = fmaxf(big, ml[c].x);
#pragma unroll
  for (int of = 16; of > 0; of >>= 1) big = fmaxf(big, __shfl_xor_sync(0xffffffffu, big, of));
  if ((d & 31) == 0) s_red[d >> 5] = big;
  __syncthreads();
  big = fmaxf(fmaxf(s_red[0], s_red[1]), fmaxf(s_red[2], s_red[3]));
  for (int c = d; c < n_chunks; c += kHeadDim) {
    const float2 v = ml[c];
    s_w[c] = v.x > -INFINITY ? expf(v.x - big) : 0.f;
  }
  __syncthreads();
  // every thread forms the same denominator in chunk order
  float denom = 0.f;
  for (int c = 0; c < n_chunks; ++c) denom += s_w[c] * ml[c].y;
  float acc = 0.f;
  const float* op = o_part + static_cast<int64_t>(row) * n_chunks * kHeadDim + d;
#pragma unroll 8
  for (int c = 0; c < n_chunks; ++c) acc += s_w[c] * op[static_cast<int64_t>(c) * kHeadDim];
  const float out = acc / denom;
  o[static_cast<int64_t>(row) * kHeadDim + d] = out;
}

}  // namespace

int attention_chunk_len() { return kChunk; }

int launch_attention(const float* part_qkv, int n_parts, int64_t mpad, const SumSq& ssq, const float2* rope_tab, int rope_mode,
                     __half* k_cache, __half* v_cache, int kv_capacity, int n_q_heads, int n_kv_heads, int pos, int n_tok,
                     const AttnScratch& scr, float* o, cudaStream_t st) {
  const int n_ctx = pos + n_tok;
  const int n_chunks = (n_ctx + kChunk - 1) / kChunk;
  if (n_chunks > scr.max_chunks) return cuda_rc(cudaErrorInvalidValue);
  const int n_rows = n_tok * (n_q_heads / n_kv_heads);
  const size_t q_bytes = static_cast<size_t>(kWarps * 16 + n_rows) * kHeadDim * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(attn_partial_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (kWarps * 16 + 64) * kHeadDim * 4);
  if (e != cudaSuccess) return cuda_rc(e);
  dim3 grid(n_chunks, n_kv_heads);
  e = launch_pdl(attn_partial_kernel, grid, dim3(kThreads), q_bytes, st, part_qkv, n_parts, mpad, static_cast<const float*>(ssq.data),
                 ssq.n_groups, ssq.width > 0 ? 1.0f / static_cast<float>(ssq.width) : 0.f, ssq.eps, rope_tab, rope_mode, k_cache, v_cache,
                 kv_capacity, n_q_heads, n_kv_heads, pos, n_tok, n_chunks, scr.o_part, scr.ml_part);
  if (e != cudaSuccess) return cuda_rc(e);
  e = launch_pdl(attn_merge_kernel, dim3(n_tok * n_q_heads), dim3(kHeadDim), static_cast<size_t>(n_chunks) * sizeof(float), st, scr.o_part,
                 scr.ml_part, n_chunks, o);
  if (e != cudaSuccess) return cuda_rc(e);
  return 2;
}

}  // namespace prima
