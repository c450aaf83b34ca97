// Grouped-query decode attention over the fp16 KV cache, split along the context.
//
// The context is cut into chunks of 128 positions, 16 positions per warp.  The query rows that share a KV head --
// the H/G heads of every token of the step, at most 64 rows -- are processed 16 at a time (one m16n8k16 tile of
// rows).  Per tile a warp computes
//   S = Q K^T   with  A = Q (16 rows x 16 dims, fp16, pre-scaled by 1/sqrt(128)),  B = K,
//   P = exp(S - max),   O = P V   with  A = P (fp16),  B = V,
// all with fp32 accumulation on the tensor cores, and keeps per query row the running maximum m, the sum l of
// exp(s - m) and the un-normalised output.  A CTA combines its warps through shared memory and leaves one partial
// result per row; attn_merge_kernel merges the partial results of a row in ascending order:
//   M = max m_c,  o = sum_c e^(m_c - M) o_c / sum_c e^(m_c - M) l_c.
// Token t of the step attends positions 0 .. pos + t (causal inside the step).
//
// The kernels also finish the fused QKV product that precedes them: every CTA forms the queries it needs from that
// product's accumulators (RMSNorm factor, rotation); the CTA that owns the step's new positions also forms the new
// keys and values, rounds them to binary16, appends them to the cache and keeps a copy in shared memory, from which
// they are used (the cache is never read back inside the kernel).
//
// Two kernels.
//  * attn_one_kernel: at most eight query rows per KV head (one token), fewer than about ten thousand positions.
//    Two CTAs per SM, one per (slot of chunks, KV head).  K and V go from global memory straight into the B-operand
//    registers with fully used 16-byte loads: the instruction's k index is only a label, so each lane is given the
//    head dimensions (for K) or positions (for V) that make its bytes contiguous in the cache, and Q / P are
//    arranged to match.  A CTA that takes several chunks carries its running state from chunk to chunk in per-warp
//    tiles in shared memory.  Optionally (PRIMA_ATTN_MERGE=fused) the merge is part of the kernel: every CTA of a
//    KV head takes a ticket after it has written its partial result, and the CTA that draws the last ticket --
//    nobody waits for anybody -- combines all of them in ascending order and writes the output rows.
//  * attn_tile_kernel<T>: steps of several tokens (T tiles of 16 rows per KV head), steps of several requests (one
//    tile per request, grid.z = request, its own cache and position) and one-token steps on long contexts.  One CTA
//    per SM; keys and values are streamed through shared-memory rings of asynchronous copies and read with
//    ldmatrix; queries and the running output tile stay in registers (see the comment at the kernel).
//
// Cache entries below `stable_below` were written before the host last waited for the stream, or by a
// kernel at least one full step upstream whose completion the host has observed; only those are read
// before the dependency wait.  Entries in [stable_below, pos) were appended by earlier steps that may
// still be in flight when this kernel starts (programmatic dependent launch orders nothing before the
// wait), so they are read after it.
//
// At short contexts latency matters more than bandwidth (the whole cache of a layer is a few microseconds of HBM
// time): old entries are requested before the wait for the predecessor kernel, all loads of the finishing step are
// issued together, and the shared-memory tiles are padded (and in attn_one_kernel swizzled) so that neither their
// stores nor their reads conflict.
#include <cstdlib>

#include "common.cuh"

namespace prima {
bool attention_merge_is_fused();
namespace {

constexpr int kChunk = 128;
constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kRowPad = kHeadDim + 4;   // floats per row of the shared-memory tiles
constexpr int kMergePre = 40;           // chunks whose partial outputs the merge kernel requests up front

__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_h2(float a, float b) {
  const __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// Column of head dim `dim` inside a padded row: blocks of 8 floats are exchanged pairwise in the
// upper half of every 64, which spreads a quad's 16-byte stores (16 floats apart) over all banks.
__device__ __forceinline__ int swz(int dim) { return dim ^ (((dim >> 5) & 1) << 3); }

// Lane (g, t) = (lane / 4, lane % 4).
//  * S tile: instruction column n = g is position (block base + g); the lane's k slots of step ks are
//    head dims  32 (ks / 2) + 8 t + 4 (ks % 2) + {0, 1}  (first register) and  + {2, 3}  (second).
//  * O tile: instruction d of 16 has column n = g at head dim  64 (d / 8) + 8 g + (d % 8); the lane's
//    k slots are the positions  2t, 2t+1, 2t+8, 2t+9  of the warp's 16.  Over the eight instructions
//    of one 64-dim half a lane therefore collects, for row g, the 16 consecutive head dims
//    64 hf + 16 t + [0, 16)  (element 0 of instruction b -> + b, element 1 -> + 8 + b).

// ---- a step of several tokens of one sequence: up to 64 query rows per KV head --------------------------
// The query rows of a KV head (tokens x heads of the group) are cut into T tiles of 16 (one m16n8k16 tile of rows
// each).  One CTA per SM; CTA (x, KV head) takes the chunks x, x + gridDim.x, ... of the cached positions [0, pos)
// and serves all T tiles, so the cache is read once.  Its warps form P teams of T warps: a team takes every P-th
// sub-chunk of 16 positions of the CTA's chunks and streams it through a ring of its own in shared memory
// (asynchronous 16-byte copies, issued by the team's threads together, run S - 1 sub-chunks ahead of the one being
// computed; the only synchronisation in the loop is the team's own named barrier), and warp tt of the team applies
// the staged keys and values to tile tt.  Keys and values reach the tensor-core instructions through ldmatrix (rows
// padded to 272 bytes, so the eight rows of a matrix fall in different banks), the rotated, scaled queries stay in
// registers as fp16 fragments, and so does the warp's running output tile (fp32), rescaled only when a row's
// maximum moved.  The positions of this step itself are not read from the cache: the CTA that owns them (the one
// after the last cached chunk, round robin) forms their keys and values from the QKV accumulators, appends them to
// the cache, and its team 0 takes them as one more sub-chunk under the causal mask.  Every CTA leaves one partial
// result (running max, sum, output) per row; the merge kernel sees gridDim.x of them.
constexpr int kStageRow = kHeadDim * 2 + 16;             // bytes of a staged row of 128 halfs
constexpr int kStageHalf = 16 * kStageRow;               // keys (or values) of 16 positions
constexpr int kStageBytes = 2 * kStageHalf;              // keys, then values
constexpr int kSubPerChunk = kChunk / 16;
template <int T>
struct TileShape {
  static constexpr int kTeams = T == 1 ? 8 : (T == 4 ? 3 : 4);
  static constexpr int kStagesOf = T == 1 ? 3 : (T == 4 ? 6 : 5);
  static constexpr int kWarpsOf = kTeams * T;
  static constexpr int kRing = kTeams * kStagesOf * kStageBytes;
  static constexpr size_t kSmem = static_cast<size_t>(kRing) + static_cast<size_t>(16 * T) * kStageRow + static_cast<size_t>(2) * kMaxStepTok * kHeadDim * sizeof(__half);
  static_assert(kWarpsOf * 16 * kRowPad * sizeof(float) <= kRing, "the warps' output tiles go over the ring");
};

__device__ __forceinline__ void cp_async16_zfill(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
// The T warps of team `team` meet (T == 1: the warp's own lanes).
template <int T>
__device__ __forceinline__ void team_sync(int team) {
  if (T == 1) __syncwarp();
  else asm volatile("bar.sync %0, %1;" ::"r"(1 + team), "n"(32 * T) : "memory");
}

// 2^x by the special-function unit (2 ulp; 2^-inf = 0).
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int T>
__global__ void __launch_bounds__(TileShape<T>::kWarpsOf * 32, 1)
attn_tile_kernel(const acc_t* __restrict__ acc, int64_t mpad, const float* __restrict__ ssq, int n_groups, float inv_width, float eps,
                 const float2* __restrict__ rope_tab, int rope_mode, __half* __restrict__ k_cache, __half* __restrict__ v_cache,
                 int kv_capacity, int n_q_heads, int n_kv_heads, int pos, int stable_below, int n_tok, int part_stride,
                 float* __restrict__ o_part, float2* __restrict__ ml_part, const AttnSeqs seqs, const Stamp stamp, const L2Ahead ahead, int* status) {
  using Shape = TileShape<T>;
  constexpr int P = Shape::kTeams, S = Shape::kStagesOf, W = Shape::kWarpsOf, kThr = W * 32;
  pdl_trigger();
  int row_base = 0;                 // first output row (request * heads) of this CTA's request
  if (seqs.n > 0) {                 // one request per blockIdx.z, one token each: its own cache and position
    const int tq = blockIdx.z;
    k_cache = seqs.k[tq];
    v_cache = seqs.v[tq];
    pos = seqs.pos[tq];
    acc += tq * mpad;
    ssq += tq * kMaxStatBlocks;
    rope_tab += tq * (kHeadDim / 2);
    row_base = tq * n_q_heads;
  }
  extern __shared__ __align__(16) uint8_t tile_smem[];
  __shared__ float s_m[W][16], s_l[W][16], s_f[W][16], s_big[T][16];
  __shared__ float s_inv[kMaxStepTok];

  const int group = n_q_heads / n_kv_heads;
  const int n_rows = n_tok * group;                  // query rows of this KV head (at most 16 T)
  float* s_o = reinterpret_cast<float*>(tile_smem);                       // [W][16][kRowPad], over the ring once the loop is done
  __half* q_h = reinterpret_cast<__half*>(tile_smem + Shape::kRing);      // [16 T][kStageRow / 2] rotated, scaled queries
  __half* new_k = q_h + 16 * T * (kStageRow / 2);                         // [n_tok][128] keys of the new positions
  __half* new_v = new_k + kMaxStepTok * kHeadDim;

  const int kv = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int team = warp / T, tt = warp % T, tl = tt * 32 + lane;      // thread tl of 32 T in its team
  const int g = lane >> 2, t = lane & 3;
  const int gx = static_cast<int>(gridDim.x), bx = static_cast<int>(blockIdx.x);
  const int n_old = (pos + kChunk - 1) / kChunk;     // chunks that hold cached positions
  const bool owns_new = bx == n_old % gx;

  const __half* kbase = k_cache + static_cast<int64_t>(kv) * kv_capacity * kHeadDim;
  const __half* vbase = v_cache + static_cast<int64_t>(kv) * kv_capacity * kHeadDim;
  uint8_t* my_ring = tile_smem + team * (S * kStageBytes);
  const uint32_t ring_u32 = static_cast<uint32_t>(__cvta_generic_to_shared(my_ring));
  // Sub-chunk i of this team is the (team + i P)-th sub-chunk of the CTA's chunks; rows at or above pos are zeros.
  const int n_cta_sub = bx < n_old ? ((n_old - 1 - bx) / gx + 1) * kSubPerChunk : 0;
  const int n_sub = n_cta_sub > team ? (n_cta_sub - team - 1) / P + 1 : 0;
  auto wbase_of = [&](int i) {
    const int j = team + i * P;
    return (bx + (j / kSubPerChunk) * gx) * kChunk + (j % kSubPerChunk) * 16;
  };
  // This thread's pieces of a sub-chunk: 16 bytes number tl % 16 of the rows tl / 16 + 2 T u.
  const int piece = tl & 15, r_first = tl >> 4;
  auto issue = [&](int i) {
    if (i < n_sub) {
      const int wbase = wbase_of(i);
      if (wbase < pos) {
        const uint32_t dst = ring_u32 + (i % S) * kStageBytes + r_first * kStageRow + 16 * piece;
        const int64_t off = static_cast<int64_t>(wbase + r_first) * kHeadDim + 8 * piece;
        const bool whole = wbase + 16 <= pos;
#pragma unroll
        for (int u = 0; u < (16 + 2 * T - 1) / (2 * T); ++u) {
          const int r = r_first + 2 * T * u;
          if (16 % (2 * T) == 0 || r < 16) {
            const bool in = whole || wbase + r < pos;
            const int64_t src = in ? off + u * (2 * T * kHeadDim) : 0;      // a row at or above pos: nothing is read, zeros are written
            cp_async16_zfill(dst + u * (2 * T * kStageRow), kbase + src, in ? 16u : 0u);
            cp_async16_zfill(dst + kStageHalf + u * (2 * T * kStageRow), vbase + src, in ? 16u : 0u);
          }
        }
      }
    }
    cp_async_commit();
  };
  // Cached positions below the watermark may be requested before the dependency wait; a sub-chunk that reaches above
  // it, and all that follow it, after the wait.
  const int pre_limit = min(pos, stable_below);
  int issued = 0;
  while (issued < S - 1 && (issued >= n_sub || wbase_of(issued) + 16 <= pre_limit || wbase_of(issued) >= pos)) issue(issued++);
  pdl_wait();
  stamp_begin(stamp);
  if (threadIdx.x == 0) l2_ahead(ahead, blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z), gridDim.x * gridDim.y * gridDim.z);
  while (issued < S - 1) issue(issued++);

  // ---- finish the QKV product for this KV head.  Items: one rotation pair of a query row, and for the CTA that owns
  //      the new positions also one pair of each new key and value.
  // 1 / sqrt(128) times log2(e): scores come out in units of log2, so that every exponential is a bare ex2; the
  // running maximum handed to the merge is converted back
  const float scale = 0.08838834764831845f * 1.4426950408889634f;
  const int n_q_items = n_rows * (kHeadDim / 2);
  const int n_items = n_q_items + (owns_new ? 2 * n_tok * (kHeadDim / 2) : 0);      // at most 4096 + 1024
  constexpr int kTrip = 8;
  for (int trip = 0; trip * kTrip * kThr < n_items; ++trip) {      // same trip count for every thread
    const int base = trip * kTrip * kThr + threadIdx.x;
    acc_t ra[kTrip], rb[kTrip];
    float2 cs[kTrip];
#pragma unroll
    for (int u = 0; u < kTrip; ++u) {
      const int idx = base + u * kThr;
      if (idx < n_items) {
        int tok, rowbase;
        const int i = idx % (kHeadDim / 2);
        if (idx < n_q_items) {
          const int r = idx / (kHeadDim / 2);
          tok = r / group;
          rowbase = (kv * group + r % group) * kHeadDim;
        } else {
          const int j = (idx - n_q_items) / (kHeadDim / 2);      // 0 .. 2 n_tok - 1: keys, then values
          tok = j % n_tok;
          rowbase = (n_q_heads + (j < n_tok ? 0 : n_kv_heads) + kv) * kHeadDim;
        }
        const int a = rope_mode == 0 ? i : 2 * i, b = rope_mode == 0 ? i + kHeadDim / 2 : 2 * i + 1;
        ra[u] = __ldcg(acc + tok * mpad + rowbase + a);
        rb[u] = __ldcg(acc + tok * mpad + rowbase + b);
        cs[u] = __ldcg(rope_tab + tok * (kHeadDim / 2) + i);
      }
    }
    if (trip == 0) {      // the RMSNorm factors, loaded while the accumulators are on their way
      if (threadIdx.x < n_tok) {
        float ss = 0.f;
        for (int gi = 0; gi < n_groups; ++gi) ss += __ldcg(ssq + threadIdx.x * kMaxStatBlocks + gi);
        s_inv[threadIdx.x] = 1.0f / sqrtf(ss * inv_width + eps);
      }
      __syncthreads();
    }
#pragma unroll
    for (int u = 0; u < kTrip; ++u) {
      const int idx = base + u * kThr;
      if (idx < n_items) {
        const int i = idx % (kHeadDim / 2);
        const int a = rope_mode == 0 ? i : 2 * i, b = rope_mode == 0 ? i + kHeadDim / 2 : 2 * i + 1;
        if (idx < n_q_items) {
          const int r = idx / (kHeadDim / 2);
          const float inv = s_inv[r / group];
          const float x = acc_value(ra[u]) * inv, y = acc_value(rb[u]) * inv;
          q_h[r * (kStageRow / 2) + a] = __float2half_rn((x * cs[u].x - y * cs[u].y) * scale);
          q_h[r * (kStageRow / 2) + b] = __float2half_rn((y * cs[u].x + x * cs[u].y) * scale);
        } else {
          const int j = (idx - n_q_items) / (kHeadDim / 2);
          const int tok = j % n_tok;
          const bool is_v = j >= n_tok;
          const float inv = s_inv[tok];
          const float x = acc_value(ra[u]) * inv, y = acc_value(rb[u]) * inv;
          const __half ha = __float2half_rn(is_v ? x : x * cs[u].x - y * cs[u].y);
          const __half hb = __float2half_rn(is_v ? y : y * cs[u].x + x * cs[u].y);
          __half* sm = (is_v ? new_v : new_k) + tok * kHeadDim;
          sm[a] = ha;
          sm[b] = hb;
          if (in_range(pos + tok >= 0 && pos + tok < kv_capacity, status)) {
            __half* gd = (is_v ? v_cache : k_cache) + (static_cast<int64_t>(kv) * kv_capacity + pos + tok) * kHeadDim;
            gd[a] = ha;
            gd[b] = hb;
          }
        }
      }
    }
  }
  __syncthreads();

  // rows g (lo) and g + 8 (hi) of this warp's tile; a dead row (beyond the last query row) has zero queries and is
  // computed like any other: its result is finite and never written
  const int row0 = 16 * tt;
  const int tile_rows = max(0, min(16, n_rows - row0));
  int row_tok[2];
  uint32_t qa[8][4];      // A fragments of the scaled queries: k step ks covers head dims 16 ks .. 16 ks + 15
#pragma unroll
  for (int hr = 0; hr < 2; ++hr) {
    const int rl = g + 8 * hr;
    const bool live = rl < tile_rows;
    row_tok[hr] = live ? (row0 + rl) / group : -1;
    const __half* qrow = q_h + (live ? row0 + rl : 0) * (kStageRow / 2);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      qa[ks][hr] = live ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 2 * t) : 0u;
      qa[ks][2 + hr] = live ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 8 + 2 * t) : 0u;
    }
  }
  float o[16][4];      // output tile: o[nb] holds head dims 8 nb + 2 t, + 1 of rows g (elements 0, 1) and g + 8 (2, 3)
#pragma unroll
  for (int nb = 0; nb < 16; ++nb) o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};      // of rows g and g + 8, the same in the four lanes of a quad

  // One sub-chunk of 16 positions staged at `stage` (shared-memory address); position wbase + c is visible to row hr
  // when it is at most last[hr].
  auto process = [&](uint32_t stage, int wbase, const int (&last)[2], bool masked) {
    float sc[2][4], sd[2][4];      // even and odd k steps apart: four chains of four dependent instructions instead of two of eight
#pragma unroll
    for (int pb = 0; pb < 2; ++pb) sc[pb][0] = sc[pb][1] = sc[pb][2] = sc[pb][3] = sd[pb][0] = sd[pb][1] = sd[pb][2] = sd[pb][3] = 0.f;
    // S = Q K^T: matrices (positions 0-7 | 8-15) x (dims 16 ks .. + 7 | + 8 .. + 15)
    const uint32_t k_addr = stage + ((lane & 7) + 8 * (lane >> 4)) * kStageRow + 16 * ((lane >> 3) & 1);
#pragma unroll
    for (int ks = 0; ks < 8; ks += 2) {
      uint32_t b0, b1, b2, b3, c0, c1, c2, c3;
      ldmatrix_x4(k_addr + 32 * ks, b0, b1, b2, b3);
      ldmatrix_x4(k_addr + 32 * ks + 32, c0, c1, c2, c3);
      mma_f16(sc[0], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b0, b1);
      mma_f16(sc[1], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b2, b3);
      mma_f16(sd[0], qa[ks + 1][0], qa[ks + 1][1], qa[ks + 1][2], qa[ks + 1][3], c0, c1);
      mma_f16(sd[1], qa[ks + 1][0], qa[ks + 1][1], qa[ks + 1][2], qa[ks + 1][3], c2, c3);
    }
#pragma unroll
    for (int pb = 0; pb < 2; ++pb)
#pragma unroll
      for (int e = 0; e < 4; ++e) sc[pb][e] += sd[pb][e];
    // ---- mask, row maxima, rescaling factors, exponentials
    float mx[2] = {-INFINITY, -INFINITY};
    if (masked) {      // (the same for the whole warp)
#pragma unroll
      for (int pb = 0; pb < 2; ++pb)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int p = wbase + 8 * pb + 2 * t + (e & 1);
          sc[pb][e] = p <= last[e >> 1] ? sc[pb][e] : -INFINITY;
        }
    }
#pragma unroll
    for (int pb = 0; pb < 2; ++pb)
#pragma unroll
      for (int e = 0; e < 4; ++e) mx[e >> 1] = fmaxf(mx[e >> 1], sc[pb][e]);
    float alpha[2], lsum[2], m_new[2];
#pragma unroll
    for (int hr = 0; hr < 2; ++hr) {
      mx[hr] = fmaxf(mx[hr], __shfl_xor_sync(0xffffffffu, mx[hr], 1));
      mx[hr] = fmaxf(mx[hr], __shfl_xor_sync(0xffffffffu, mx[hr], 2));
      // the reference point of a row moves only when a score exceeds it by more than 2^8: until then the exponentials
      // are at most 256 (exact enough in fp16, harmless in the fp32 sums) and the output tile needs no rescaling
      m_new[hr] = mx[hr] > m_run[hr] + 8.0f ? mx[hr] : m_run[hr];
      alpha[hr] = m_run[hr] > -INFINITY ? fast_exp2(m_run[hr] - m_new[hr]) : 1.0f;      // nothing accumulated yet: the tile is zero
      lsum[hr] = 0.f;
    }
    uint32_t pa[4];      // A fragment of P: rows g, g + 8 x positions 2t, 2t+1 (first block of 8) and 8 + 2t, + 1
#pragma unroll
    for (int pb = 0; pb < 2; ++pb) {
      float pv[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int hr = e >> 1;
        pv[e] = m_new[hr] > -INFINITY ? fast_exp2(sc[pb][e] - m_new[hr]) : 0.f;
        lsum[hr] += pv[e];
      }
      pa[2 * pb] = pack_h2(pv[0], pv[1]);        // row g
      pa[2 * pb + 1] = pack_h2(pv[2], pv[3]);    // row g + 8
    }
#pragma unroll
    for (int hr = 0; hr < 2; ++hr) {
      lsum[hr] += __shfl_xor_sync(0xffffffffu, lsum[hr], 1);
      lsum[hr] += __shfl_xor_sync(0xffffffffu, lsum[hr], 2);
      l_run[hr] = l_run[hr] * alpha[hr] + lsum[hr];
      m_run[hr] = m_new[hr];
    }
    if (!__all_sync(0xffffffffu, alpha[0] == 1.0f && alpha[1] == 1.0f)) {      // some row's maximum moved
#pragma unroll
      for (int nb = 0; nb < 16; ++nb) {
        o[nb][0] *= alpha[0]; o[nb][1] *= alpha[0];
        o[nb][2] *= alpha[1]; o[nb][3] *= alpha[1];
      }
    }
    // ---- O += P V: transposed matrices (positions 0-7 | 8-15) x (dims 16 j .. + 7 | + 8 .. + 15)
    const uint32_t v_addr = stage + kStageHalf + ((lane & 7) + 8 * ((lane >> 3) & 1)) * kStageRow + 16 * (lane >> 4);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      uint32_t b0, b1, b2, b3;
      ldmatrix_x4_trans(v_addr + 32 * j, b0, b1, b2, b3);
      mma_f16(o[2 * j], pa[0], pa[1], pa[2], pa[3], b0, b1);
      mma_f16(o[2 * j + 1], pa[0], pa[1], pa[2], pa[3], b2, b3);
    }
  };

  {
    int last[2];
#pragma unroll
    for (int hr = 0; hr < 2; ++hr) last[hr] = pos - 1;      // every row sees every cached position
    for (int i = 0; i < n_sub; ++i) {
      cp_async_wait<S - 2>();      // all but the newest S - 2 groups: sub-chunk i has landed (this thread's pieces)
      team_sync<T>(team);          // ... and the team's; the stage of sub-chunk i - 1 is free
      issue(i + S - 1);
      const int wbase = wbase_of(i);
      if (wbase < pos) process(ring_u32 + (i % S) * kStageBytes, wbase, last, wbase + 16 > pos);
    }
  }
  cp_async_wait<0>();
  if (owns_new && team == 0) {      // the positions of this step, zero rows behind them, in stage 0 of team 0's ring
    team_sync<T>(team);
    for (int idx = tl; idx < 256; idx += 32 * T) {
      const int r = idx >> 4, piece = idx & 15;
      const uint4 zero = make_uint4(0, 0, 0, 0);
      *reinterpret_cast<uint4*>(my_ring + r * kStageRow + 16 * piece) = r < n_tok ? *reinterpret_cast<const uint4*>(new_k + r * kHeadDim + 8 * piece) : zero;
      *reinterpret_cast<uint4*>(my_ring + kStageHalf + r * kStageRow + 16 * piece) =
          r < n_tok ? *reinterpret_cast<const uint4*>(new_v + r * kHeadDim + 8 * piece) : zero;
    }
    team_sync<T>(team);
    int last[2];
#pragma unroll
    for (int hr = 0; hr < 2; ++hr) last[hr] = pos + max(row_tok[hr], 0);      // causal among the new positions
    process(ring_u32, pos, last, true);
  }
  if (t == 0) {      // (back to natural units: the merge and the one-token kernel use e^x)
    s_m[warp][g] = m_run[0] * 0.6931471805599453f;
    s_m[warp][g + 8] = m_run[1] * 0.6931471805599453f;
    s_l[warp][g] = l_run[0];
    s_l[warp][g + 8] = l_run[1];
  }
  __syncthreads();      // every team is done with its ring: the tiles may go over it
#pragma unroll
  for (int nb = 0; nb < 16; ++nb) {
    *reinterpret_cast<float2*>(s_o + (warp * 16 + g) * kRowPad + 8 * nb + 2 * t) = make_float2(o[nb][0], o[nb][1]);
    *reinterpret_cast<float2*>(s_o + (warp * 16 + g + 8) * kRowPad + 8 * nb + 2 * t) = make_float2(o[nb][2], o[nb][3]);
  }
  if (threadIdx.x < W * 16) {      // weight of warp w's tile in the CTA's result for its row
    const int w = threadIdx.x >> 4, r = threadIdx.x & 15;
    float big = -INFINITY;
#pragma unroll
    for (int pp = 0; pp < P; ++pp) big = fmaxf(big, s_m[pp * T + w % T][r]);
    const float mine = s_m[w][r];
    s_f[w][r] = mine > -INFINITY ? expf(mine - big) : 0.f;
    if (w < T) s_big[w][r] = big;
  }
  __syncthreads();
  // thread (row, four head dims) adds up the teams' tiles: one partial result of the CTA per row, numbered by blockIdx.x
  for (int idx = threadIdx.x; idx < n_rows * (kHeadDim / 4); idx += kThr) {
    const int rr = idx / (kHeadDim / 4), d4 = (idx % (kHeadDim / 4)) * 4;
    const int tile = rr >> 4, r = rr & 15;
    float4 accum = make_float4(0.f, 0.f, 0.f, 0.f);
    float l = 0.f;
#pragma unroll
    for (int pp = 0; pp < P; ++pp) {
      const int w = pp * T + tile;
      const float f = s_f[w][r];
      const float4 v = *reinterpret_cast<const float4*>(s_o + (w * 16 + r) * kRowPad + d4);
      l += f * s_l[w][r];
      accum.x += f * v.x; accum.y += f * v.y; accum.z += f * v.z; accum.w += f * v.w;
    }
    const int tok = rr / group, head = kv * group + rr % group;
    const int64_t slot = (static_cast<int64_t>(row_base) + static_cast<int64_t>(tok) * n_q_heads + head) * part_stride + blockIdx.x;
    if (!in_range(static_cast<int>(blockIdx.x) < part_stride, status)) continue;
    *reinterpret_cast<float4*>(o_part + slot * kHeadDim + d4) = accum;
    if (d4 == 0) ml_part[slot] = make_float2(s_big[tile][r], l);
  }
  stamp_end(stamp);
}

// ---- at most eight query rows per KV head (one token per request), merge included ------------------
// A CTA that takes several chunks carries its running (max, sum, output) from chunk to chunk: a warp
// keeps the un-normalised output of its positions in its own tile in shared memory (every lane re-reads
// and re-writes only its own 32 floats, so the chunk loop has no barrier and the warps' loads and
// arithmetic overlap freely); the warps are combined once, at the end, and the CTA leaves ONE partial
// result, numbered by blockIdx.x.  Then the ticket: the CTA that finds all the others' partial results
// written combines them (ascending order, so the bits do not depend on who came last) and writes the
// output rows of its KV head; with a single CTA per (request, KV head) the partial result is normalised
// and written directly.
constexpr int kMaxParts = 320;      // partial results per (request, KV head): at most 2 CTAs per SM / KV heads

__global__ void __launch_bounds__(kThreads, 2)
attn_one_kernel(const acc_t* __restrict__ acc, int64_t mpad, const float* __restrict__ ssq, int n_groups, float inv_width, float eps,
                const float2* __restrict__ rope_tab, int rope_mode, __half* __restrict__ k_cache, __half* __restrict__ v_cache,
                int kv_capacity, int n_q_heads, int n_kv_heads, int pos, int stable_below, int n_chunks, int part_stride,
                float* __restrict__ o_part, float2* __restrict__ ml_part, int* __restrict__ tickets, float* __restrict__ o,
                const AttnSeqs seqs, const Stamp stamp, const L2Ahead ahead, int* status) {
  pdl_trigger();
  int row_base = 0;                 // first output row (request * heads) of this CTA's request
  if (seqs.n > 0) {                 // one request per blockIdx.z: its own cache and position
    const int tq = blockIdx.z;
    k_cache = seqs.k[tq];
    v_cache = seqs.v[tq];
    pos = seqs.pos[tq];
    n_chunks = (pos + kChunk) / kChunk;
    if (static_cast<int>(blockIdx.x) >= n_chunks) return;
    acc += tq * mpad;
    ssq += tq * kMaxStatBlocks;
    rope_tab += tq * (kHeadDim / 2);
    row_base = tq * n_q_heads;
  }
  extern __shared__ __align__(16) float dyn_smem[];
  __shared__ float s_m[kWarps][8], s_l[kWarps][8], s_f[kWarps][8], s_big[8];
  __shared__ float s_inv;
  __shared__ int s_ticket;

  const int group = n_q_heads / n_kv_heads;                            // query rows served by this CTA, at most 8
  float* s_o = dyn_smem;                                               // [kWarps][8][kRowPad]
  float* q_s = s_o + kWarps * 8 * kRowPad;                             // [group][kRowPad] rotated queries of this KV head
  __half* new_k = reinterpret_cast<__half*>(q_s + 8 * kRowPad);        // [128] key of the new position
  __half* new_v = new_k + kHeadDim;

  const int kv = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int n_parts = min(static_cast<int>(gridDim.x), n_chunks);

  uint4 kreg[2][4];      // [position block of 8][32-dim slice]
  uint4 vreg[4][2];      // [k-slot position][64-dim half]
  const __half* kbase = k_cache + static_cast<int64_t>(kv) * kv_capacity * kHeadDim;
  const __half* vbase = v_cache + static_cast<int64_t>(kv) * kv_capacity * kHeadDim;
  auto load_old = [&](int wbase, int limit) {
#pragma unroll
    for (int pb = 0; pb < 2; ++pb) {
      const int p = wbase + 8 * pb + g;
#pragma unroll
      for (int j = 0; j < 4; ++j)
        kreg[pb][j] = p < limit ? __ldcg(reinterpret_cast<const uint4*>(kbase + static_cast<int64_t>(p) * kHeadDim + 32 * j + 8 * t)) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int pi = 0; pi < 4; ++pi) {
      const int p = wbase + 2 * t + (pi & 1) + 8 * (pi >> 1);
#pragma unroll
      for (int hf = 0; hf < 2; ++hf)
        vreg[pi][hf] = p < limit ? __ldcg(reinterpret_cast<const uint4*>(vbase + static_cast<int64_t>(p) * kHeadDim + 64 * hf + 8 * g)) : make_uint4(0, 0, 0, 0);
    }
  };
  // The entry of this step comes from shared memory.
  auto patch_new = [&](int wbase) {
    if (pos < wbase || pos >= wbase + 16) return;
#pragma unroll
    for (int pb = 0; pb < 2; ++pb) {
      if (wbase + 8 * pb + g == pos) {
#pragma unroll
        for (int j = 0; j < 4; ++j) kreg[pb][j] = *reinterpret_cast<const uint4*>(new_k + 32 * j + 8 * t);
      }
    }
#pragma unroll
    for (int pi = 0; pi < 4; ++pi) {
      if (wbase + 2 * t + (pi & 1) + 8 * (pi >> 1) == pos) {
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) vreg[pi][hf] = *reinterpret_cast<const uint4*>(new_v + 64 * hf + 8 * g);
      }
    }
  };

  int chunk = blockIdx.x;
  const int pre_limit = min(pos, stable_below);
  load_old(chunk * kChunk + warp * 16, pre_limit);
  pdl_wait();
  stamp_begin(stamp);
  if (pre_limit < pos && chunk * kChunk + warp * 16 + 16 > pre_limit) load_old(chunk * kChunk + warp * 16, pos);

  // ---- finish the QKV product for this KV head.  Items: one rotation pair of a query row, and for the
  //      CTA that owns the chunk with the new position also one pair of the new key and of the new value.
  const bool owner = (pos / kChunk) % static_cast<int>(gridDim.x) == static_cast<int>(blockIdx.x);
  const int n_q_items = group * (kHeadDim / 2);
  const int n_items = n_q_items + (owner ? 2 * (kHeadDim / 2) : 0);      // at most 640: three per thread
  {
    constexpr int kTrip = 3;
    acc_t ra[kTrip], rb[kTrip];
    float2 cs[kTrip];
#pragma unroll
    for (int u = 0; u < kTrip; ++u) {
      const int idx = threadIdx.x + u * kThreads;
      if (idx < n_items) {
        const int i = idx % (kHeadDim / 2);
        int row0;
        if (idx < n_q_items) row0 = (kv * group + idx / (kHeadDim / 2)) * kHeadDim;
        else row0 = (n_q_heads + (idx - n_q_items < kHeadDim / 2 ? 0 : n_kv_heads) + kv) * kHeadDim;
        const int a = rope_mode == 0 ? i : 2 * i, b = rope_mode == 0 ? i + kHeadDim / 2 : 2 * i + 1;
        ra[u] = __ldcg(acc + row0 + a);
        rb[u] = __ldcg(acc + row0 + b);
        cs[u] = __ldcg(rope_tab + i);
      }
    }
    if (threadIdx.x == 0) {      // the RMSNorm factor, loaded while the accumulators are on their way
      float ss = 0.f;
      for (int gi = 0; gi < n_groups; ++gi) ss += __ldcg(ssq + gi);
      s_inv = 1.0f / sqrtf(ss * inv_width + eps);
    }
    __syncthreads();
    const float inv = s_inv;
#pragma unroll
    for (int u = 0; u < kTrip; ++u) {
      const int idx = threadIdx.x + u * kThreads;
      if (idx < n_items) {
        const int i = idx % (kHeadDim / 2);
        const int a = rope_mode == 0 ? i : 2 * i, b = rope_mode == 0 ? i + kHeadDim / 2 : 2 * i + 1;
        const float x = acc_value(ra[u]) * inv, y = acc_value(rb[u]) * inv;
        if (idx < n_q_items) {
          const int r = idx / (kHeadDim / 2);
          q_s[r * kRowPad + swz(a)] = x * cs[u].x - y * cs[u].y;
          q_s[r * kRowPad + swz(b)] = y * cs[u].x + x * cs[u].y;
        } else {
          const bool is_v = idx - n_q_items >= kHeadDim / 2;
          const __half ha = __float2half_rn(is_v ? x : x * cs[u].x - y * cs[u].y);
          const __half hb = __float2half_rn(is_v ? y : y * cs[u].x + x * cs[u].y);
          __half* sm = is_v ? new_v : new_k;
          sm[a] = ha;
          sm[b] = hb;
          if (in_range(pos >= 0 && pos < kv_capacity, status)) {
            __half* gd = (is_v ? v_cache : k_cache) + (static_cast<int64_t>(kv) * kv_capacity + pos) * kHeadDim;
            gd[a] = ha;
            gd[b] = hb;
          }
        }
      }
    }
  }
  __syncthreads();

  const float scale = 0.08838834764831845f;   // 1 / sqrt(128)
  const bool live = g < group;
  const float* qrow = q_s + (live ? g : 0) * kRowPad;
  float* so = s_o + (warp * 8 + g) * kRowPad;
#pragma unroll
  for (int hf = 0; hf < 2; ++hf)
#pragma unroll
    for (int q = 0; q < 4; ++q) *reinterpret_cast<float4*>(so + swz(64 * hf + 16 * t + 4 * q)) = make_float4(0.f, 0.f, 0.f, 0.f);
  float m_run = -INFINITY, l_run = 0.f;      // of row g, the same in the four lanes of a quad
  for (bool first = true; chunk < n_chunks; chunk += gridDim.x, first = false) {
    const int wbase = chunk * kChunk + warp * 16;
    if (!first) load_old(wbase, pos);
    patch_new(wbase);
    float sc[2][4];
#pragma unroll
    for (int pb = 0; pb < 2; ++pb) sc[pb][0] = sc[pb][1] = sc[pb][2] = sc[pb][3] = 0.f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
      if (live) {
        a = *reinterpret_cast<const float4*>(qrow + swz(32 * j + 8 * t));
        b = *reinterpret_cast<const float4*>(qrow + swz(32 * j + 8 * t) + 4);
      }
      const uint32_t qa0 = pack_h2(a.x * scale, a.y * scale), qa2 = pack_h2(a.z * scale, a.w * scale);
      const uint32_t qb0 = pack_h2(b.x * scale, b.y * scale), qb2 = pack_h2(b.z * scale, b.w * scale);
#pragma unroll
      for (int pb = 0; pb < 2; ++pb) {      // rows 8..15 of the tile do not exist: zero operands
        mma_f16(sc[pb], qa0, 0u, qa2, 0u, kreg[pb][j].x, kreg[pb][j].y);
        mma_f16(sc[pb], qb0, 0u, qb2, 0u, kreg[pb][j].z, kreg[pb][j].w);
      }
    }
    float mx = -INFINITY;
#pragma unroll
    for (int pb = 0; pb < 2; ++pb)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int p = wbase + 8 * pb + 2 * t + e;
        const bool ok = live && p <= pos;
        sc[pb][e] = ok ? sc[pb][e] : -INFINITY;
        mx = fmaxf(mx, sc[pb][e]);
      }
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    const float m_new = fmaxf(m_run, mx);
    const float alpha = m_run > -INFINITY ? expf(m_run - m_new) : 1.0f;      // nothing accumulated yet: the tile is zero
    float lsum = 0.f;
    uint32_t pa[2];
#pragma unroll
    for (int pb = 0; pb < 2; ++pb) {
      const float p0 = m_new > -INFINITY ? expf(sc[pb][0] - m_new) : 0.f;
      const float p1 = m_new > -INFINITY ? expf(sc[pb][1] - m_new) : 0.f;
      lsum += p0 + p1;
      pa[pb] = pack_h2(p0, p1);
    }
    lsum += __shfl_xor_sync(0xffffffffu, lsum, 1);
    lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
    l_run = l_run * alpha + lsum;
    m_run = m_new;
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
#pragma unroll
      for (int bh = 0; bh < 2; ++bh) {
        float oc[4][4];
#pragma unroll
        for (int bb = 0; bb < 4; ++bb) {
          const int b = 4 * bh + bb, j = b >> 1;
          const uint32_t sel = (b & 1) ? 0x7632u : 0x5410u;
          const uint32_t* v0 = reinterpret_cast<const uint32_t*>(&vreg[0][hf]);
          const uint32_t* v1 = reinterpret_cast<const uint32_t*>(&vreg[1][hf]);
          const uint32_t* v2 = reinterpret_cast<const uint32_t*>(&vreg[2][hf]);
          const uint32_t* v3 = reinterpret_cast<const uint32_t*>(&vreg[3][hf]);
          const uint32_t b0 = __byte_perm(v0[j], v1[j], sel);
          const uint32_t b1 = __byte_perm(v2[j], v3[j], sel);
          oc[bb][0] = oc[bb][1] = oc[bb][2] = oc[bb][3] = 0.f;
          mma_f16(oc[bb], pa[0], 0u, pa[1], 0u, b0, b1);
        }
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          float4* dst = reinterpret_cast<float4*>(so + swz(64 * hf + 16 * t + 8 * e + 4 * bh));
          const float4 old = *dst;
          *dst = make_float4(fmaf(old.x, alpha, oc[0][e]), fmaf(old.y, alpha, oc[1][e]), fmaf(old.z, alpha, oc[2][e]), fmaf(old.w, alpha, oc[3][e]));
        }
      }
    }
  }
  // this CTA's cache reads are over: from here on HBM has nothing to do for it
  if (threadIdx.x == 0) l2_ahead(ahead, blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z), gridDim.x * gridDim.y * gridDim.z);
  if (t == 0) {
    s_m[warp][g] = m_run;
    s_l[warp][g] = l_run;
  }
  __syncthreads();
  if (threadIdx.x < kWarps * 8) {
    const int w = threadIdx.x >> 3, r = threadIdx.x & 7;
    float big = -INFINITY;
#pragma unroll
    for (int ww = 0; ww < kWarps; ++ww) big = fmaxf(big, s_m[ww][r]);
    const float mine = s_m[w][r];
    s_f[w][r] = mine > -INFINITY ? expf(mine - big) : 0.f;
    if (w == 0) s_big[r] = big;
  }
  __syncthreads();
  // thread (row r, four head dims) adds up the eight warps' tiles
  const int r = threadIdx.x >> 5, d4 = lane * 4;
  const int64_t out_row = static_cast<int64_t>(row_base) + kv * group + r;
  float4 accum = make_float4(0.f, 0.f, 0.f, 0.f);
  float l = 0.f;
  if (r < group) {
    const int col = swz(d4);
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      const float f = s_f[w][r];
      const float4 v = *reinterpret_cast<const float4*>(s_o + (w * 8 + r) * kRowPad + col);
      l += f * s_l[w][r];
      accum.x += f * v.x; accum.y += f * v.y; accum.z += f * v.z; accum.w += f * v.w;
    }
  }
  if (n_parts == 1 && tickets != nullptr) {      // nothing to merge
    if (r < group) *reinterpret_cast<float4*>(o + out_row * kHeadDim + d4) = make_float4(accum.x / l, accum.y / l, accum.z / l, accum.w / l);
    stamp_end(stamp);
    return;
  }
  if (r < group && in_range(static_cast<int>(blockIdx.x) < part_stride, status)) {
    const int64_t slot = out_row * part_stride + blockIdx.x;
    *reinterpret_cast<float4*>(o_part + slot * kHeadDim + d4) = accum;
    if (lane == 0) ml_part[slot] = make_float2(s_big[r], l);
  }
  if (tickets == nullptr) {      // the merge is a kernel of its own
    stamp_end(stamp);
    return;
  }
  // ---- the ticket: partial results first, visible to the whole GPU, then the count
  __threadfence();
  __syncthreads();
  int* ticket = tickets + (seqs.n > 0 ? static_cast<int>(blockIdx.z) : 0) * n_kv_heads + kv;
  if (threadIdx.x == 0) {
    const int drawn = atomicAdd(ticket, 1);
    if (drawn == n_parts - 1) *ticket = 0;      // all have arrived: ready for the next launch
    s_ticket = drawn;
  }
  __syncthreads();
  if (s_ticket != n_parts - 1) {
    stamp_end(stamp);
    return;
  }
  __threadfence();
  // ---- merge: warp r owns output row r.  Weights e^(m_c - M) of the parts go to shared memory (the tiles
  //      are no longer needed), then every lane adds up its four head dims over the parts in ascending order.
  float* s_w = s_o + r * kMaxParts;      // kMaxParts floats per row; 8 rows fit in the first tiles
  if (r < group) {
    const float2* ml = ml_part + out_row * part_stride;
    float big = -INFINITY;
    for (int c = lane; c < n_parts; c += 32) big = fmaxf(big, __ldcg(ml + c).x);
#pragma unroll
    for (int of = 16; of > 0; of >>= 1) big = fmaxf(big, __shfl_xor_sync(0xffffffffu, big, of));
    float den = 0.f;
    for (int c = lane; c < n_parts; c += 32) {
      const float2 v = __ldcg(ml + c);
      const float w = v.x > -INFINITY ? expf(v.x - big) : 0.f;
      s_w[c] = w;
      den += w * v.y;
    }
#pragma unroll
    for (int of = 16; of > 0; of >>= 1) den += __shfl_xor_sync(0xffffffffu, den, of);
    __syncwarp();
    const float* op = o_part + out_row * part_stride * kHeadDim + d4;
    float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
    int c = 0;
    for (; c + 8 <= n_parts; c += 8) {      // eight loads in flight
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = __ldcg(reinterpret_cast<const float4*>(op + static_cast<int64_t>(c + u) * kHeadDim));
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const float w = s_w[c + u];
        sum.x += w * v[u].x; sum.y += w * v[u].y; sum.z += w * v[u].z; sum.w += w * v[u].w;
      }
    }
    for (; c < n_parts; ++c) {
      const float4 v = __ldcg(reinterpret_cast<const float4*>(op + static_cast<int64_t>(c) * kHeadDim));
      const float w = s_w[c];
      sum.x += w * v.x; sum.y += w * v.y; sum.z += w * v.z; sum.w += w * v.w;
    }
    *reinterpret_cast<float4*>(o + out_row * kHeadDim + d4) = make_float4(sum.x / den, sum.y / den, sum.z / den, sum.w / den);
  }
  stamp_end(stamp);
}

// One block of 128 threads per (token, head): merge the chunks in ascending order.  Thread d owns
// head dim d.  The partial outputs of the first kMergePre chunks are requested before anything
// else, together with the (max, sum) pairs, so that the kernel costs one round trip to L2.
__global__ void __launch_bounds__(kHeadDim)
attn_merge_kernel(const float* __restrict__ o_part, const float2* __restrict__ ml_part, int n_chunks, int chunk_stride, int n_q_heads,
                  float* __restrict__ o, const AttnSeqs seqs, const Stamp stamp) {
  pdl_trigger();
  pdl_wait();
  if (seqs.n > 0) n_chunks = min(n_chunks, (seqs.pos[blockIdx.x / n_q_heads] + kChunk) / kChunk);      // the row's own request
  extern __shared__ float s_w[];         // [n_chunks] weights e^(m_c - M), then [n_chunks] weights times l_c
  float* s_wl = s_w + n_chunks;
  __shared__ float s_red[4];
  const int row = blockIdx.x;            // tok * H + head
  const int d = threadIdx.x;
  const float2* ml = ml_part + static_cast<int64_t>(row) * chunk_stride;
  const float* op = o_part + static_cast<int64_t>(row) * chunk_stride * kHeadDim + d;
  float pre[kMergePre];
#pragma unroll
  for (int c = 0; c < kMergePre; ++c)
    if (c < n_chunks) pre[c] = __ldcg(op + static_cast<int64_t>(c) * kHeadDim);
  const float2 ml0 = d < n_chunks ? __ldcg(ml + d) : make_float2(-INFINITY, 0.f);      // this thread's first chunk
  float big = ml0.x;
  for (int c = d + kHeadDim; c < n_chunks; c += kHeadDim) big = fmaxf(big, __ldcg(ml + c).x);
#pragma unroll
  for (int of = 16; of > 0; of >>= 1) big = fmaxf(big, __shfl_xor_sync(0xffffffffu, big, of));
  if ((d & 31) == 0) s_red[d >> 5] = big;
  __syncthreads();
  big = fmaxf(fmaxf(s_red[0], s_red[1]), fmaxf(s_red[2], s_red[3]));
  for (int c = d; c < n_chunks; c += kHeadDim) {
    const float2 v = c == d ? ml0 : __ldcg(ml + c);
    const float w = v.x > -INFINITY ? expf(v.x - big) : 0.f;
    s_w[c] = w;
    s_wl[c] = w * v.y;
  }
  __syncthreads();
  // every thread forms the same denominator in chunk order
  float denom = 0.f;
#pragma unroll 8
  for (int c = 0; c < n_chunks; ++c) denom += s_wl[c];
  float accum = 0.f;
#pragma unroll
  for (int c = 0; c < kMergePre; ++c)
    if (c < n_chunks) accum += s_w[c] * pre[c];
#pragma unroll 8
  for (int c = kMergePre; c < n_chunks; ++c) accum += s_w[c] * __ldcg(op + static_cast<int64_t>(c) * kHeadDim);
  o[static_cast<int64_t>(row) * kHeadDim + d] = accum / denom;
  stamp_end(stamp);
}

constexpr size_t kOneSmemBytes = static_cast<size_t>(kWarps * 8 + 8) * kRowPad * sizeof(float) + 2 * kHeadDim * sizeof(__half);
static_assert(8 * kMaxParts <= kWarps * 8 * kRowPad, "the merge weights reuse the tiles");

}  // namespace

int attention_chunk_len() { return kChunk; }

// Where the partial results of a one-token step are merged.  Default: a second, small kernel (one block per
// output row: the reads of all rows proceed in parallel).  PRIMA_ATTN_MERGE=fused (read once per process): inside
// the attention kernel, by the last CTA of each KV head to finish; one launch less, but that CTA reads its eight
// rows' partial results alone, which measured 1.7 us per layer slower at 4096 positions on the 70B shape.
bool attention_merge_is_fused() {
  static const bool fused = [] {
    const char* v = getenv("PRIMA_ATTN_MERGE");
    return v && v[0] == 'f';
  }();
  return fused;
}

static int configure_kernels() {
  static bool configured[kMaxDevices] = {};
  int dev = -1;
  if (first_launch_on_device(configured, &dev)) {
    cudaError_t e0 = cudaSuccess;
    auto configure_tile = [&](auto kernel, size_t bytes) {
      if (e0 == cudaSuccess) e0 = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes));
      if (e0 == cudaSuccess) e0 = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    };
    configure_tile(attn_tile_kernel<1>, TileShape<1>::kSmem);
    configure_tile(attn_tile_kernel<2>, TileShape<2>::kSmem);
    configure_tile(attn_tile_kernel<3>, TileShape<3>::kSmem);
    configure_tile(attn_tile_kernel<4>, TileShape<4>::kSmem);
    if (e0 == cudaSuccess) e0 = cudaFuncSetAttribute(attn_one_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kOneSmemBytes));
    if (e0 == cudaSuccess) e0 = cudaFuncSetAttribute(attn_one_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e0 != cudaSuccess) return cuda_rc(e0);
    if (dev >= 0) configured[dev] = true;
  }
  return 0;
}

int launch_attention(const acc_t* acc_qkv, int64_t mpad, const SumSq& ssq, const float2* rope_tab, int rope_mode, __half* k_cache,
                     __half* v_cache, int kv_capacity, int n_q_heads, int n_kv_heads, int pos, int stable_below, int n_tok,
                     const AttnScratch& scr, float* o, int sm_count, cudaStream_t st) {
  const int n_ctx = pos + n_tok;
  const int n_chunks = (n_ctx + kChunk - 1) / kChunk;
  if (n_chunks > scr.max_chunks) return cuda_rc(cudaErrorInvalidValue);
  const int group = n_q_heads / n_kv_heads;
  const int n_rows = n_tok * group;
  const int rc = configure_kernels();
  if (rc != 0) return rc;
  const float inv_width = ssq.width > 0 ? 1.0f / static_cast<float>(ssq.width) : 0.f;
  // Two CTAs fit on an SM: with more chunks than that, a CTA takes several (gridDim.x apart).
  const int per_head = std::min(kMaxParts, std::max(1, 2 * sm_count / n_kv_heads));
  dim3 grid(std::min(n_chunks, per_head), n_kv_heads);
  const AttnSeqs none{};
  // one token: up to about ten thousand positions the kernel that keeps its positions in registers (two CTAs per SM,
  // everything requested before the dependency wait) is faster; beyond, the streaming kernel (measured: 10.9 against
  // 14.3 us per layer at 4096 positions, 25.8 against 22.3 at 16384, 40.2 against 32.4 at 32768)
  constexpr int kLongContextChunks = 80;
  if (n_tok == 1 && n_chunks < kLongContextChunks) {
    int* tickets = attention_merge_is_fused() ? scr.tickets : nullptr;
    cudaError_t e = launch_pdl(attn_one_kernel, grid, dim3(kThreads), kOneSmemBytes, st, acc_qkv, mpad, static_cast<const float*>(ssq.data),
                               ssq.n_groups, inv_width, ssq.eps, rope_tab, rope_mode, k_cache, v_cache, kv_capacity, n_q_heads, n_kv_heads,
                               pos, stable_below, n_chunks, scr.max_chunks, scr.o_part, scr.ml_part, tickets, o, none, scr.stamp, scr.ahead, scr.status);
    if (e != cudaSuccess) return cuda_rc(e);
    if (tickets) return 1;
    e = launch_pdl(attn_merge_kernel, dim3(n_q_heads), dim3(kHeadDim), static_cast<size_t>(2 * grid.x) * sizeof(float), st, scr.o_part,
                   scr.ml_part, static_cast<int>(grid.x), scr.max_chunks, n_q_heads, o, none, scr.stamp);
    return e == cudaSuccess ? 2 : cuda_rc(e);
  }
  // several tokens: one CTA per (slot of chunks, KV head), one CTA per SM, all tiles of 16 query rows in the CTA
  const int n_tiles = (n_rows + 15) / 16;
  if (n_tiles > 4) return cuda_rc(cudaErrorInvalidValue);
  const int slots = std::min(kMaxParts, std::max(1, sm_count / n_kv_heads));
  dim3 tgrid(std::min(n_chunks, slots), n_kv_heads);
  auto launch_tile = [&](auto kernel, int warps, size_t bytes) {
    return launch_pdl(kernel, tgrid, dim3(warps * 32), bytes, st, acc_qkv, mpad, static_cast<const float*>(ssq.data), ssq.n_groups, inv_width,
                      ssq.eps, rope_tab, rope_mode, k_cache, v_cache, kv_capacity, n_q_heads, n_kv_heads, pos, stable_below, n_tok,
                      scr.max_chunks, scr.o_part, scr.ml_part, none, scr.stamp, scr.ahead, scr.status);
  };
  cudaError_t e = n_tiles == 1   ? launch_tile(attn_tile_kernel<1>, TileShape<1>::kWarpsOf, TileShape<1>::kSmem)
                  : n_tiles == 2 ? launch_tile(attn_tile_kernel<2>, TileShape<2>::kWarpsOf, TileShape<2>::kSmem)
                  : n_tiles == 3 ? launch_tile(attn_tile_kernel<3>, TileShape<3>::kWarpsOf, TileShape<3>::kSmem)
                                 : launch_tile(attn_tile_kernel<4>, TileShape<4>::kWarpsOf, TileShape<4>::kSmem);
  if (e != cudaSuccess) return cuda_rc(e);
  e = launch_pdl(attn_merge_kernel, dim3(n_tok * n_q_heads), dim3(kHeadDim), static_cast<size_t>(2 * tgrid.x) * sizeof(float), st,
                 scr.o_part, scr.ml_part, static_cast<int>(tgrid.x), scr.max_chunks, n_q_heads, o, none, scr.stamp);
  if (e != cudaSuccess) return cuda_rc(e);
  return 2;
}

int launch_attention_seqs(const acc_t* acc_qkv, int64_t mpad, const SumSq& ssq, const float2* rope_tab, int rope_mode, const AttnSeqs& seqs,
                          int stable_below, int kv_capacity, int n_q_heads, int n_kv_heads, const AttnScratch& scr, float* o, int sm_count,
                          cudaStream_t st) {
  if (seqs.n < 1 || seqs.n > kMaxTok) return cuda_rc(cudaErrorInvalidValue);
  int max_chunks = 1;
  for (int t = 0; t < seqs.n; ++t) max_chunks = std::max(max_chunks, (seqs.pos[t] + kChunk) / kChunk);
  if (max_chunks > scr.max_chunks) return cuda_rc(cudaErrorInvalidValue);
  const int rc = configure_kernels();
  if (rc != 0) return rc;
  if (seqs.n >= 2) {
    // several requests: the streaming kernel with one tile of query rows (the heads of the group), one CTA per SM in
    // all; a CTA beyond its request's chunks leaves an empty partial result, which the merge gives no weight
    const int slots = std::min(kMaxParts, std::max(1, sm_count / (n_kv_heads * seqs.n)));
    dim3 tgrid(std::min(max_chunks, slots), n_kv_heads, seqs.n);
    cudaError_t e = launch_pdl(attn_tile_kernel<1>, tgrid, dim3(TileShape<1>::kWarpsOf * 32), TileShape<1>::kSmem, st, acc_qkv, mpad,
                               static_cast<const float*>(ssq.data), ssq.n_groups, ssq.width > 0 ? 1.0f / static_cast<float>(ssq.width) : 0.f, ssq.eps,
                               rope_tab, rope_mode, static_cast<__half*>(nullptr), static_cast<__half*>(nullptr), kv_capacity, n_q_heads, n_kv_heads,
                               0, stable_below, 1, scr.max_chunks, scr.o_part, scr.ml_part, seqs, scr.stamp, scr.ahead, scr.status);
    if (e != cudaSuccess) return cuda_rc(e);
    const AttnSeqs none{};
    e = launch_pdl(attn_merge_kernel, dim3(seqs.n * n_q_heads), dim3(kHeadDim), static_cast<size_t>(2 * tgrid.x) * sizeof(float), st, scr.o_part,
                   scr.ml_part, static_cast<int>(tgrid.x), scr.max_chunks, n_q_heads, o, none, scr.stamp);
    return e == cudaSuccess ? 2 : cuda_rc(e);
  }
  // a single request: the one-token kernel, about one wave of CTAs (two per SM)
  const int per_head = std::min(kMaxParts, std::max(1, 2 * sm_count / (n_kv_heads * seqs.n)));
  dim3 grid(std::min(max_chunks, per_head), n_kv_heads, seqs.n);      // CTAs beyond a request's own chunks leave at once
  int* tickets = attention_merge_is_fused() ? scr.tickets : nullptr;
  cudaError_t e = launch_pdl(attn_one_kernel, grid, dim3(kThreads), kOneSmemBytes, st, acc_qkv, mpad, static_cast<const float*>(ssq.data),
                             ssq.n_groups, ssq.width > 0 ? 1.0f / static_cast<float>(ssq.width) : 0.f, ssq.eps, rope_tab, rope_mode,
                             static_cast<__half*>(nullptr), static_cast<__half*>(nullptr), kv_capacity, n_q_heads, n_kv_heads, 0, stable_below,
                             max_chunks, scr.max_chunks, scr.o_part, scr.ml_part, tickets, o, seqs, scr.stamp, scr.ahead, scr.status);
  if (e != cudaSuccess) return cuda_rc(e);
  if (tickets) return 1;
  e = launch_pdl(attn_merge_kernel, dim3(seqs.n * n_q_heads), dim3(kHeadDim), static_cast<size_t>(2 * grid.x) * sizeof(float), st, scr.o_part,
                 scr.ml_part, static_cast<int>(grid.x), scr.max_chunks, n_q_heads, o, seqs, scr.stamp);
  return e == cudaSuccess ? 2 : cuda_rc(e);
}

}  // namespace prima
