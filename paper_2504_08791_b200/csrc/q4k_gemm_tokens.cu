// Q4_K product for five to sixteen tokens per step: the tokens are the columns of the tensor-core product.
#include "gemv_device.cuh"

namespace prima {
namespace {
using namespace gemv_detail;

// ---- several tokens per step: the tokens are the columns of the tensor-core product ----------------
//
// With five or more tokens (verification of draft tokens, or one token of each of several requests) the
// product is a small dense contraction and the int8 instruction m16n8k32 is used as one: A = the 32
// weights of ONE sub-block for 16 rows (two row tiles), B = the activations of that sub-block for 8
// tokens, once with their high and once with their low bytes.  The weights are read once for all
// tokens; nine to sixteen tokens are two column blocks of eight, worked on by two warps that share every
// batch of weights in shared memory (NB = 2).
// Same tiled matrix, same ring of bulk copies and exact integer sums as the one-token kernel; what differs:
//  * A unit stores (row g, sub-block j) as one 16-byte piece, but the instruction wants from lane
//    (g, t) bytes 4t..4t+3 of every sub-block of row g: exactly what a matrix load (ldmatrix) of the
//    eight rows' pieces delivers.  Word t of a sub-block holds weights 8t..8t+7, whose even nibbles
//    become k slots 4t..4t+3 and odd nibbles k slots 16+4t..+3.
//  * Lane (g, t) supplies column g of B, i.e. token g of the block: for each sub-block the four words
//    (high/low bytes x even/odd weights) of its quarter t.  The quantised activations of a column go
//    through shared memory once to reach the lanes in that arrangement.
//  * The activations of a token are 16-bit integers with ONE step for the 256 values of the column,
//    s = max|x| / 32639, so that the sums over the sub-blocks can stay in the integers:
//        partial[row][tok] = s[tok] * (d * sum_j sc_j I_j  -  dmin * sum_j m_j X_j),
//    I_j = 256 * high + low from the two instructions (the high and low parts are summed apart),
//    X_j = the sum of the sub-block's 32 integers.
//  * The second sum is itself a contraction over the eight sub-blocks, shared by all rows of a tile:
//    A = the mins m_j of 16 rows as bytes (k slots 0..7), B = X_j of 8 tokens, cut into three signed
//    bytes X = b0 + 256 b1 + 65536 b2 (|X| < 2^20), one instruction per byte.
//  * The instruction leaves lane (g, t) the complete sums of rows g and g+8 for tokens 2t and 2t+1:
//    no reduction over the quad.
// NB = 1: two CTAs of SG warps per SM, ring of 2 batches per warp, warp w works on column group * SG + w as
// in the one-token kernel.  NB = 2: one CTA of 2 SG warps per SM; warps w and SG + w form a pair on column
// group * SG + w with ONE ring of 4 batches: the first warp of the pair requests the copies, both wait on
// the same mbarriers, each multiplies the batch with its own eight tokens, and a named barrier of the pair
// (64 threads) hands a slot back before it is requested again.  The ring slots that follow the last
// requested one double as the buffers (one per warp of the pair) through which a warp's quantised
// activations are rearranged, before their first copies are requested.
template <int NB>
struct TokCfg {
  static constexpr int kRingTok = NB == 1 ? 2 : 4;
  static constexpr int kCols = 8 * NB;           // token columns
  static constexpr int kCtasPerSm = NB == 1 ? 2 : 1;
};

// activation buffer of one column block inside a ring slot
constexpr int kXsQBytes = 8 * 32 * 16;            // [token][lane] 16 bytes: hi even, hi odd, lo even, lo odd of a quarter sub-block
constexpr int kXsXBytes = 8 * 3 * 8;              // [token][byte of X][sub-block]
constexpr int kXsStepBytes = 8 * 4;               // [token] step
static_assert(kXsQBytes + kXsXBytes + kXsStepBytes <= kBatchBytes, "the activation buffer of a column block must fit a ring slot");

// Four 8x8 matrices of 16-bit elements from shared memory: lane l gives the address of row l % 8 of
// matrix l / 8 (16 bytes each); lane (g, t) receives bytes 4t..4t+3 of row g of each matrix.
__device__ __forceinline__ void ldmatrix_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}

// 256 * high + low as a float: the two 32-bit sums are each below 2^25 in magnitude, their combination
// needs up to 33 bits, so it is formed in fp32 (relative error 2^-24, far below the other roundings).
__device__ __forceinline__ float scaled_sum(int high, int low) { return fmaf(static_cast<float>(high), 256.0f, static_cast<float>(low)); }

// One header row of a unit: d, dmin and the four 24-bit field groups
// f[t] = sc_t | sc_{t+4} << 6 | m_t << 12 | m_{t+4} << 18.
struct RowScales {
  float d, dmin;
  uint32_t f[4];
  __device__ __forceinline__ int sc(int j) const { return (f[j & 3] >> (j < 4 ? 0 : 6)) & 63u; }
};
__device__ __forceinline__ RowScales decode_row(const uint4& h) {
  RowScales r;
  const float2 df = __half22float2(*reinterpret_cast<const __half2*>(&h.x));
  r.d = df.x;
  r.dmin = df.y;
  r.f[0] = h.y;                 // the top byte of words 1..3 carries a piece of f[3]; sc() and min_bytes() mask it away
  r.f[1] = h.z;
  r.f[2] = h.w;
  r.f[3] = (h.y >> 24) | ((h.z >> 24) << 8) | ((h.w >> 24) << 16);
  return r;
}
// The mins m_{4t} .. m_{4t+3} of the row as four bytes (lanes t = 0, 1; zero for t = 2, 3): the lane's part
// of the A operand of the second sum.  m_j sits at bit 12 (j < 4) or 18 (j >= 4) of f[j & 3].
__device__ __forceinline__ uint32_t min_bytes(const RowScales& r, uint32_t shift, uint32_t mask) {
  const uint32_t lo = __byte_perm(r.f[0] >> shift, r.f[1] >> shift, 0x0040u);      // bytes: f0, f1
  const uint32_t hi = __byte_perm(r.f[2] >> shift, r.f[3] >> shift, 0x0040u);      // bytes: f2, f3
  return __byte_perm(lo, hi, 0x5410u) & mask;
}

// Quantise the warp's 256 staged activations of one token with one step for all of them; lane l
// holds quarter l % 4 of sub-block l / 4 as in quantise_lane; `sum` is the sub-block's sum of x_q.
__device__ __forceinline__ LaneQuant quantise_lane_column(const float (&v)[8]) {
  float amax = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(v[i]));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  const bool ok = amax > 0.f && amax < 3.0e38f;
  const float inv_step = ok ? 32639.0f / amax : 0.f;
  int sum = 0;
  uint32_t hi[2] = {0, 0}, lo[2] = {0, 0};
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    int xq = __float2int_rn(v[i] * inv_step);
    xq = max(-32639, min(32639, xq));
    sum += xq;
    const int l = ((xq + 128) & 255) - 128;      // signed low byte
    const int h = (xq - l) >> 8;                 // signed high byte, |h| <= 127
    hi[i & 1] |= (static_cast<uint32_t>(h) & 0xffu) << (8 * (i >> 1));
    lo[i & 1] |= (static_cast<uint32_t>(l) & 0xffu) << (8 * (i >> 1));
  }
  sum += __shfl_xor_sync(0xffffffffu, sum, 1);
  sum += __shfl_xor_sync(0xffffffffu, sum, 2);
  LaneQuant r;
  r.q = make_uint4(hi[0], hi[1], lo[0], lo[1]);
  r.step = ok ? amax / 32639.0f : 0.f;
  r.sum = sum;
  return r;
}

template <int NB>
size_t gemv_tokens_smem_bytes(int sg) {
  using C = TokCfg<NB>;
  return static_cast<size_t>(sg) * C::kRingTok * kBatchBytes + static_cast<size_t>((sg * C::kRingTok + 15) & ~15) * 8 +   // ring, mbarriers
         static_cast<size_t>(2) * kMaxWarps * kBatch * kRowsPerTile * C::kCols * sizeof(float) +                            // reduction buffer
         static_cast<size_t>(kMaxWarps) * C::kCols * sizeof(float);                                                          // sums of squares
}

// Barrier of the two warps of a pair (NB = 2); barrier 0 is the CTA's.
__device__ __forceinline__ void pair_sync(int id) { asm volatile("bar.sync %0, 64;" ::"r"(id) : "memory"); }

template <int NB>
__global__ void __launch_bounds__(NB * kMaxWarps * 32, TokCfg<NB>::kCtasPerSm) gemv_tokens_kernel(const GemvParams P) {
  using C = TokCfg<NB>;
  constexpr int kRingTok = C::kRingTok;
  constexpr int kCols = C::kCols;
  pdl_trigger();
  extern __shared__ __align__(128) uint8_t smem[];
  const uint8_t* __restrict__ w = P.w;
  const int n_rt = P.n_rt, n_sb = P.n_sb, sg = P.sg, n_tok = P.n_tok_total;
  const int n_warps = sg;                 // column warps; the CTA has NB * sg warps
  acc_t* __restrict__ acc_out = P.acc;
  const int64_t mpad = P.mpad;
  int* __restrict__ status = P.status;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + static_cast<size_t>(n_warps) * kRingTok * kBatchBytes);
  float* red = reinterpret_cast<float*>(bars + ((n_warps * kRingTok + 15) & ~15));       // [2][warps][kBatch][8 rows][kCols tokens]
  float* s_red = red + 2 * kMaxWarps * kBatch * kRowsPerTile * kCols;                    // [warps][kCols tokens]

  const int lane = threadIdx.x & 31;
  const int tb = NB == 1 ? 0 : static_cast<int>(threadIdx.x >> 5) / sg;       // token block of this warp: tokens 8 tb .. 8 tb + 7
  const int warp = static_cast<int>(threadIdx.x >> 5) - tb * sg;               // column of this warp inside the group
  const int g = lane >> 2, t = lane & 3;

  // fixed, even shares as in the one-token kernel
  const int n_groups = n_sb / sg;
  const int n_pos = n_groups * n_rt;
  int p0 = 0, p1 = 0;
  const int per_group = gridDim.x / n_groups;
  if (per_group >= 1) {
    const int grp = blockIdx.x % n_groups, i = blockIdx.x / n_groups;
    if (i < per_group) {
      p0 = grp * n_rt + static_cast<int>(static_cast<int64_t>(n_rt) * i / per_group);
      p1 = grp * n_rt + static_cast<int>(static_cast<int64_t>(n_rt) * (i + 1) / per_group);
    }
  } else {
    p0 = static_cast<int>(static_cast<int64_t>(n_pos) * blockIdx.x / gridDim.x);
    p1 = static_cast<int>(static_cast<int64_t>(n_pos) * (blockIdx.x + 1) / gridDim.x);
  }
  auto clear_arrays = [&]() {
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < P.zero0_n; i += stride) P.zero0[i] = 0;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < P.zero1_n; i += stride) P.zero1[i] = 0;
  };
  if (p0 >= p1) {
    pdl_wait();
    stamp_begin(P.stamp);
    clear_arrays();
    stamp_end(P.stamp);
    return;
  }

  uint8_t* my_ring = smem + static_cast<size_t>(warp) * kRingTok * kBatchBytes;
  const uint32_t ring_u32 = smem_addr(my_ring);
  const uint32_t bar_u32 = smem_addr(bars + warp * kRingTok);
  if (lane == 0 && tb == 0) {
#pragma unroll
    for (int i = 0; i < kRingTok; ++i) mbar_init(bar_u32 + 8 * i, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncwarp();
  if (NB == 2) pair_sync(1 + warp);      // the partner sees initialised mbarriers

  Walk pf, cur;
  cur.init(p0, p1, n_rt);
  int n_in_flight = 0;
  int rslot = 0;
  auto request = [&]() {
    const int nb = pf.batch();
    if (lane == 0 && tb == 0) {
      const uint8_t* src = w + (static_cast<int64_t>(pf.grp * sg + warp) * n_rt + pf.rt) * kUnitBytes;
      // (range-checked build: the batch lies inside the matrix; a request that does not is left out and its wait runs out)
      if (in_range(src >= w && src + nb * kUnitBytes <= w + static_cast<int64_t>(n_sb) * n_rt * kUnitBytes && nb >= 1 && nb <= kBatch, status)) {
        mbar_expect_tx(bar_u32 + 8 * rslot, nb * kUnitBytes);
        bulk_load(ring_u32 + rslot * kBatchBytes, src, nb * kUnitBytes, bar_u32 + 8 * rslot, stream_once_policy());
      }
    }
    pf.next(nb);
    ++n_in_flight;
    if (++rslot == kRingTok) rslot = 0;
  };

  // B operands of the lane: token g of the warp's block, sub-block j: high or low bytes of the even or odd weights of
  // quarter t; xm: the three byte planes of X_{4t} .. X_{4t+3} of that token (lanes t = 0, 1; zero otherwise).
  // step: of the lane's output tokens 2t and 2t+1 of the block.
  uint32_t x_he[8], x_ho[8], x_le[8], x_lo[8];
  uint32_t xm[3];
  float step[2];
  int parity = 0;
  bool alive = true;
  bool waited = false;
  bool first_wait = true;
  RingDrain drain;
  int slot = 0;
  uint32_t phase = 0;
  constexpr uint32_t E = 0x0f0f0f0fu;
  const uint32_t m_shift = 12u + 6u * (t & 1), m_mask = t < 2 ? 0x3f3f3f3fu : 0u;
  // ldmatrix: lane l addresses row l % 8 of matrix l / 8 = the piece of (row l % 8, sub-block l / 8 of the half)
  const uint32_t piece = static_cast<uint32_t>(kUnitHdrBytes + unit_piece_slot(lane & 7, lane >> 3) * 16);

  while (!cur.done()) {
    // ---- a segment.  The ring is empty: all slots but the NB that follow (in ring order) the last
    //      requested one are requested now; those serve as the activation buffers first.
    const int seg_end = min(p1, (cur.grp + 1) * n_rt);
    pf.init(cur.pos, seg_end, n_rt);
#pragma unroll
    for (int i = 0; i < kRingTok - NB; ++i)
      if (alive && !pf.done()) request();
    if (!waited) {
      pdl_wait();
      waited = true;
      stamp_begin(P.stamp);
      if (threadIdx.x == 0) l2_ahead(P.ahead, blockIdx.x, gridDim.x);
      clear_arrays();
    }
    {
      const int col = cur.grp * sg + warp;
      uint8_t* buf = my_ring + ((rslot + tb) % kRingTok) * kBatchBytes;      // this warp's buffer
      uint4* xs_q = reinterpret_cast<uint4*>(buf);
      uint8_t* xs_x = buf + kXsQBytes;
      float* xs_step = reinterpret_cast<float*>(buf + kXsQBytes + kXsXBytes);
      auto publish = [&](int k, const LaneQuant& lq, float ssv, bool live) {      // k: token inside the block
        xs_q[k * 32 + lane] = lq.q;
        if (t == 0) {      // the quad's leader: the sub-block's sum as three signed bytes
          const int x = lq.sum;
          const int b0 = ((x + 128) & 255) - 128;
          const int r1 = (x - b0) >> 8;
          const int b1 = ((r1 + 128) & 255) - 128;
          const int b2 = (r1 - b1) >> 8;
          xs_x[(k * 3 + 0) * 8 + g] = static_cast<uint8_t>(b0);
          xs_x[(k * 3 + 1) * 8 + g] = static_cast<uint8_t>(b1);
          xs_x[(k * 3 + 2) * 8 + g] = static_cast<uint8_t>(b2);
        }
        if (lane == 0) xs_step[k] = lq.step;
        if (P.kind == kResidual && live) {
          float a = ssv;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
          if (lane == 0) s_red[warp * kCols + 8 * tb + k] = a;
        }
      };
      LaneQuant zero;
      zero.q = make_uint4(0, 0, 0, 0);
      zero.step = 0.f;
      zero.sum = 0;
      for (int k = 0; k < 8; k += 2) {      // two tokens per round trip
        const int tok = 8 * tb + k;
        if (tok + 1 < n_tok) {
          float v[2][8];
          float ss2[2];
          stage_warp<2>(P, col, tok, v, ss2);
          publish(k, quantise_lane_column(v[0]), ss2[0], true);
          publish(k + 1, quantise_lane_column(v[1]), ss2[1], true);
        } else if (tok < n_tok) {
          float v[1][8];
          float ss1[1];
          stage_warp<1>(P, col, tok, v, ss1);
          publish(k, quantise_lane_column(v[0]), ss1[0], true);
          publish(k + 1, zero, 0.f, false);
        } else {
          publish(k, zero, 0.f, false);
          publish(k + 1, zero, 0.f, false);
        }
      }
      __syncwarp();
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint4 q = xs_q[g * 32 + 4 * j + t];
        x_he[j] = q.x; x_ho[j] = q.y; x_le[j] = q.z; x_lo[j] = q.w;
      }
#pragma unroll
      for (int s = 0; s < 3; ++s) xm[s] = t < 2 ? *reinterpret_cast<const uint32_t*>(xs_x + (g * 3 + s) * 8 + 4 * t) : 0u;
      step[0] = xs_step[2 * t];
      step[1] = xs_step[2 * t + 1];
      __syncwarp();
      // the generic-proxy reads of the buffers are done; order them before the copies that overwrite them
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      if (NB == 2) pair_sync(1 + warp);
#pragma unroll
      for (int b = 0; b < NB; ++b)
        if (alive && !pf.done()) request();
    }
    if (P.kind == kResidual) {
      __syncthreads();
      if (threadIdx.x < n_tok) {
        float a = 0.f;
        for (int ww = 0; ww < sg; ++ww) a += s_red[ww * kCols + threadIdx.x];
        P.ssq_out[threadIdx.x * kMaxStatBlocks + cur.grp] = a;
      }
      __syncthreads();
    }
    while (cur.pos < seg_end) {
      const int nb = cur.batch();
      if (alive) {
        const bool ok = mbar_wait(bar_u32 + 8 * slot, phase, first_wait ? P.first_wait_polls : kWaitLimit);
        first_wait = false;
        if (!__all_sync(0xffffffffu, ok)) {
          alive = false;
          drain.note(slot, phase, n_in_flight);
          if (lane == 0) atomicOr(status, 1);
        }
      }
      --n_in_flight;
      const uint8_t* base = my_ring + slot * kBatchBytes;
      float* red_w = red + ((parity * kMaxWarps + warp) * kBatch) * kRowsPerTile * kCols + 8 * tb;
#pragma unroll 1
      for (int pr = 0; pr < kBatch / 2; ++pr) {
        if (2 * pr >= nb) break;
        const uint8_t* u0 = base + (2 * pr) * kUnitBytes;
        const uint8_t* u1 = u0 + kUnitBytes;
        const RowScales r0 = decode_row(*reinterpret_cast<const uint4*>(u0 + g * 16));
        const RowScales r1 = decode_row(*reinterpret_cast<const uint4*>(u1 + g * 16));
        const uint32_t a_u0 = smem_addr(u0) + piece, a_u1 = smem_addr(u1) + piece;
        // sum_j sc_j * (high, low sums)   [row g / g+8][token 2t / 2t+1]
        int accH[4] = {0, 0, 0, 0}, accL[4] = {0, 0, 0, 0};
#pragma unroll
        for (int jh = 0; jh < 2; ++jh) {
          // word t of (row g, sub-block 4 jh + i), i = 0..3, for both tiles: each matrix load reads the 16-byte
          // pieces of rows 0..7 for four sub-blocks and hands lane (g, t) bytes 4t..4t+3
          uint32_t w0[4], w1[4];
          ldmatrix_x4(w0[0], w0[1], w0[2], w0[3], a_u0 + 512 * jh);
          ldmatrix_x4(w1[0], w1[1], w1[2], w1[3], a_u1 + 512 * jh);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int j = 4 * jh + i;
            const uint32_t a0 = w0[i] & E, a1 = w1[i] & E, a2 = (w0[i] >> 4) & E, a3 = (w1[i] >> 4) & E;
            const int sc0 = r0.sc(j), sc1 = r1.sc(j);
            int dh[4], dl[4];
            mma_u8s8_zero(dh, a0, a1, a2, a3, x_he[j], x_ho[j]);
            mma_u8s8_zero(dl, a0, a1, a2, a3, x_le[j], x_lo[j]);
#pragma unroll
            for (int c = 0; c < 2; ++c) {
              accH[c] += sc0 * dh[c];
              accL[c] += sc0 * dl[c];
              accH[2 + c] += sc1 * dh[2 + c];
              accL[2 + c] += sc1 * dl[2 + c];
            }
          }
        }
        // the second sum: mins (16 rows x 8 sub-blocks) times X (8 sub-blocks x 8 tokens), one byte plane at a time
        const uint32_t am0 = min_bytes(r0, m_shift, m_mask), am1 = min_bytes(r1, m_shift, m_mask);
        int m0[4], m1[4], m2[4];
        mma_u8s8_zero(m0, am0, am1, 0u, 0u, xm[0], 0u);
        mma_u8s8_zero(m1, am0, am1, 0u, 0u, xm[1], 0u);
        mma_u8s8_zero(m2, am0, am1, 0u, 0u, xm[2], 0u);
        float y[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int mx = m0[c] + m1[c] * 256 + m2[c] * 65536;      // sum_j m_j X_j, below 2^29
          const float dd = c < 2 ? r0.d : r1.d, dm = c < 2 ? r0.dmin : r1.dmin;
          y[c] = step[c & 1] * (dd * scaled_sum(accH[c], accL[c]) - dm * static_cast<float>(mx));
        }
        // rows g of tiles 2 pr and 2 pr + 1, tokens 2t and 2t + 1 of the block
        *reinterpret_cast<float2*>(red_w + ((2 * pr) * kRowsPerTile + g) * kCols + 2 * t) = make_float2(y[0], y[1]);
        *reinterpret_cast<float2*>(red_w + ((2 * pr + 1) * kRowsPerTile + g) * kCols + 2 * t) = make_float2(y[2], y[3]);
      }
      // the whole warp has consumed the slot: hand it back and request the next batch
      __syncwarp();
      if (NB == 2) pair_sync(1 + warp);
      if (alive && !pf.done()) request();
      __syncthreads();
      // warp-ordered sum of the SG warps' partials: thread = (tile of the batch, row, token)
      for (int idx = threadIdx.x; idx < kBatch * kRowsPerTile * kCols; idx += blockDim.x) {
        const int i = idx / (kRowsPerTile * kCols);
        const int row = (idx / kCols) % kRowsPerTile;
        const int tok = idx % kCols;
        if (i < nb && tok < n_tok) {
          const float* src = red + (parity * kMaxWarps * kBatch) * kRowsPerTile * kCols + idx;
          float sum = src[0];
#pragma unroll
          for (int ww = 1; ww < kMaxWarps; ++ww)
            if (ww < sg) sum += src[ww * kBatch * kRowsPerTile * kCols];
          if (!(fabsf(sum) < kAccLimit)) atomicOr(status, 2);
          const int64_t at = acc_position(P.out_order, (cur.rt + i) * kRowsPerTile + row);
          if (in_range(at >= 0 && at < mpad && tok < P.n_tok_total, status)) atomicAdd(acc_out + static_cast<int64_t>(tok) * mpad + at, acc_from(sum));
        }
      }
      parity ^= 1;
      if (++slot == kRingTok) {
        slot = 0;
        phase ^= 1u;
      }
      cur.next(nb);
    }
  }
  if (!alive) drain.drain(bar_u32, kRingTok);
  stamp_end(P.stamp);
}

template <int NB>
cudaError_t launch_tokens(const GemvParams& P, int64_t grid, cudaStream_t st) {
  auto kern = gemv_tokens_kernel<NB>;
  static bool configured[kMaxDevices] = {};
  int dev = -1;
  if (first_launch_on_device(configured, &dev)) {
    const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(gemv_tokens_smem_bytes<NB>(kMaxWarps)));
    if (e != cudaSuccess) return e;
    if (dev >= 0) configured[dev] = true;
  }
  return launch_pdl(kern, dim3(static_cast<unsigned>(grid)), dim3(NB * P.sg * 32), gemv_tokens_smem_bytes<NB>(P.sg), st, P);
}

}  // namespace

int gemv_tokens_ctas_per_sm(int n_tok) { return n_tok <= 8 ? 2 : 1; }

cudaError_t launch_gemv_tokens(const gemv_detail::GemvParams& P, int64_t grid, cudaStream_t st) {
  return P.n_tok_total <= 8 ? launch_tokens<1>(P, grid, st) : launch_tokens<2>(P, grid, st);
}

}  // namespace prima
