// Dequantise-fused Q4_K matrix-vector / small-n matrix product, streaming formulation.
//
// Work decomposition.  The matrix is a grid of units (row tile of 8 rows  x  super-block column of
// 256 weights, 1152 bytes each, see common.cuh) stored column-major.  The n_sb columns are taken in
// groups of SG adjacent columns (SG = the largest divisor of n_sb that is <= 8); a CTA has SG warps,
// warp w always works on column  group*SG + w.  CTA b of a persistent grid (2 CTAs per SM) works for
// group b mod n_groups and takes an even, contiguous share of that group's row tiles, so all CTAs
// get the same number of tiles to within one.  A CTA walks its range in batches of up to 4
// consecutive row tiles of one group (a batch never crosses a group boundary), so each warp's part
// of a batch is one contiguous piece of HBM of up to 4608 bytes, and the warp keeps its column's
// 256 activations in registers for the whole walk.
//
// Data movement.  Each warp owns a ring of kRing batch slots in shared memory.  Lane 0 requests a
// batch with one 1-D bulk asynchronous copy (TMA) that signals an mbarrier with its byte count;
// the warp waits on the mbarrier (bounded: a wait that does not end raises the status word and the
// kernel drains and returns), reads its three 16-byte pieces per unit with ordinary shared loads,
// and after the batch is consumed lane 0 re-arms the slot with the next request.  Memory-level
// parallelism is therefore set by the ring, not by registers or occupancy.
//
// Arithmetic.  Lane (g, t) = (lane / 4, lane % 4) owns row g of the tile and sub-blocks t and
// 4 + t of the super-block.  The activations of a sub-block are held as 16-bit integers
// x_q = round(x / s_j), |x_q| <= 32639, with one fp32 step s_j = max|x| / 32639 per sub-block,
// split into two signed bytes x_q = 256 hi + lo.  Nibbles are masked in place into unsigned bytes
// (even nibbles as q, odd nibbles as 16 q, shifted back after the sums).  I_j = sum q * x_q is an
// exact integer below 2^24, and so are sc_j * I_j and m_j * sum(x_q) in 32 bits; the only rounding
// errors are the 16-bit step of x (about 2e-5 of a typical activation) and a few fp32 operations
// per sub-block:  partial = sum_j s_j * (d * sc_j * I_j  -  dmin * m_j * sum(x_q)).
// Two interchangeable inner products compute I_j:
//   * dp4a: 4-way byte dot products on the integer pipe (hi and lo parts separately);
//   * mma:  the int8 tensor-core instruction m16n8k32.  Rows 0-7 / 8-15 of the A tile are two
//           consecutive row tiles; the 32 k-slots are two 16-byte words' worth of nibbles of the four
//           sub-blocks held by the lane quad; the 8 columns of B are (sub-block of the quad) x
//           (hi, lo), with a lane's activation bytes in its own sub-block's columns and zeros
//           elsewhere, so D[row][2t], D[row][2t+1] are exactly lane (row, t)'s hi and lo sums.
//           With several tokens, one such instruction per token.
// With RMSNorm fused, x is multiplied by the gain before quantisation and the scalar
// rsqrt(mean(x^2) + eps) is applied to the fp32 partial.
//
// Output.  A lane's four tile partials of a batch are reduced over the quad with a transposing
// shuffle (lane t ends with tile t's row sum), the SG warps of the CTA add theirs through shared
// memory in warp order (one barrier per batch, double-buffered), giving one partial sum per (column
// group, row, token), which is added into the row's 64-bit fixed-point accumulator
// acc[tok * mpad + row] with an integer atomic (see common.cuh): the sum over the column groups is
// exact in the integers, so the bits do not depend on the order in which CTAs arrive.
#include <cstdlib>

#include "gemv_device.cuh"

namespace prima {

int gemv_group_size(int64_t n_sb) {
  for (int sg = 8; sg > 1; --sg)
    if (n_sb % sg == 0) return sg;
  return 1;
}

namespace {
using namespace gemv_detail;

// ---- integer inner products -----------------------------------------------------------------------
__device__ __forceinline__ int dp4a_us(uint32_t a, uint32_t b, int c) {   // unsigned bytes x signed bytes
  int d;
  asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// The 32 activations of one sub-block as signed bytes: hi[2w + p] / lo[2w + p] hold the high / low
// bytes of x_q for weights 8w + p, 8w + p + 2, 8w + p + 4, 8w + p + 6 (p = 0 even nibbles, 1 odd).
struct SubX {
  uint32_t hi[8], lo[8];
  float step;   // s_j
  int sum;      // sum of x_q
};

// Quantise the lane's 8 staged values with one step per 32-weight sub-block (see LaneQuant).
__device__ __forceinline__ LaneQuant quantise_lane(const float (&v)[8]) {
  float amax = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(v[i]));
  amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
  amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
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

// Collect sub-block j (0..7) from the lanes 4j .. 4j+3 that quantised it.
__device__ __forceinline__ void gather_sub(const LaneQuant& mine, int j, SubX& out) {
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    const int src = 4 * j + w;
    out.hi[2 * w] = __shfl_sync(0xffffffffu, mine.q.x, src);
    out.hi[2 * w + 1] = __shfl_sync(0xffffffffu, mine.q.y, src);
    out.lo[2 * w] = __shfl_sync(0xffffffffu, mine.q.z, src);
    out.lo[2 * w + 1] = __shfl_sync(0xffffffffu, mine.q.w, src);
  }
  out.step = __shfl_sync(0xffffffffu, mine.step, 4 * j);
  out.sum = __shfl_sync(0xffffffffu, mine.sum, 4 * j);
}

// What a lane keeps of one sub-block for the multiplications.
//   dp4a variant: all 16 byte registers.
//   mma variant:  the B-operand registers of the lane: its hi bytes if it sits in column 2t, its lo
//                 bytes if in column 2t+1, zeros otherwise (8 registers), plus step and sum.
template <bool MMA>
struct LaneX;
template <>
struct LaneX<false> {
  uint32_t hi[8], lo[8];
  float step;
  int sum;
  __device__ __forceinline__ void set(const SubX& s, int, int) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      hi[i] = s.hi[i];
      lo[i] = s.lo[i];
    }
    step = s.step;
    sum = s.sum;
  }
};
template <>
struct LaneX<true> {
  uint32_t b[8];
  float step;
  int sum;
  __device__ __forceinline__ void set(const SubX& s, int g, int t) {
    const bool mine = (g >> 1) == t;
    const bool low = g & 1;
#pragma unroll
    for (int i = 0; i < 8; ++i) b[i] = mine ? (low ? s.lo[i] : s.hi[i]) : 0u;
    step = s.step;
    sum = s.sum;
  }
};

// I = sum over the 32 weights of one 16-byte chunk of q * x_q, dp4a variant.
__device__ __forceinline__ int chunk_dot(const uint4& q, const LaneX<false>& x) {
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
  int he = 0, ho = 0, le = 0, lo = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint32_t e = w[i] & 0x0f0f0f0fu, o = w[i] & 0xf0f0f0f0u;
    he = dp4a_us(e, x.hi[2 * i], he);
    ho = dp4a_us(o, x.hi[2 * i + 1], ho);
    le = dp4a_us(e, x.lo[2 * i], le);
    lo = dp4a_us(o, x.lo[2 * i + 1], lo);
  }
  return he * 256 + le + ((ho * 256 + lo) >> 4);
}

// Two row tiles (u0 -> rows 0-7, u1 -> rows 8-15) of one chunk, mma variant: the lane's I for u0, u1.
__device__ __forceinline__ void chunk_dot2(const uint4& q_u0, const uint4& q_u1, const LaneX<true>& x, int& i_u0, int& i_u1) {
  int ce[4] = {0, 0, 0, 0}, co[4] = {0, 0, 0, 0};
  constexpr uint32_t E = 0x0f0f0f0fu, O = 0xf0f0f0f0u;
  mma_u8s8(ce, q_u0.x & E, q_u1.x & E, q_u0.y & E, q_u1.y & E, x.b[0], x.b[2]);
  mma_u8s8(co, q_u0.x & O, q_u1.x & O, q_u0.y & O, q_u1.y & O, x.b[1], x.b[3]);
  mma_u8s8(ce, q_u0.z & E, q_u1.z & E, q_u0.w & E, q_u1.w & E, x.b[4], x.b[6]);
  mma_u8s8(co, q_u0.z & O, q_u1.z & O, q_u0.w & O, q_u1.w & O, x.b[5], x.b[7]);
  i_u0 = ce[0] * 256 + ce[1] + ((co[0] * 256 + co[1]) >> 4);
  i_u1 = ce[2] * 256 + ce[3] + ((co[2] * 256 + co[3]) >> 4);
}
__device__ __forceinline__ void chunk_dot2(const uint4& q_u0, const uint4& q_u1, const LaneX<false>& x, int& i_u0, int& i_u1) {
  i_u0 = chunk_dot(q_u0, x);
  i_u1 = chunk_dot(q_u1, x);
}

// Header of one unit row -> the lane's scale factors.
struct LaneScales {
  float d, dmin;
  int sc_lo, sc_hi, m_lo, m_hi;
};
__device__ __forceinline__ LaneScales decode_header(const uint4& h, uint32_t sel_a, uint32_t sel_b) {
  LaneScales r;
  const float2 df = __half22float2(*reinterpret_cast<const __half2*>(&h.x));
  r.d = df.x;
  r.dmin = df.y;
  const uint32_t f = __byte_perm(__byte_perm(h.y, h.z, sel_a), h.w, sel_b);
  r.sc_lo = f & 63u;
  r.sc_hi = (f >> 6) & 63u;
  r.m_lo = (f >> 12) & 63u;
  r.m_hi = (f >> 18) & 63u;
  return r;
}
__device__ __forceinline__ float unit_partial(const LaneScales& s, int i0, int i1, float step_a, int sum_a, float step_b, int sum_b) {
  const float a0 = static_cast<float>(s.sc_lo * i0), a1 = static_cast<float>(s.sc_hi * i1);
  const float b0 = static_cast<float>(s.m_lo * sum_a), b1 = static_cast<float>(s.m_hi * sum_b);
  return step_a * (s.d * a0 - s.dmin * b0) + step_b * (s.d * a1 - s.dmin * b1);
}

template <int NTOK, bool MMA>
__global__ void __launch_bounds__(kMaxWarps * 32, (NTOK == 1 ? 2 : 1)) gemv_partials_kernel(const GemvParams P) {
  pdl_trigger();
  extern __shared__ __align__(128) uint8_t smem[];
  // layout: [warps][kRing][4608] batches, [warps][kRing] mbarriers, the reduction buffer
  // [2][NTOK][kMaxWarps][kBatch][8], a small scratch for the sums of squares
  const int n_warps = blockDim.x >> 5;
  const uint8_t* __restrict__ w = P.w;
  const int n_rt = P.n_rt, n_sb = P.n_sb, sg = P.sg, tok0 = P.tok0;
  acc_t* __restrict__ acc_out = P.acc;
  const int64_t mpad = P.mpad;
  int* __restrict__ status = P.status;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + static_cast<size_t>(n_warps) * kRing * kBatchBytes);
  float* red = reinterpret_cast<float*>(bars + ((n_warps * kRing + 15) & ~15));   // keeps what follows 128-byte aligned
  float* s_red = red + 2 * NTOK * kMaxWarps * kBatch * kRowsPerTile;   // [warps][NTOK]

  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  // This CTA's range of (group, row tile) positions.  When the grid has at least one CTA per column
  // group, every group gets the same number of CTAs and a range never crosses a group boundary (a
  // crossing costs a second activation load in mid-stream, which only that CTA pays and everybody
  // waits for); otherwise the positions are cut evenly.
  const int n_groups = n_sb / sg;
  const int n_pos = n_groups * n_rt;
  int p0 = 0, p1 = 0;
  const int per_group = gridDim.x / n_groups;
  if (per_group >= 1) {
    // CTAs of one group are spread evenly over the launch order (CTA b works for group b mod
    // n_groups): CTAs that start later, or share an SM with an older CTA, run a little slower, and
    // every group should get the same mix of them.
    const int grp = blockIdx.x % n_groups, i = blockIdx.x / n_groups;
    if (i < per_group) {
      p0 = grp * n_rt + static_cast<int>(static_cast<int64_t>(n_rt) * i / per_group);
      p1 = grp * n_rt + static_cast<int>(static_cast<int64_t>(n_rt) * (i + 1) / per_group);
    }
  } else {
    p0 = static_cast<int>(static_cast<int64_t>(n_pos) * blockIdx.x / gridDim.x);
    p1 = static_cast<int>(static_cast<int64_t>(n_pos) * (blockIdx.x + 1) / gridDim.x);
  }
  // Every CTA of the grid, also one without positions, clears its share of the accumulator arrays
  // whose readers are done once the predecessor kernel is.
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

  const uint8_t* my_ring = smem + static_cast<size_t>(warp) * kRing * kBatchBytes;
  const uint32_t ring_u32 = smem_addr(my_ring);
  const uint32_t bar_u32 = smem_addr(bars + warp * kRing);
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < kRing; ++i) mbar_init(bar_u32 + 8 * i, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncwarp();

  Walk pf, cur;                 // next batch to request / batch being computed
  cur.init(p0, p1, n_rt);
  int n_in_flight = 0;          // requested and not yet waited for
  int rslot = 0;                // ring slot of the next request (requests and waits go round the ring in step)
  auto request = [&]() {
    const int nb = pf.batch();
    if (lane == 0) {
      const uint8_t* src = w + (static_cast<int64_t>(pf.grp * sg + warp) * n_rt + pf.rt) * kUnitBytes;
      // (range-checked build: the batch lies inside the matrix; a request that does not is left out and its wait runs out)
      if (in_range(src >= w && src + nb * kUnitBytes <= w + static_cast<int64_t>(n_sb) * n_rt * kUnitBytes && nb >= 1 && nb <= kBatch, status)) {
        mbar_expect_tx(bar_u32 + 8 * rslot, nb * kUnitBytes);
        bulk_load(ring_u32 + rslot * kBatchBytes, src, nb * kUnitBytes, bar_u32 + 8 * rslot, stream_once_policy());
      }
    }
    pf.next(nb);
    ++n_in_flight;
    if (++rslot == kRing) rslot = 0;
  };

  const int my_piece = kUnitHdrBytes + unit_piece_slot(g, t) * 16;      // this lane's nibble piece inside a unit
  // lane-constant byte selectors that pull this lane's 24-bit field group out of header words 1..3
  const uint32_t sel_a = t == 1 ? 0x7654u : (t == 3 ? 0x0073u : 0x3210u);
  const uint32_t sel_b = t == 2 ? 0x7654u : (t == 3 ? 0x0710u : 0x3210u);

  LaneX<MMA> xa[NTOK], xb[NTOK];   // sub-blocks t and 4 + t of the current column
  int parity = 0;
  bool alive = true;
  bool waited = false;
  bool first_wait = true;
  RingDrain drain;
  int slot = 0;                  // ring slot of the next wait
  uint32_t phase = 0;

  while (!cur.done()) {
    // ---- a segment: the positions of one column group.  The ring is empty here: fill it, then
    //      (after the dependency wait) stage and quantise this column's activations in registers.
    const int seg_end = min(p1, (cur.grp + 1) * n_rt);
    pf.init(cur.pos, seg_end, n_rt);
#pragma unroll
    for (int i = 0; i < kRing; ++i)
      if (alive && !pf.done()) request();
    if (!waited) {      // the first weight batches are on their way; everything below depends on the predecessor kernel
      pdl_wait();
      waited = true;
      stamp_begin(P.stamp);
      if (threadIdx.x == 0) l2_ahead(P.ahead, blockIdx.x, gridDim.x);
      clear_arrays();
    }
    {
      float v[NTOK][8];
      float ss[NTOK];
      stage_warp<NTOK>(P, cur.grp * sg + warp, tok0, v, ss);
#pragma unroll
      for (int k = 0; k < NTOK; ++k) {
        const LaneQuant lq = quantise_lane(v[k]);
        SubX tmp;
        gather_sub(lq, t, tmp);
        xa[k].set(tmp, g, t);
        gather_sub(lq, 4 + t, tmp);
        xb[k].set(tmp, g, t);
      }
      if (P.kind == kResidual) {   // sums of squares of the group: lanes, then warps, in a fixed order
#pragma unroll
        for (int k = 0; k < NTOK; ++k) {
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) ss[k] += __shfl_xor_sync(0xffffffffu, ss[k], o);
          if (lane == 0) s_red[warp * NTOK + k] = ss[k];
        }
        __syncthreads();
        if (threadIdx.x < NTOK) {
          float a = 0.f;
          for (int ww = 0; ww < n_warps; ++ww) a += s_red[ww * NTOK + threadIdx.x];
          P.ssq_out[(tok0 + threadIdx.x) * kMaxStatBlocks + cur.grp] = a;
        }
        __syncthreads();
      }
    }
    while (cur.pos < seg_end) {
    const int nb = cur.batch();
    if (alive) {
      const bool ok = mbar_wait(bar_u32 + 8 * slot, phase, first_wait ? P.first_wait_polls : kWaitLimit);
      first_wait = false;
      if (!__all_sync(0xffffffffu, ok)) {      // the same verdict in every lane
        alive = false;
        drain.note(slot, phase, n_in_flight);
        if (lane == 0) atomicOr(status, 1);
      }
    }
    --n_in_flight;
    const uint8_t* base = my_ring + slot * kBatchBytes;
    float acc[NTOK][kBatch];
#pragma unroll
    for (int pr = 0; pr < kBatch / 2; ++pr) {
      const uint8_t* u0 = base + (2 * pr) * kUnitBytes;
      const uint8_t* u1 = u0 + kUnitBytes;
      const LaneScales s0 = decode_header(*reinterpret_cast<const uint4*>(u0 + g * 16), sel_a, sel_b);
      const LaneScales s1 = decode_header(*reinterpret_cast<const uint4*>(u1 + g * 16), sel_a, sel_b);
      const uint4 qa0 = *reinterpret_cast<const uint4*>(u0 + my_piece);
      const uint4 qa1 = *reinterpret_cast<const uint4*>(u1 + my_piece);
      const uint4 qb0 = *reinterpret_cast<const uint4*>(u0 + my_piece + 512);
      const uint4 qb1 = *reinterpret_cast<const uint4*>(u1 + my_piece + 512);
#pragma unroll
      for (int k = 0; k < NTOK; ++k) {
        int ia0, ia1, ib0, ib1;
        chunk_dot2(qa0, qa1, xa[k], ia0, ia1);
        chunk_dot2(qb0, qb1, xb[k], ib0, ib1);
        acc[k][2 * pr] = unit_partial(s0, ia0, ib0, xa[k].step, xa[k].sum, xb[k].step, xb[k].sum);
        acc[k][2 * pr + 1] = unit_partial(s1, ia1, ib1, xa[k].step, xa[k].sum, xb[k].step, xb[k].sum);
      }
    }
    // the whole warp has consumed the slot: hand it back and request the next batch
    __syncwarp();
    if (alive && !pf.done()) request();

    // quad reduction with transposition: lane t ends with the row sum of tile t
#pragma unroll
    for (int k = 0; k < NTOK; ++k) {
      const bool odd = t & 1, upper = t & 2;
      float k0 = odd ? acc[k][1] : acc[k][0];
      const float s0 = odd ? acc[k][0] : acc[k][1];
      float k1 = odd ? acc[k][3] : acc[k][2];
      const float s1 = odd ? acc[k][2] : acc[k][3];
      k0 += __shfl_xor_sync(0xffffffffu, s0, 1);
      k1 += __shfl_xor_sync(0xffffffffu, s1, 1);
      float kk = upper ? k1 : k0;
      const float ss = upper ? k0 : k1;
      kk += __shfl_xor_sync(0xffffffffu, ss, 2);
      red[(((parity * NTOK + k) * kMaxWarps + warp) * kBatch + t) * kRowsPerTile + g] = kk;
    }
    __syncthreads();
    // warp-ordered sum of the SG warps' partials: one thread per (token, tile of the batch, row)
    for (int idx = threadIdx.x; idx < NTOK * kBatch * kRowsPerTile; idx += blockDim.x) {
      const int k = idx / (kBatch * kRowsPerTile);
      const int i = (idx / kRowsPerTile) % kBatch;
      const int row = idx % kRowsPerTile;
      if (i < nb) {
        const float* src = red + ((parity * NTOK + k) * kMaxWarps * kBatch + i) * kRowsPerTile + row;
        float sum = src[0];
        for (int ww = 1; ww < sg; ++ww) sum += src[ww * kBatch * kRowsPerTile];
        if (!(fabsf(sum) < kAccLimit)) atomicOr(status, 2);
        const int64_t at = acc_position(P.out_order, (cur.rt + i) * kRowsPerTile + row);
        if (in_range(at >= 0 && at < mpad && tok0 + k < P.n_tok_total, status)) atomicAdd(acc_out + static_cast<int64_t>(tok0 + k) * mpad + at, acc_from(sum));
      }
    }
    parity ^= 1;
    if (++slot == kRing) {
      slot = 0;
      phase ^= 1u;
    }
    cur.next(nb);
    }
  }
  // A wait gave up: copies may still be on their way to this CTA's shared memory.
  if (!alive) drain.drain(bar_u32, kRing);
  stamp_end(P.stamp);
}

size_t gemv_smem_bytes(int sg, int n_tok) {
  return static_cast<size_t>(sg) * kRing * kBatchBytes + static_cast<size_t>((sg * kRing + 15) & ~15) * 8 +
         static_cast<size_t>(2) * n_tok * kMaxWarps * kBatch * kRowsPerTile * sizeof(float) +
         static_cast<size_t>(kMaxWarps) * n_tok * sizeof(float);
}

template <int NTOK, bool MMA>
cudaError_t launch_one(const GemvParams& P, int64_t grid, cudaStream_t st) {
  auto kern = gemv_partials_kernel<NTOK, MMA>;
  static bool configured[kMaxDevices] = {};
  int dev = -1;
  if (first_launch_on_device(configured, &dev)) {
    const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(gemv_smem_bytes(kMaxWarps, NTOK)));
    if (e != cudaSuccess) return e;
    if (dev >= 0) configured[dev] = true;
  }
  return launch_pdl(kern, dim3(static_cast<unsigned>(grid)), dim3(P.sg * 32), gemv_smem_bytes(P.sg, NTOK), st, P);
}

template <bool MMA>
cudaError_t launch_n(int n, const GemvParams& P, int64_t grid, cudaStream_t st) {
  switch (n) {
    case 1: return launch_one<1, MMA>(P, grid, st);
    case 2: return launch_one<2, MMA>(P, grid, st);
    case 3: return launch_one<3, MMA>(P, grid, st);
    default: return launch_one<4, MMA>(P, grid, st);
  }
}

}  // namespace

// Which inner product the GEMV uses.  Environment variable PRIMA_GEMV_KERNEL = "dp4a" or "mma"
// (read once per process); the tensor-core variant is the default.
bool gemv_uses_tensor_cores() {
  static const bool mma = [] {
    const char* v = getenv("PRIMA_GEMV_KERNEL");
    return !(v && v[0] == 'd');
  }();
  return mma;
}

int launch_gemv_partials(const TiledMat& w, GemvIn& in, int n_tok, acc_t* acc, int sm_count, cudaStream_t st) {
  if (w.n_rt == 0 || w.n_sb == 0) return 0;
  if (w.n_rt * w.n_sb >= (int64_t(1) << 31)) return cuda_rc(cudaErrorInvalidValue);
  const int sg = gemv_group_size(w.n_sb);
  const int64_t n_pos = (w.n_sb / sg) * w.n_rt;
  in.ssq_out.n_groups = static_cast<int>(w.n_sb / sg);
  in.ssq_out.width = w.cols;
  GemvParams P;
  P.w = w.data; P.n_rt = static_cast<int>(w.n_rt); P.n_sb = static_cast<int>(w.n_sb); P.sg = sg;
  P.kind = in.kind; P.x = in.x; P.h_in = in.h_in; P.h_out = in.h_out; P.acc_in = in.acc_in;
  P.mpad_in = in.mpad_in; P.gain = in.gain; P.ssq_out = in.ssq_out.data; P.ssq_in = in.ssq_in.data; P.n_ssq_in = in.ssq_in.n_groups;
  P.inv_width_in = in.ssq_in.width > 0 ? 1.0f / static_cast<float>(in.ssq_in.width) : 0.f;
  P.eps_in = in.ssq_in.eps;
  P.n_tok_total = n_tok; P.acc = acc; P.mpad = w.mpad(); P.status = in.status;
  P.zero0 = in.zero0; P.zero0_n = in.zero0_n; P.zero1 = in.zero1; P.zero1_n = in.zero1_n;
  P.out_order = in.out_order;
  P.stamp = in.stamp;
  P.ahead = in.ahead;
  P.first_wait_polls = in.first_wait_polls ? in.first_wait_polls - 1 : kWaitLimit;
  if ((in.out_order == kOrderResidual && w.mpad() % 256 != 0) || (in.out_order == kOrderSwiglu && w.mpad() % 512 != 0)) return cuda_rc(cudaErrorInvalidValue);
  int launches = 0;
  if (n_tok >= 4 && gemv_uses_tensor_cores()) {
    // 4..16 tokens: one pass over the weights with the tokens as columns of the tensor-core product (up to 3
    // tokens the one-token formulation with one instruction per token is faster; measured on 6 layers of the 70B
    // shape: 0.89 against 1.08 ms at 2 tokens, 1.08 against 1.12 at 3, 1.35 against 1.16 at 4)
    int64_t grid = static_cast<int64_t>(sm_count) * std::max(1, gemv_tokens_ctas_per_sm(n_tok) * kMaxWarps / sg);
    if (grid > n_pos) grid = n_pos;
    P.tok0 = 0;
    const cudaError_t e = launch_gemv_tokens(P, grid, st);
    if (e != cudaSuccess) return cuda_rc(e);
    return 1;
  }
  int tok = 0;
  while (tok < n_tok) {
    // up to 4 tokens per pass; more tokens are split as evenly as possible over the fewest passes
    const int left = n_tok - tok;
    const int passes = (left + 3) / 4;
    const int chunk = (left + passes - 1) / passes;
    const int warps_per_sm = chunk == 1 ? 16 : 8;
    int64_t grid = static_cast<int64_t>(sm_count) * std::max(1, warps_per_sm / sg);
    if (grid > n_pos) grid = n_pos;
    P.tok0 = tok;
    const cudaError_t e = gemv_uses_tensor_cores() ? launch_n<true>(chunk, P, grid, st) : launch_n<false>(chunk, P, grid, st);
    if (e != cudaSuccess) return cuda_rc(e);
    P.zero0_n = P.zero1_n = 0;   // cleared by the first pass
    ++launches;
    tok += chunk;
  }
  return launches;
}

}  // namespace prima
