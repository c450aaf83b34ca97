// Device-side pieces shared by the two streaming products over the tiled Q4_K matrix (q4k_gemv.cu: one
// token, or up to four with one tensor-core instruction per token; q4k_gemm_tokens.cu: five to eight
// tokens as the columns of the tensor-core product): the ring of bulk copies, the kernel parameters,
// the staging step that finishes the producer's output, and the walk over a CTA's share of the matrix.
#pragma once

#include "common.cuh"

namespace prima {
namespace gemv_detail {

constexpr int kMaxWarps = 8;
constexpr int kBatch = 4;                    // row tiles per batch (= lanes of a quad)
constexpr int kBatchBytes = kBatch * kUnitBytes;
constexpr int kRing = 3;                     // batches in flight per warp
constexpr uint32_t kWaitLimit = 1u << 24;    // polls of one mbarrier wait before the kernel gives up


// ---- asynchronous bulk copies (TMA, 1-D) into a per-warp ring, completion through mbarriers ------
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// The weights are read once per token and never again before hundreds of MB of other weights have
// passed: they are marked evict-first in L2, so that the small arrays the kernels hand to each other
// (partial sums, the residual stream, gains, statistics) stay resident instead of being pushed out.
__device__ __forceinline__ uint64_t stream_once_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
               "l"(__cvta_generic_to_global(src)), "r"(bytes), "r"(bar), "l"(policy)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false if the phase did not complete within `limit` polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t limit = kWaitLimit) {
  for (uint32_t i = 0; i < limit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}

// Book-keeping of a warp's ring for the case that a wait gives up.  Requests and waits go round the
// ring in step, so the copies still on their way when a wait fails are those of the failing slot and
// of the slots requested after it.  The warp issues no further requests, goes through the rest of
// its loop without touching the ring (it must keep taking part in the CTA's barriers), and before
// the CTA exits -- which releases the shared memory the copies are heading for -- gives every one of
// those slots one more bounded wait.
struct RingDrain {
  int slot = 0, n = 0;
  uint32_t phase = 0;
  __device__ __forceinline__ void note(int failing_slot, uint32_t failing_phase, int outstanding) {
    slot = failing_slot;
    phase = failing_phase;
    n = outstanding;
  }
  __device__ __forceinline__ void drain(uint32_t bar0, int ring) {
    for (int i = 0; i < n; ++i) {
      mbar_wait(bar0 + 8 * slot, phase);
      if (++slot == ring) {
        slot = 0;
        phase ^= 1u;
      }
    }
    n = 0;
  }
};

// D(16x8, s32) += A(16x32, u8, row) * B(32x8, s8, col)
__device__ __forceinline__ void mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}


// The same with a zero accumulator: D = A * B (no registers have to be cleared for it).
__device__ __forceinline__ void mma_u8s8_zero(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(0));
}

// Quantise the warp's 256 staged activations, every lane its own 8 values: lane l holds quarter
// l % 4 of sub-block l / 4, i.e. exactly word l % 4 of that sub-block's byte registers
// (q = [hi even, hi odd, lo even, lo odd]).  Maximum and sum over the sub-block come from shuffles.
struct LaneQuant {
  uint4 q;
  float step;
  int sum;
};
// Kernel parameters (see GemvIn in common.cuh).
struct GemvParams {
  const uint8_t* w;
  int n_rt, n_sb, sg;
  int kind;
  const float* x;
  const float* h_in;
  float* h_out;
  const acc_t* acc_in;
  int64_t mpad_in;
  const float* gain;
  float* ssq_out;
  const float* ssq_in;
  int n_ssq_in;
  float inv_width_in, eps_in;
  int tok0, n_tok_total;
  acc_t* acc;
  int64_t mpad;
  acc_t* zero0;
  int64_t zero0_n;
  acc_t* zero1;
  int64_t zero1_n;
  int out_order;
  int* status;
  Stamp stamp;
  L2Ahead ahead;
  uint32_t first_wait_polls;   // poll limit of a warp's first wait (kWaitLimit in normal use; a test lowers it to exercise the give-up path)
};

// Loads of what another kernel wrote go to L2 directly.
__device__ __forceinline__ float4 ld_l2(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ ulonglong2 ld_l2(const acc_t* p) { return __ldcg(reinterpret_cast<const ulonglong2*>(p)); }

// A warp stages the 256 activations of its column s for NTOK tokens in registers, finishing the
// producer's output on the way; lane l owns columns 8l .. 8l+7 (v[k][0..7]).  ss[k] receives the
// lane's share of the sum of squares (kResidual).  This step sits on the critical path between two
// products and a round trip to L2 takes about a microsecond, so every load of a token is issued
// before any is used.
template <int NTOK, int K0, int N>
__device__ __forceinline__ void stage_tokens(const GemvParams& P, int s, int tok_first, float (&v)[NTOK][8], float (&ss)[NTOK]) {
  const int lane = threadIdx.x & 31;
  const int64_t cols = static_cast<int64_t>(P.n_sb) * 256;
  const int64_t k0 = static_cast<int64_t>(s) * 256 + 8 * lane;
  // Tokens K0 .. K0 + N - 1 of the pass: their loads come first (one round trip), then the arithmetic.
  if (P.kind == kPlain) {
    float4 a[NTOK], b[NTOK];
#pragma unroll
    for (int k = K0; k < K0 + N; ++k) {
      const float* x = P.x + static_cast<int64_t>(tok_first + k) * cols + k0;
      a[k] = ld_l2(x);
      b[k] = ld_l2(x + 4);
    }
#pragma unroll
    for (int k = K0; k < K0 + N; ++k) {
      ss[k] = 0.f;
      v[k][0] = a[k].x; v[k][1] = a[k].y; v[k][2] = a[k].z; v[k][3] = a[k].w;
      v[k][4] = b[k].x; v[k][5] = b[k].y; v[k][6] = b[k].z; v[k][7] = b[k].w;
    }
  } else if (P.kind == kResidual) {
    float4 h0[NTOK], h1[NTOK];
    ulonglong2 a[NTOK][4];
    const bool has_acc = P.acc_in != nullptr;
#pragma unroll
    for (int k = K0; k < K0 + N; ++k) {
      const int64_t row = static_cast<int64_t>(tok_first + k);
      h0[k] = ld_l2(P.h_in + row * cols + k0);
      h1[k] = ld_l2(P.h_in + row * cols + k0 + 4);
      if (has_acc) {
        const acc_t* ain = P.acc_in + row * P.mpad_in + static_cast<int64_t>(s) * 256;   // kOrderResidual
#pragma unroll
        for (int i = 0; i < 4; ++i) a[k][i] = ld_l2(ain + 2 * (32 * i + lane));
      }
    }
    const float4 g0 = __ldg(reinterpret_cast<const float4*>(P.gain + k0)), g1 = __ldg(reinterpret_cast<const float4*>(P.gain + k0 + 4));
    const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
    for (int k = K0; k < K0 + N; ++k) {
      const int64_t row = static_cast<int64_t>(tok_first + k);
      float r[8] = {h0[k].x, h0[k].y, h0[k].z, h0[k].w, h1[k].x, h1[k].y, h1[k].z, h1[k].w};
      if (has_acc) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          r[2 * i] += acc_value(a[k][i].x);
          r[2 * i + 1] += acc_value(a[k][i].y);
        }
      }
      *reinterpret_cast<float4*>(P.h_out + row * cols + k0) = make_float4(r[0], r[1], r[2], r[3]);
      *reinterpret_cast<float4*>(P.h_out + row * cols + k0 + 4) = make_float4(r[4], r[5], r[6], r[7]);
      ss[k] = ((r[0] * r[0] + r[1] * r[1]) + (r[2] * r[2] + r[3] * r[3])) + ((r[4] * r[4] + r[5] * r[5]) + (r[6] * r[6] + r[7] * r[7]));
#pragma unroll
      for (int i = 0; i < 8; ++i) v[k][i] = r[i] * gg[i];
    }
  } else {   // kSwiglu: the previous product's fused rows 2c (gate) and 2c+1 (up): 16 consecutive accumulators
    ulonglong2 a[NTOK][8];
    float ssq[NTOK];
#pragma unroll
    for (int k = K0; k < K0 + N; ++k) {
      const acc_t* ain = P.acc_in + static_cast<int64_t>(tok_first + k) * P.mpad_in + static_cast<int64_t>(s) * 512;   // kOrderSwiglu
#pragma unroll
      for (int i = 0; i < 8; ++i) a[k][i] = ld_l2(ain + 2 * (32 * i + lane));
    }
#pragma unroll
    for (int k = K0; k < K0 + N; ++k) {
      ssq[k] = 0.f;
      const float* sp = P.ssq_in + (tok_first + k) * kMaxStatBlocks;
      for (int g0 = 0; g0 < P.n_ssq_in; g0 += 8) {     // groups added in ascending order
        float sq[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (g0 + i < P.n_ssq_in) sq[i] = __ldcg(sp + g0 + i);
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (g0 + i < P.n_ssq_in) ssq[k] += sq[i];
      }
    }
#pragma unroll
    for (int k = K0; k < K0 + N; ++k) {
      ss[k] = 0.f;
      const float inv = 1.0f / sqrtf(ssq[k] * P.inv_width_in + P.eps_in);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float gt = acc_value(a[k][i].x) * inv, up = acc_value(a[k][i].y) * inv;
        v[k][i] = gt / (1.0f + expf(-gt)) * up;
      }
    }
  }
}

// One or two tokens: one round trip.  Three or four tokens are staged one at a time: with their
// activation registers (20 per token) there is no room for more loads in flight without spills.
template <int NTOK>
__device__ __forceinline__ void stage_warp(const GemvParams& P, int s, int tok_first, float (&v)[NTOK][8], float (&ss)[NTOK]) {
  static_assert(NTOK <= 4, "at most four tokens per pass of this kernel");
  if constexpr (NTOK <= 2) {
    stage_tokens<NTOK, 0, NTOK>(P, s, tok_first, v, ss);
  } else {
    stage_tokens<NTOK, 0, 1>(P, s, tok_first, v, ss);
    stage_tokens<NTOK, 1, 1>(P, s, tok_first, v, ss);
    stage_tokens<NTOK, 2, 1>(P, s, tok_first, v, ss);
    if constexpr (NTOK == 4) stage_tokens<NTOK, 3, 1>(P, s, tok_first, v, ss);
  }
}

// Walk over the (group, row tile) positions pos .. end-1 in batches of at most kBatch tiles that do
// not cross a group boundary.
struct Walk {
  int pos, end, grp, rt, n_rt;
  __device__ __forceinline__ void init(int p, int e, int n_rt_) {
    pos = p;
    end = e;
    n_rt = n_rt_;
    grp = p / n_rt_;
    rt = p - grp * n_rt_;
  }
  __device__ __forceinline__ bool done() const { return pos >= end; }
  __device__ __forceinline__ int batch() const { return min(kBatch, min(end - pos, n_rt - rt)); }
  __device__ __forceinline__ void next(int nb) {
    pos += nb;
    rt += nb;
    if (rt == n_rt) {
      rt = 0;
      ++grp;
    }
  }
};

}  // namespace gemv_detail

// Launches the 4..16-token kernel on `grid` CTAs (defined in q4k_gemm_tokens.cu); CTAs of that kernel per SM.
int gemv_tokens_ctas_per_sm(int n_tok);
cudaError_t launch_gemv_tokens(const gemv_detail::GemvParams& P, int64_t grid, cudaStream_t st);

}  // namespace prima
