// Shared declarations of the CUDA sources: tiled weight layout, launch interfaces, small helpers.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>

namespace prima {

// ---------------------------------------------------------------------------------------------
// Tiled weight layout (what a Q4_K matrix looks like in HBM after loading)
//
// A "unit" is the 8 super-blocks found at the crossing of one row tile (8 consecutive rows) and one
// super-block column s (256 consecutive weights): 8 * 144 = 1152 bytes, the same bytes as the
// source blocks, rearranged so that one warp reads it with three 16-byte loads per lane:
//
//   bytes    0..127   headers: row g (0..7) at g*16: word0 = d | dmin << 16 (binary16 bits),
//                     words 1..3 = the sixteen 6-bit fields regrouped per lane quad position t:
//                     f_t = sc_t | sc_{t+4} << 6 | m_t << 12 | m_{t+4} << 18  (24 bits, t = 0..3)
//                     word1 = f_0 | (f_3 & 0xff) << 24, word2 = f_1 | (f_3 >> 8 & 0xff) << 24,
//                     word3 = f_2 | (f_3 >> 16) << 24
//   bytes  128..639   nibbles of sub-blocks 0..3: the 16-byte piece of (row g, sub-block t), its 32
//                     weights, sits at piece slot  4 g + (t ^ ((g >> 1) & 3))  (unit_piece_slot below)
//   bytes  640..1151  the same for sub-blocks 4..7 (piece of (row g, sub-block 4 + t))
// The exchange of pieces inside a row serves two readers at once: lane (g, t) of a warp reading its own
// piece (any eight consecutive lanes then cover eight different 16-byte bank groups), and a matrix load
// (ldmatrix) of the eight rows' pieces of ONE sub-block, which also wants eight different bank groups.
//
// Inside a 16-byte sub-block chunk, word w (0..3) holds weights 8w..8w+7, weight 8w+i in bits
// 4i..4i+3, so that (word & 0x0f0f0f0f) is four weights (8w, 8w+2, 8w+4, 8w+6) as unsigned bytes and
// ((word >> 4) & 0x0f0f0f0f) the other four: ready-made operands of the 4-way byte dot product.
//
// Units are stored column-major over the (row tile, super-block column) grid:
//   offset(s, rt) = (s * n_rt + rt) * 1152
// so that a warp that walks down the rows at a fixed column s -- which lets it keep its 256
// activations in registers -- streams one contiguous byte range.
// Rows are padded with zero blocks up to a multiple of 8.
// ---------------------------------------------------------------------------------------------
constexpr int kUnitBytes = 1152;
// Slot (of 16 bytes, inside a 512-byte nibble tile) of the piece of (row g, sub-block t of the tile's four).
__host__ __device__ constexpr int unit_piece_slot(int g, int t) { return 4 * g + (t ^ ((g >> 1) & 3)); }
constexpr int kUnitHdrBytes = 128;
constexpr int kRowsPerTile = 8;
constexpr int kBlockBytes = 144;
constexpr int kMaxTok = 16;        // tokens of a step of independent requests (one each)
constexpr int kMaxStepTok = 8;     // tokens of a step of one sequence (causal among themselves)
constexpr int kMaxStatBlocks = 256;
constexpr int kHeadDim = 128;

// In-situ timing of one launch (prima_profile_enable mode 2): t0 receives the earliest %globaltimer
// reading (ns) at which a CTA got past its dependency wait, t1 the latest at which a CTA finished.
// Intervals of consecutive kernels of a stream do not overlap (a kernel passes its wait only after its
// predecessor has completed), so their sum never exceeds the time of the step they belong to.
struct Stamp {
  unsigned long long* t0 = nullptr;   // device words, or null: not stamped
  unsigned long long* t1 = nullptr;
};

// Weights that a later kernel of the queue will stream, asked into L2 ahead of time by a kernel that leaves HBM idle
// (attention and the product after it, which reads what attention had fetched).  Nothing waits for these requests.
struct L2Ahead {
  const uint8_t* ptr[2] = {nullptr, nullptr};      // device, 16-byte aligned
  unsigned long long bytes[2] = {0, 0};            // multiples of 16
};

struct TiledMat {
  uint8_t* data = nullptr;   // device, n_sb * n_rt * 1152 bytes
  int64_t rows = 0;          // logical rows (of the fused matrix)
  int64_t cols = 0;
  int64_t n_rt = 0;          // row tiles = ceil(rows / 8)
  int64_t n_sb = 0;          // cols / 256
  size_t bytes() const { return static_cast<size_t>(n_sb) * n_rt * kUnitBytes; }
  int64_t mpad() const { return n_rt * kRowsPerTile; }
};

// Sums of squares of a vector, one per column group of the product that consumed it first:
// ssq[tok * kMaxStatBlocks + group].  rsqrt(sum over groups / width + eps) is the RMSNorm factor.
// Normalisation is *deferred*: a product with a normalised input multiplies by gain only and leaves
// partial sums that still lack the scalar factor; whoever consumes those partial sums applies it.
struct SumSq {
  float* data = nullptr;     // device, [kMaxTok][kMaxStatBlocks]
  int n_groups = 0;
  int64_t width = 0;         // length of the vector the sums belong to
  float eps = 0.f;
};

// ---- launch interfaces (definitions in the .cu files) ----------------------------------------
// Each returns the number of kernels it launched (for accounting) or a negative cudaError_t.

// Standard-layout dequantisation (bit-exact definition of the format).
int launch_dequant_std(const uint8_t* blocks, int64_t n_sb, float* out, cudaStream_t st);

// Re-tile `rows_src` rows of a standard-layout matrix into dst; source row r lands at fused row
// dst_row0 + r * dst_row_stride.
int launch_retile(const uint8_t* src, int64_t rows_src, int64_t n_sb, TiledMat dst, int64_t dst_row0,
                  int64_t dst_row_stride, cudaStream_t st);

// ---- fixed-point accumulators --------------------------------------------------------------------
// A product is computed as partial sums over groups of super-block columns by different CTAs.  The
// partial sums of one output element are added into a 64-bit fixed-point accumulator (two's
// complement, 32 fractional bits) with integer atomics: integer addition is associative, so the
// result does not depend on the order in which the CTAs arrive -- the bits are the same from run
// to run and under any split into windows -- and whoever consumes the product reads ONE word per
// element instead of one per group.  Range +-2^31, resolution 2^-32 per partial sum; a partial sum
// outside +-2^27 raises the device status word.  An accumulator array must be all zero when the
// product that adds into it starts; the kernels clear the arrays behind their readers.
using acc_t = unsigned long long;
constexpr float kAccScale = 4294967296.0f;                 // 2^32
constexpr float kAccInvScale = 2.3283064365386963e-10f;    // 2^-32
constexpr float kAccLimit = 134217728.0f;                  // 2^27

// Number of adjacent super-block columns one CTA of the GEMV works on (largest divisor of n_sb
// that is <= 8).
int gemv_group_size(int64_t n_sb);
bool gemv_uses_tensor_cores();

// acc[t * mpad + r] += sum over the weights of column group p of W[r][k] * xhat[t][k], for every
// group p.  A warp stages the 256 activations of its column in registers, finishing the producer's
// output on the way (GemvIn.kind):
//   kPlain    xhat = x
//   kResidual v = h_in + value(acc_in) (acc_in = the accumulators of the previous product, or null);
//             v is written to h_out (the new residual stream), its sum of squares over the group to
//             ssq_out, and xhat = v * gain (the RMSNorm scalar is left to the consumer of `acc`)
//   kSwiglu   xhat[k] = silu(G) * U with G, U = inv * the values of acc_in for fused rows 2k, 2k+1 of
//             the previous (gate/up) product, inv from ssq_in
// After its dependency wait the kernel also clears the accumulator arrays zero0 / zero1 (arrays
// whose last reader was the predecessor kernel or an earlier one).
//
// Order of the accumulators inside a token's mpad words (GemvIn.out_order of the producer): a
// consumer's lane owns 8 consecutive columns, and with the plain order its 16-byte loads would each
// touch a different 128-byte line.  The producer therefore stores in the order in which the
// consumer's warp reads, so that every load instruction of the warp covers 512 contiguous bytes:
//   kOrderRows      element r at r (read by the attention and output finishers)
//   kOrderResidual  for a kResidual consumer: inside every block of 256 rows, the pair of rows
//                   (2p, 2p+1) sits at pair position 32 (p % 4) + p / 4
//   kOrderSwiglu    for a kSwiglu consumer: inside every block of 512 fused rows (256 columns), the
//                   (gate, up) pair of column w sits at pair position 32 (w % 8) + w / 8
enum GemvKind { kPlain = 0, kResidual = 1, kSwiglu = 2 };
enum AccOrder { kOrderRows = 0, kOrderResidual = 1, kOrderSwiglu = 2 };
struct GemvIn {
  int kind = kPlain;
  const float* x = nullptr;        // kPlain: [n_tok][cols]
  const float* h_in = nullptr;     // kResidual: [n_tok][cols]
  float* h_out = nullptr;          // kResidual: [n_tok][cols], must not alias h_in
  const acc_t* acc_in = nullptr;   // kResidual (optional) / kSwiglu: [n_tok][mpad_in]
  int64_t mpad_in = 0;
  const float* gain = nullptr;     // kResidual: [cols]
  SumSq ssq_out;                   // kResidual: written (n_groups is set by the launcher)
  SumSq ssq_in;                    // kSwiglu: read
  int out_order = kOrderRows;      // order of the accumulators this product leaves (padded rows a multiple of 256 / 512 for kOrderResidual / kOrderSwiglu)
  acc_t* zero0 = nullptr;          // accumulator arrays to clear, with their lengths
  int64_t zero0_n = 0;
  acc_t* zero1 = nullptr;
  int64_t zero1_n = 0;
  int* status = nullptr;           // device word: bit 0 set if a bounded wait gave up, bit 1 if a partial sum was out of range
  uint32_t first_wait_polls = 0;   // 0: the ordinary limit; otherwise the poll limit of every warp's first wait + 1 (test hook)
  Stamp stamp;
  L2Ahead ahead;                   // requested by the CTAs once the predecessor kernel is done
};
int launch_gemv_partials(const TiledMat& w, GemvIn& in, int n_tok, acc_t* acc, int sm_count, cudaStream_t st);

// y[t][r] = scale_t * value(acc[t * mpad + r]), scale_t = the RMSNorm factor from ssq when
// ssq.data != nullptr, else 1; every accumulator is cleared after it has been read.
int launch_finish_acc(acc_t* acc, int64_t mpad, int64_t rows, int n_tok, float* y, const SumSq& ssq, cudaStream_t st);
// out[t][r] = h[t][r] + value of row r's accumulator, stored in kOrderResidual (the residual stream
// leaving a window); clears acc behind the read and the array zero0.
int launch_finish_residual(acc_t* acc, int64_t mpad, int64_t rows, int n_tok, const float* h, float* out, acc_t* zero0, int64_t zero0_n,
                           cudaStream_t st);

// y[t][r] = scale_t * sum over the n_parts partial sums (ascending), scale_t = the RMSNorm factor
// from ssq when ssq.data != nullptr, else 1.
int launch_finish_plain(const float* part, int64_t n_parts, int64_t mpad, int64_t rows, int n_tok, float* y, const SumSq& ssq,
                        cudaStream_t st);
// cos/sin table for positions pos..pos+n_tok-1: tab[t][i] = (cos, sin)(pos_t * theta^(-2i/128)),
// evaluated in double precision.
int launch_rope_table(float2* tab, int pos, int n_tok, float theta, cudaStream_t st);

// Grouped-query decode attention over the fp16 cache, split along the context, merged by
// log-sum-exp.  The queries, and the new keys and values, are taken from the accumulators of the
// fused QKV product (rows [q heads | k heads | v heads] x 128): scaled by the RMSNorm factor
// from ssq, rotated with the cos/sin table; the new K and V are appended to the cache (binary16) at
// positions pos + t by the CTAs whose chunk holds them.  Cache layout [G][capacity][128].
// o: [n_tok][H*128] fp32.
struct AttnScratch {
  float* o_part;    // [n_tok*H][n_chunks][128]
  float2* ml_part;  // [n_tok*H][n_chunks]  (running max, running sum)
  int max_chunks;
  int* tickets;     // [kMaxTok][G], all zero between launches (see attn_one_kernel)
  Stamp stamp;      // of the next attention launch (both kernels share it)
  L2Ahead ahead;    // requested by the CTAs of the next attention launch as they start
  int* status = nullptr;      // the context's status word (range-checked build: bit 2)
};
// Several independent requests in one launch: token t of the step belongs to a request with its own
// cache (k[t], v[t]) and position pos[t]; rows, statistics, rotary table and outputs of token t are
// the t-th slices of the arrays that launch_attention takes.
struct AttnSeqs {
  __half* k[kMaxTok];
  __half* v[kMaxTok];
  int pos[kMaxTok];
  int n = 0;
};
// stable_below: cache entries at positions below it may be read before the kernel's dependency wait (see attention.cu).
int launch_attention_seqs(const acc_t* acc_qkv, int64_t mpad, const SumSq& ssq, const float2* rope_tab, int rope_mode, const AttnSeqs& seqs,
                          int stable_below, int kv_capacity, int n_q_heads, int n_kv_heads, const AttnScratch& scr, float* o, int sm_count,
                          cudaStream_t st);
int launch_attention(const acc_t* acc_qkv, int64_t mpad, const SumSq& ssq, const float2* rope_tab, int rope_mode,
                     __half* k_cache, __half* v_cache, int kv_capacity, int n_q_heads, int n_kv_heads, int pos, int stable_below, int n_tok,
                     const AttnScratch& scr, float* o, int sm_count, cudaStream_t st);
int attention_chunk_len();

// Embedding lookup from a standard-layout table, and greedy argmax.
int launch_embed(const uint8_t* table_std, int64_t n_sb_per_row, const int32_t* dev_tokens, int n_tok, float* out,
                 cudaStream_t st);
int launch_argmax(const float* logits, int64_t vocab, int n_tok, float* scratch_val, int32_t* scratch_idx,
                  int32_t* dev_out, cudaStream_t st);
constexpr int kArgmaxBlocks = 128;

inline int cuda_rc(cudaError_t e) { return e == cudaSuccess ? 0 : -static_cast<int>(e); }

// Function attributes (dynamic shared memory size, carve-out) are per device and do not change:
// each launcher sets them the first time it runs on a device, not at every launch (a call costs the
// host more than a microsecond, and with six launches per layer the host must stay ahead of the GPU).
// `done` is the launcher's own table of kMaxDevices flags; returns true when the caller must set them.
constexpr int kMaxDevices = 64;
inline bool first_launch_on_device(bool (&done)[kMaxDevices], int* device_out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    *device_out = -1;
    return true;
  }
  *device_out = dev;
  return !done[dev];
}

// ---- programmatic dependent launch -------------------------------------------------------------
// Every kernel of the forward pass is launched with programmatic stream serialisation: it may
// start while its predecessor in the stream is still running.  A kernel calls pdl_trigger() first
// thing (its successor may then be scheduled as soon as resources free up) and pdl_wait() before
// it reads anything a predecessor wrote or writes anything a predecessor may still read; what it
// does before pdl_wait() (set-up, prefetching immutable weights) overlaps the predecessor's tail.
#ifdef __CUDACC__
__device__ __forceinline__ float acc_value(acc_t a) { return static_cast<float>(static_cast<long long>(a)) * kAccInvScale; }
// Position of row r (fused row for kOrderSwiglu) inside a token's accumulators.
__device__ __forceinline__ int64_t acc_position(int order, int64_t r) {
  if (order == kOrderResidual) {
    const int64_t p = (r & 255) >> 1;
    return (r & ~int64_t(255)) + 2 * (32 * (p & 3) + (p >> 2)) + (r & 1);
  }
  if (order == kOrderSwiglu) {
    const int64_t w = (r >> 1) & 255;
    return (r & ~int64_t(511)) + 2 * (32 * (w & 7) + (w >> 3)) + (r & 1);
  }
  return r;
}
__device__ __forceinline__ acc_t acc_from(float v) { return static_cast<acc_t>(__float2ll_rn(v * kAccScale)); }

__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Called by every thread of the CTA: right after the dependency wait / at the very end.
__device__ __forceinline__ void stamp_begin(const Stamp& s) {
  if (s.t0 && threadIdx.x == 0) atomicMin(s.t0, global_ns());
}
__device__ __forceinline__ void stamp_end(const Stamp& s) {
  if (s.t1) {
    __syncthreads();
    if (threadIdx.x == 0) atomicMax(s.t1, global_ns());
  }
}

// Called by one thread of each CTA: CTA `cta` of `n_ctas` asks for every n_ctas-th piece of 16 KiB of both spans.
__device__ __forceinline__ void l2_ahead(const L2Ahead& a, unsigned cta, unsigned n_ctas) {
  constexpr unsigned long long kPiece = 16384;
#pragma unroll
  for (int s = 0; s < 2; ++s) {
    const unsigned long long bytes = a.bytes[s];
    for (unsigned long long off = cta * kPiece; off < bytes; off += n_ctas * kPiece) {
      const unsigned size = static_cast<unsigned>(min(kPiece, bytes - off));
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(a.ptr[s] + off), "r"(size) : "memory");
    }
  }
}

// Range-checked build (-DPRIMA_BOUNDS): an index outside its array raises bit 2 of the status word and the access is
// skipped; nothing traps.  In the ordinary build the check costs nothing.
#ifdef PRIMA_BOUNDS
__device__ __forceinline__ bool in_range(bool ok, int* status) {
  if (!ok && status) atomicOr(status, 4);
  return ok;
}
#else
__device__ __forceinline__ bool in_range(bool, int*) { return true; }
#endif

__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

}  // namespace prima
