/*
 * prima.h -- C ABI of the B200 layer-window decoder for Q4_K models.
 *
 * The library executes the per-token forward pass of a contiguous WINDOW of transformer layers,
 * the unit of work one device performs per round in pipelined-ring parallelism (paper Section 3.1,
 * "Pipelined-ring parallelism (PRP) with prefetching"; Appendix A.12, "Mmap- and prefetch-based
 * PRP": an 80-layer model on 4 devices with window 10 runs layers 1-10/11-20/21-30/31-40 in round
 * one and 41-50/.../71-80 in round two).  What enters and leaves a window is the hidden state,
 * e fp32 values per token, 4e bytes (Appendix A.3, network communication latency and device copy
 * time).  Each layer keeps its own fp16 KV cache, which grows by 2(h_k e_k + h_v e_v) bytes per
 * token and is read in full, 2(h_k e_k + h_v e_v) n_kv bytes, at every step (Appendix A.3, KV
 * cache copy time and device loading time).  The input layer is a lookup table and the output
 * layer produces the logits (Appendix A.3, computation latency).  Draft tokens of speculative
 * decoding are verified by one batched pass of n_tok tokens (Appendix A.9 "Run Prima.cpp with
 * Speculative Decoding"; Appendix A.12 "Speculative decoding").
 *
 * Weights are stored in the 4.5-bit Q4_K block format the paper names (Section 4; Appendix A.3,
 * the set Q of quantisation types).  The paper does not print the bit layout; this library
 * defines it as follows.  A super-block covers 256 consecutive weights of one row and is 144
 * bytes, little endian:
 *     bytes 0-1    d     IEEE binary16
 *     bytes 2-3    dmin  IEEE binary16
 *     bytes 4-15   s[0..11]: eight 6-bit scales sc_j and eight 6-bit mins m_j, j = 0..7
 *                    j < 4 : sc_j = s[j] & 63                      m_j = s[j+4] & 63
 *                    j >= 4: sc_j = (s[j+4] & 15) | (s[j-4] >> 6) << 4
 *                            m_j  = (s[j+4] >> 4) | (s[j]   >> 6) << 4
 *     bytes 16-143 qs[0..127]: byte qs[32p+i] (p = 0..3, i = 0..31) holds weight 64p+i in its low
 *                  nibble and weight 64p+32+i in its high nibble
 *     weight k = d * sc_j * q_k - dmin * m_j,  j = k / 32.
 * A matrix W[rows x cols] is rows * (cols/256) super-blocks, row-major; cols % 256 == 0.
 *
 * Conventions.  Every function returns PRIMA_OK (0) or a negative error code; nothing throws,
 * aborts or traps the GPU.  "dev" pointers are CUDA device pointers on the context's device,
 * "host" pointers are ordinary host memory.  All work is queued on the context's stream; calls
 * return without waiting unless stated.  The library owns the memory it allocates (weights in its
 * own tiled layout, KV cache, scratch); the caller owns every buffer it passes in.
 */
#ifndef PRIMA_H
#define PRIMA_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PRIMA_OK 0
#define PRIMA_ERR_ARG (-1)        /* bad argument; nothing was modified or launched            */
#define PRIMA_ERR_STATE (-2)      /* a needed tensor has not been loaded                        */
#define PRIMA_ERR_CUDA (-3)       /* a CUDA call failed; see prima_last_error                   */
#define PRIMA_ERR_NOMEM (-4)      /* device allocation failed                                   */
#define PRIMA_ERR_DEVICE (-5)     /* a kernel reported a failed self-check (status word)        */

#define PRIMA_Q4K_BLOCK_BYTES 144
#define PRIMA_Q4K_BLOCK_WEIGHTS 256
#define PRIMA_MAX_N_TOK 8   /* tokens of one sequence per step (prima_forward_window)            */
#define PRIMA_MAX_N_SEQ 16  /* requests per step (prima_forward_window_seqs), columns of a product  */

/* tensor ids for prima_load_q4k_weights */
enum {
  PRIMA_ATTN_NORM = 0, /* fp32 [hidden]                 per layer */
  PRIMA_WQ = 1,        /* Q4_K [n_q_heads*head_dim x hidden]       */
  PRIMA_WK = 2,        /* Q4_K [n_kv_heads*head_dim x hidden]      */
  PRIMA_WV = 3,        /* Q4_K [n_kv_heads*head_dim x hidden]      */
  PRIMA_WO = 4,        /* Q4_K [hidden x n_q_heads*head_dim]       */
  PRIMA_FFN_NORM = 5,  /* fp32 [hidden]                            */
  PRIMA_W_GATE = 6,    /* Q4_K [ffn x hidden]                      */
  PRIMA_W_UP = 7,      /* Q4_K [ffn x hidden]                      */
  PRIMA_W_DOWN = 8,    /* Q4_K [hidden x ffn]                      */
  PRIMA_OUT_NORM = 9,  /* fp32 [hidden]                 layer = -1 */
  PRIMA_W_HEAD = 10,   /* Q4_K [vocab x hidden]         layer = -1 */
  PRIMA_TOK_EMBD = 11  /* Q4_K [vocab x hidden]         layer = -1 */
};

typedef struct prima_ctx prima_ctx; /* opaque, owned by the library */

/* Model shape; plain data, copied by prima_ctx_create. */
typedef struct {
  int32_t n_layers;
  int32_t hidden;      /* e; multiple of 256                                                    */
  int32_t n_q_heads;   /* H                                                                     */
  int32_t n_kv_heads;  /* G; H % G == 0, H / G <= 8                                             */
  int32_t head_dim;    /* must be 128                                                           */
  int32_t ffn;         /* F; multiple of 256                                                    */
  int32_t vocab;       /* V                                                                     */
  int32_t kv_capacity; /* positions per layer in the fp16 KV cache                              */
  int32_t max_n_tok;   /* largest number of tokens of a step, 1..PRIMA_MAX_N_SEQ (prima_forward_window
                          itself takes at most PRIMA_MAX_N_TOK)                                 */
  float rms_eps;
  float rope_theta;
  int32_t rope_mode;   /* 0: rotate pairs (i, i + head_dim/2); 1: pairs (2i, 2i+1)              */
  int32_t device;      /* CUDA ordinal                                                          */
} prima_model_config;

/* Create a context on cfg->device.  `cuda_stream` is a cudaStream_t (or NULL for the default
 * stream) on which all work of this context is queued.  Allocates scratch buffers; the KV cache
 * of a layer and its weights are allocated when first loaded.  Errors: PRIMA_ERR_ARG for an
 * inconsistent shape, PRIMA_ERR_NOMEM / PRIMA_ERR_CUDA otherwise; *out is NULL on error. */
int prima_ctx_create(const prima_model_config* cfg, void* cuda_stream, prima_ctx** out);

/* Wait for the stream, then free every device buffer the context allocated. */
int prima_ctx_destroy(prima_ctx* ctx);

/* Load one tensor (the paper's model is a file of such tensors; Section 3.1).  Q4_K tensors:
 * `data` holds rows*(cols/256)*144 bytes in the layout above; norm tensors: fp32[cols], rows = 1.
 * `data` may be host or device memory; the library copies it into its own layout before
 * returning (this call synchronises the stream), the caller may free `data` afterwards.
 * layer = -1 for PRIMA_OUT_NORM / PRIMA_W_HEAD / PRIMA_TOK_EMBD.  A shape that disagrees with the
 * config, cols % 256 != 0, a wrong nbytes, an unknown id or a layer out of range return
 * PRIMA_ERR_ARG and leave the context unchanged. */
int prima_load_q4k_weights(prima_ctx* ctx, int layer, int tensor_id, const void* data,
                           int64_t rows, int64_t cols, int64_t nbytes);

/* Run layers [layer_begin, layer_end) (one window of the ring schedule) on n_tok tokens at cache
 * positions pos .. pos+n_tok-1.  hidden_in / hidden_out: dev, fp32, [n_tok x hidden] row-major,
 * may alias.  Per layer: RMSNorm, Q/K/V projections, rotary embedding, append of K and V to the
 * fp16 cache, grouped-query attention over positions 0..pos+t for token t (causal inside the
 * step), output projection and residual, RMSNorm, SwiGLU feed-forward and residual.  Windows of
 * one step must be issued in ascending layer order; any split of the layer range into windows
 * gives bit-identical results.  Errors (no launch): a layer of the range is not fully loaded
 * (PRIMA_ERR_STATE); bad range, pos < 0, pos + n_tok > kv_capacity, n_tok outside 1..max_n_tok,
 * NULL pointers (PRIMA_ERR_ARG).
 * Range: the products are summed in 64-bit fixed point with 32 fractional bits (order-independent,
 * hence the bit-identical results); a partial sum of a projection beyond +-2^27 (1.3e8) raises the
 * status word, which prima_sync reports as PRIMA_ERR_DEVICE (the outputs of that step are then
 * invalid).  Contributions below 2^-33 in absolute value are rounded away. */
int prima_forward_window(prima_ctx* ctx, int layer_begin, int layer_end, const float* hidden_in,
                         float* hidden_out, int pos, int n_tok);

/* One step of several independent requests (the paper's serving mode: Appendix A.11 "Ablation
 * Study on Multi-Request Workloads" / A.12, requests merged per token step, each with its own KV cache).  Token t belongs to
 * sequence seq[t] (0..63, each at most once per step) and sits at position pos[t] of that sequence's
 * cache; the projections run over all n_seq tokens together (the weights are read once), attention
 * runs per token over its own sequence's cache, to which the token's K and V are appended.
 * Sequence 0 is the cache that prima_forward_window and prima_kv_load use; the cache of another
 * sequence is allocated (zero-filled) the first time it is named.  seq, pos: host int32[n_seq];
 * hidden_in / hidden_out: dev fp32 [n_seq x hidden].  Errors as prima_forward_window, plus
 * PRIMA_ERR_ARG for a sequence id out of range or named twice and PRIMA_ERR_NOMEM if a cache cannot
 * be allocated. */
int prima_forward_window_seqs(prima_ctx* ctx, int layer_begin, int layer_end, const float* hidden_in,
                              float* hidden_out, const int32_t* seq, const int32_t* pos, int n_seq);

/* Output layer: logits[t][v] = W_head . RMSNorm(hidden[t]; out_norm).  hidden: dev fp32
 * [n_tok x hidden]; logits: dev fp32 [n_tok x vocab]. */
int prima_logits(prima_ctx* ctx, const float* hidden, int n_tok, float* logits);

/* Input layer (lookup table): hidden_out[t] = dequantised row tokens[t] of PRIMA_TOK_EMBD.
 * tokens: host int32[n_tok]; hidden_out: dev fp32 [n_tok x hidden]. */
int prima_embed(prima_ctx* ctx, const int32_t* tokens, int n_tok, float* hidden_out);

/* Greedy choice per token: index of the largest logit, lowest index on ties.  logits: dev fp32
 * [n_tok x vocab]; tokens_out: host int32[n_tok].  Waits for the result. */
int prima_argmax(prima_ctx* ctx, const float* logits, int n_tok, int32_t* tokens_out);

/* Write / read fp16 cache entries of one layer.  k, v: host, [n_pos][n_kv_heads][head_dim]
 * binary16 bit patterns.  Both calls synchronise.  Used to prefill a context and by tests. */
int prima_kv_load(prima_ctx* ctx, int layer, int pos_begin, int n_pos, const uint16_t* k, const uint16_t* v);
int prima_kv_read(prima_ctx* ctx, int layer, int pos_begin, int n_pos, uint16_t* k, uint16_t* v);
/* The same for the cache of sequence `seq` (0..63; sequence 0 is the cache of the calls above). */
int prima_kv_load_seq(prima_ctx* ctx, int seq, int layer, int pos_begin, int n_pos, const uint16_t* k, const uint16_t* v);
int prima_kv_read_seq(prima_ctx* ctx, int seq, int layer, int pos_begin, int n_pos, uint16_t* k, uint16_t* v);

/* Wait for all queued work; returns PRIMA_ERR_DEVICE if a kernel raised the status word (a
 * partial sum outside the accumulator range, a bounded wait inside a kernel that gave up, or, in the
 * library built with -DPRIMA_BOUNDS, an index outside its array: that access is skipped) and
 * PRIMA_ERR_CUDA if the stream reports an error.  A raised status word is reported once; the
 * outputs of the steps queued since the previous prima_sync are then invalid, and before it returns
 * prima_sync clears the status word and the library's internal accumulators, so the context can go
 * on with the next step (the KV cache keeps whatever the failed step appended: re-run the step
 * at the same positions, which overwrites those entries). */
int prima_sync(prima_ctx* ctx);

/* Failures of prima_forward_window / prima_forward_window_seqs / prima_logits:
 *   - argument and state errors are found before anything is queued or allocated;
 *   - PRIMA_ERR_NOMEM of prima_forward_window_seqs (a sequence's cache could not be allocated) is
 *     also returned before anything is queued: the caches of every (layer, sequence) pair of the
 *     window are allocated first, the launches follow;
 *   - PRIMA_ERR_CUDA from a launch in the middle of a window: the kernels queued before it still
 *     run, hidden_out is not valid, and the library queues the clearing of its accumulators behind
 *     them, so a later call computes from a clean state. */

/* Options of a context.  PRIMA_OPT_FIRST_WAIT_POLLS (for tests of the failure path): how many
 * times the first wait of every warp of the streaming kernels polls for its first batch of weights
 * before it gives up (0: gives up at once); -1 restores the ordinary limit of 2^24 polls.  A wait
 * that gives up raises the status word (see prima_sync); the kernel still waits, with the
 * ordinary limit, for every copy it requested before it returns.
 * PRIMA_OPT_FAIL_AFTER_LAUNCHES (for tests of the failure path, host side only): after `value` more
 * launch steps of this context the next one is refused with PRIMA_ERR_CUDA as if the runtime had
 * rejected it (nothing is sent to the GPU for it), once; -1 switches the injection off. */
#define PRIMA_OPT_FIRST_WAIT_POLLS 1
#define PRIMA_OPT_FAIL_AFTER_LAUNCHES 2

/* A model larger than the device's memory (the paper's case: Section 3.1, "Pipelined-ring parallelism (PRP) with
 * prefetching"; Appendix A.1-A.2: the weights of the windows that do not fit are (re)loaded while other work
 * runs, so that loading overlaps with computing).  Here the slow tier is pinned host memory instead of a disk:
 *   PRIMA_OPT_RESIDENT_LAYERS  the first `value` layers keep their matrices on the device; the matrices of the
 *       layers from `value` on live in pinned host memory (in the library's tiled layout) and are streamed to the
 *       device every time they are needed; -1 or n_layers: everything resident (default).
 *   PRIMA_OPT_STREAM_SLOTS     number of device buffers, each holding one streamed layer (2..16, default 2).
 * Both must be set before the first layer matrix is loaded.  The matrices of a streamed layer must be loaded
 * layer by layer (all seven of one layer before those of the next streamed layer; PRIMA_ERR_STATE otherwise).
 * prima_forward_window then waits, on the context's stream, only for the copy of the layer it is about to run
 * (one cudaMemcpyAsync per matrix on a second stream, ordered by events), and queues the copies of the streamed
 * layers that come next in decoding order (cyclically: after the last layer comes the first streamed layer of
 * the next token), as many as there are other slots, so that they stream in underneath the computation.  KV
 * caches, norm gains and the input / output layers stay on the device.  Results are bit-identical to those of a
 * fully resident context.  prima_stream_stats: bytes copied host-to-device for streamed layers since the context
 * was created, and the summed duration of those copies in milliseconds (waits for the copy stream). */
#define PRIMA_OPT_RESIDENT_LAYERS 3
#define PRIMA_OPT_STREAM_SLOTS 4
/* PRIMA_OPT_L2_AHEAD_BYTES, PRIMA_OPT_L2_AHEAD_O_BYTES: attention reads little and leaves HBM idle, and so does the
 * short O product (Section 4's footnote: decoding is bound by the memory stream, so every idle stretch of it is
 * lost time).  In a step of one token the attention kernel of a layer therefore asks for the first `value` bytes
 * of the gate/up matrix, the long stream that comes next, into L2, with requests nothing waits for, and the O
 * product for the PRIMA_OPT_L2_AHEAD_O_BYTES that follow them.  -1 (default): a sixteenth of the matrix each;
 * 0 switches one off; otherwise a multiple of 16 up to 2^30.  Results do not depend on them.  May be set at any
 * time between steps. */
#define PRIMA_OPT_L2_AHEAD_BYTES 5
#define PRIMA_OPT_L2_AHEAD_O_BYTES 6
int prima_ctx_set_option(prima_ctx* ctx, int option, int64_t value);
int prima_stream_stats(prima_ctx* ctx, int64_t* bytes_copied, double* copy_ms);

/* Text of the most recent error of this context (never NULL; "" if none).  With ctx == NULL,
 * the most recent error of a context-free call on this thread. */
const char* prima_last_error(prima_ctx* ctx);

/* Number of kernels this context has launched since it was created (for accounting). */
int64_t prima_launch_count(prima_ctx* ctx);

/* Device-side timing by kernel class, for measurement runs (the counterpart of the paper's device
 * profiler, which measures how fast weights and KV cache reach the cores: Appendix A.3, device
 * loading time).  enable(ctx, mode) discards what was recorded and selects
 *   mode 0: off;
 *   mode 1: every launch of the listed classes is bracketed by a pair of CUDA events on the context's
 *           stream.  This serialises the launches (a kernel no longer overlaps its predecessor's
 *           tail), so it times each kernel in isolation and perturbs the step;
 *   mode 2: every kernel of the listed classes stamps the GPU's nanosecond timer itself: the earliest
 *           moment a CTA got past its wait for the predecessor kernel, and the latest moment a CTA
 *           finished.  The launch sequence is unchanged, so these are the kernels' times inside the
 *           running step; intervals of consecutive kernels do not overlap, their sum is at most the
 *           step time.  Room for 32,768 launches between two calls of enable.
 * read waits for the stream and returns, for one class, the summed time in milliseconds, the number
 * of kernel launches and the algorithmic bytes they had to move (Q4_K weight bytes of the matrices,
 * or K and V bytes of the attended positions). */
#define PRIMA_PROF_GEMV 0
#define PRIMA_PROF_ATTENTION 1
/* mode 2 only: the products of one kind (a subset of PRIMA_PROF_GEMV) */
#define PRIMA_PROF_GEMV_QKV 16
#define PRIMA_PROF_GEMV_O 17
#define PRIMA_PROF_GEMV_GATE_UP 18
#define PRIMA_PROF_GEMV_DOWN 19
#define PRIMA_PROF_GEMV_HEAD 20
int prima_profile_enable(prima_ctx* ctx, int mode);
int prima_profile_read(prima_ctx* ctx, int klass, double* ms_total, int64_t* launches, int64_t* algo_bytes);

/* ---- context-free exports of the two primitives (tests and micro-benchmarks) ---------------- */

/* Dequantise n_superblocks blocks (dev, standard 144-byte layout) to fp32 (dev, 256 per block).
 * The result is the exact value d*sc*q - dmin*m rounded once to binary32.  `stream` is a
 * cudaStream_t or NULL. */
int prima_dequant_q4k(const void* dev_blocks, int64_t n_superblocks, float* dev_out, void* stream);

/* y[c][r] = sum_k W[r][k] x[c][k] for c < n_cols (1..16).  dev_w: standard layout; dev_x: fp32
 * [n_cols x cols]; dev_y: fp32 [n_cols x rows].  Allocates and frees its own temporary buffers
 * (tiled copy of W and scratch) and waits for completion; meant for testing single projections.
 * Returns PRIMA_ERR_DEVICE if a partial sum left the accumulator range (see prima_forward_window).
 * For timing, use prima_gemv_plan_* below. */
int prima_gemv_q4k(const void* dev_w, int64_t rows, int64_t cols, const float* dev_x, int n_cols,
                   float* dev_y, void* stream);

/* A resident, tiled copy of one matrix for repeated products (what a loaded layer tensor is
 * inside a context).  create copies and re-tiles dev_w (synchronises); run queues one product on
 * `stream` with no allocation and no synchronisation; destroy frees. */
typedef struct prima_gemv_plan prima_gemv_plan;
int prima_gemv_plan_create(const void* dev_w, int64_t rows, int64_t cols, int max_n_cols, prima_gemv_plan** out);
int prima_gemv_plan_run(prima_gemv_plan* plan, const float* dev_x, int n_cols, float* dev_y, void* stream);
int prima_gemv_plan_destroy(prima_gemv_plan* plan);

/* ---- the other weight formats of the paper's set Q (Appendix A.3, computation latency: Q = {Q4_K, Q5_K, Q6_K,
 * Q8_0, FP16, FP32}; checkpoints called "Q4K" mix them).  The paper prints none of the layouts; these are the
 * public ones of the file format its system reads:
 *   PRIMA_FMT_Q8_0  34-byte block of 32 weights: binary16 d, 32 signed bytes q;  weight = d * q
 *   PRIMA_FMT_Q6_K  210-byte super-block of 256 weights: ql[128], qh[64], signed byte scales sc[16], binary16 d;
 *                   weight k = d * sc[k/16] * (v_k - 32); with k = 128 n + 32 i + l the low four bits of v_k are in
 *                   byte ql[64 n + 32 (i & 1) + l] (low nibble for i < 2, high nibble otherwise) and its high two
 *                   bits are bits 2i, 2i+1 of byte qh[32 n + l]
 *   PRIMA_FMT_F16   binary16 values
 *   PRIMA_FMT_Q4_K  the 144-byte super-block described at the top (the calls below forward to the _q4k calls)
 * Matrices are row-major, cols a multiple of 256.  prima_dequant_fmt: n_blocks blocks (dev) -> fp32 (dev), the exact
 * value (no rounding is needed: it fits binary32).  prima_gemv_fmt: y[c][r] = sum_k W[r][k] x[c][k], 1 <= n_cols <= 4;
 * dev_w in its standard layout, read in place (nothing is allocated or re-tiled), at an even address.  Shared
 * memory must hold the activations of all columns (4 bytes a value for FP16 matrices; for the block formats 16-bit
 * integers with one fp32 step per 32 values, as in the Q4_K path, 3 bytes a value with cols rounded up to 2048) plus
 * two rows of the matrix (FP16) or the warps' copy rings (block formats: 35 KiB at least) within 200 KiB
 * (PRIMA_ERR_ARG otherwise, with a message in prima_fmt_last_error).  dev_w must lie in an allocation whose size is
 * a multiple of 16 bytes, as every cudaMalloc allocation is: rows are fetched in 16-byte pieces from the boundary at
 * or below their first byte to the boundary at or above their last.  Per row |y - y_ref| <= 1e-3 * sum |w x|
 * (activation step <= 2^-15 of a block's largest value, exact integer sums per group, fp32 accumulation over
 * groups).  Queued on `stream`, no waiting. */
#define PRIMA_FMT_Q4_K 0
#define PRIMA_FMT_Q6_K 1
#define PRIMA_FMT_Q8_0 2
#define PRIMA_FMT_F16 3
int prima_fmt_block_weights(int fmt);   /* weights per block (0: unknown format) */
int prima_fmt_block_bytes(int fmt);     /* bytes per block */
int prima_dequant_fmt(int fmt, const void* dev_blocks, int64_t n_blocks, float* dev_out, void* stream);
int prima_gemv_fmt(int fmt, const void* dev_w, int64_t rows, int64_t cols, const float* dev_x, int n_cols,
                   float* dev_y, void* stream);
const char* prima_fmt_last_error(void);

/* The same product as prima_gemv_q4k for callers that cannot allocate device memory: programs that
 * gave all of the GPU's memory to their own arena at start-up, or latency-critical loops in which
 * cudaMalloc / cudaFree (which may stall the device, and may fail late) are not allowed.  The paper
 * has no counterpart of this call; it exists only for such callers.
 *   dev_w: standard 144-byte block layout, rows*(cols/256) blocks; dev_x: fp32 [n_cols x cols];
 *   dev_y: fp32 [n_cols x rows]; all device memory owned by the caller; stream: cudaStream_t or NULL.
 * Nothing is allocated or freed, here or in anything it calls: the partial sums live in a 16 MiB
 * array built into the library (each GPU that loads the library holds it until exit).  Limit:
 * rows * (cols/256) * n_cols <= 4,194,304; larger products return PRIMA_ERR_ARG with a message
 * that says so.  The first call on a device looks up the array's device address and remembers it
 * for that device ordinal; make that first call before any stream capture begins, and with the
 * CUDA context current that all later calls will use: the address belongs to that context (the
 * runtime's primary context, normally), so after cudaDeviceReset, or under a different driver-API
 * context on the same device, the remembered address is stale and this call must not be used.  The call queues its kernels on `stream` and
 * returns without waiting.  All calls on a device share the array: calls whose kernels may
 * overlap on the GPU (different streams without ordering) corrupt each other; calls ordered on a
 * stream, or by events, are safe, and nothing has to be cleared between them.
 * prima_gemv_q4k_noalloc_error returns this thread's last message from this call ("" if none). */
int prima_gemv_q4k_noalloc(const void* dev_w, int64_t rows, int64_t cols, const float* dev_x, int n_cols,
                           float* dev_y, void* stream);
const char* prima_gemv_q4k_noalloc_error(void);

#ifdef __cplusplus
}
#endif
#endif /* PRIMA_H */
