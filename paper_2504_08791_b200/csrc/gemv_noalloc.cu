// prima_gemv_q4k_noalloc: the Q4_K matrix-vector product for callers that must not allocate.
//
// Who needs this.  Some programs hand the whole GPU to their own memory manager when they start
// (a serving engine with a pre-sized arena, a runtime that forbids driver allocations once it is
// up) or sit in a latency-critical loop where cudaMalloc / cudaFree -- which may stall the device
// and can fail late -- are not acceptable.  prima_gemv_q4k allocates a re-tiled copy of the matrix
// and a partial-sum buffer on every call; this entry point allocates nothing.  It reads the matrix
// in the standard 144-byte block layout directly and keeps its partial sums in a fixed array that
// is part of the library image, so every GPU that loads the library carries that array (16 MiB)
// until the process exits.
//
// How it computes.  Same decomposition as the streaming kernel: one partial sum per (row,
// super-block column, input column), written to scratch, then summed over the super-block columns
// in ascending order by the ordinary finishing kernel.  The partial itself is computed here in
// fp32 on the dequantised weights (one warp per row and super-block column).
//
// Sharing.  All calls on a device use the same scratch array.  Every partial that a call reads was
// written by that same call, so nothing needs clearing between calls; but two calls whose kernels
// overlap on the GPU (different streams, no ordering between them) overwrite each other's partial
// sums and give wrong results.  Keep calls on one device ordered.
//
// Contexts.  The array's device address is looked up once per device ordinal, on the first call, and
// remembered.  That address belongs to the CUDA context that was current on the device at that
// moment (normally the runtime's primary context).  A caller that later resets the device
// (cudaDeviceReset) or makes a different driver-API context current on the same device must not
// use this entry point afterwards: the remembered address would be stale.
#include <cstdio>
#include <mutex>

#include "../../include/prima.h"
#include "common.cuh"

namespace {

constexpr int64_t kScratchFloats = int64_t(4) << 20;   // 4 Mi floats = 16 MiB
static __device__ __align__(256) float g_noalloc_scratch[kScratchFloats];

constexpr int kMaxDevices = 64;
float* g_scratch_ptr[kMaxDevices] = {};   // device address of the array, per device ordinal
std::mutex g_setup_mutex;
thread_local char g_noalloc_error[256] = "";

// One warp per (row, super-block column); lane l owns bytes 4l..4l+3 of the 128 nibble bytes, i.e.
// weights 64p+i..64p+i+3 (low nibbles) and 64p+32+i..+3 (high nibbles) with p = l / 8, i = 4 (l % 8).
__global__ void gemv_std_partials_kernel(const uint8_t* __restrict__ w, int64_t rows, int64_t n_sb, const float* __restrict__ x,
                                         int n_cols, float* __restrict__ part) {
  const int lane = threadIdx.x & 31;
  const int64_t unit = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (unit >= rows * n_sb) return;
  const int64_t row = unit / n_sb, s = unit % n_sb;
  const uint8_t* sb = w + unit * prima::kBlockBytes;
  const float d = __half2float(__ushort_as_half(static_cast<unsigned short>(sb[0] | (sb[1] << 8))));
  const float dmin = __half2float(__ushort_as_half(static_cast<unsigned short>(sb[2] | (sb[3] << 8))));
  const uint8_t* sc = sb + 4;
  const int p = lane >> 3, i = (lane & 7) * 4;
  const int jl = 2 * p, jh = 2 * p + 1;
  uint32_t sc_l, m_l, sc_h, m_h;
  if (jl < 4) { sc_l = sc[jl] & 63u; m_l = sc[jl + 4] & 63u; }
  else { sc_l = (sc[jl + 4] & 15u) | ((sc[jl - 4] >> 6) << 4); m_l = (sc[jl + 4] >> 4) | ((sc[jl] >> 6) << 4); }
  if (jh < 4) { sc_h = sc[jh] & 63u; m_h = sc[jh + 4] & 63u; }
  else { sc_h = (sc[jh + 4] & 15u) | ((sc[jh - 4] >> 6) << 4); m_h = (sc[jh + 4] >> 4) | ((sc[jh] >> 6) << 4); }
  const float a_l = d * static_cast<float>(sc_l), b_l = dmin * static_cast<float>(m_l);
  const float a_h = d * static_cast<float>(sc_h), b_h = dmin * static_cast<float>(m_h);
  float wl[4], wh[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const uint32_t byte = sb[16 + 32 * p + i + k];
    wl[k] = fmaf(a_l, static_cast<float>(byte & 15u), -b_l);
    wh[k] = fmaf(a_h, static_cast<float>(byte >> 4), -b_h);
  }
  const int64_t cols = n_sb * 256;
  for (int c = 0; c < n_cols; ++c) {
    const float* xc = x + static_cast<int64_t>(c) * cols + s * 256 + 64 * p + i;
    float acc = 0.f;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      acc = fmaf(wl[k], xc[k], acc);
      acc = fmaf(wh[k], xc[32 + k], acc);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) part[(s * n_cols + c) * rows + row] = acc;
  }
}

int noalloc_fail(int code, const char* msg) {
  snprintf(g_noalloc_error, sizeof(g_noalloc_error), "%s", msg);
  return code;
}

}  // namespace

extern "C" {

int prima_gemv_q4k_noalloc(const void* dev_w, int64_t rows, int64_t cols, const float* dev_x, int n_cols, float* dev_y,
                           void* stream) {
  if (!dev_w || !dev_x || !dev_y) return noalloc_fail(PRIMA_ERR_ARG, "prima_gemv_q4k_noalloc: null pointer");
  if (rows < 1 || cols < 256 || cols % 256 != 0 || n_cols < 1 || n_cols > PRIMA_MAX_N_TOK)
    return noalloc_fail(PRIMA_ERR_ARG, "prima_gemv_q4k_noalloc: rows >= 1, cols a positive multiple of 256 and 1 <= n_cols <= 8 are required");
  const int64_t n_sb = cols / 256;
  // every factor is bounded before it enters a product, so that nothing wraps around for absurd sizes
  if (n_sb > kScratchFloats || rows > kScratchFloats / n_sb || rows * n_sb > kScratchFloats / n_cols) {
    snprintf(g_noalloc_error, sizeof(g_noalloc_error),
             "prima_gemv_q4k_noalloc: rows * (cols/256) * n_cols = %.0f exceeds the built-in scratch of %lld floats",
             static_cast<double>(rows) * static_cast<double>(n_sb) * n_cols, static_cast<long long>(kScratchFloats));
    return PRIMA_ERR_ARG;
  }
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) return noalloc_fail(PRIMA_ERR_CUDA, "prima_gemv_q4k_noalloc: cudaGetDevice failed");
  float* scratch = nullptr;
  {
    // First call on this device: ask the runtime where this device's copy of the array lives.  The
    // array's name is only a host-side handle; the kernel needs the address obtained here.
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[dev]) {
      float* p = nullptr;
      e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_noalloc_scratch);
      if (e != cudaSuccess || !p) {
        snprintf(g_noalloc_error, sizeof(g_noalloc_error), "prima_gemv_q4k_noalloc: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        return PRIMA_ERR_CUDA;
      }
      g_scratch_ptr[dev] = p;
    }
    scratch = g_scratch_ptr[dev];
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int warps_per_block = 8;
  const int64_t units = rows * n_sb;
  const int64_t grid = (units + warps_per_block - 1) / warps_per_block;
  if (grid > 0x7fffffff) return noalloc_fail(PRIMA_ERR_ARG, "prima_gemv_q4k_noalloc: matrix too large");
  gemv_std_partials_kernel<<<static_cast<unsigned>(grid), warps_per_block * 32, 0, st>>>(static_cast<const uint8_t*>(dev_w), rows, n_sb,
                                                                                        dev_x, n_cols, scratch);
  e = cudaGetLastError();
  if (e != cudaSuccess) {
    snprintf(g_noalloc_error, sizeof(g_noalloc_error), "prima_gemv_q4k_noalloc: launch failed: %s", cudaGetErrorString(e));
    return PRIMA_ERR_CUDA;
  }
  const int k = prima::launch_finish_plain(scratch, n_sb, rows, rows, n_cols, dev_y, prima::SumSq(), st);
  if (k < 0) return noalloc_fail(PRIMA_ERR_CUDA, "prima_gemv_q4k_noalloc: finishing kernel failed to launch");
  return PRIMA_OK;
}

const char* prima_gemv_q4k_noalloc_error(void) { return g_noalloc_error; }

}  // extern "C"
