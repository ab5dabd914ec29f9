// Allocation-free entry point: the vision-aware redundancy (first term of Eq. 1) with all of
// its scratch in a fixed device array that is part of the library image.
//
// Who needs this: code that runs where device allocation is off limits.  The usual case is a
// step/enqueue callback of a serving engine that has handed every byte of device memory to its
// own pool at start-up: a cudaMalloc there can fail outright, and even when it succeeds it
// synchronises the whole device and stalls every other stream of the engine.  Such a caller
// cannot create a ficoco context (ficoco_create allocates), but it can still pass input and
// output buffers it already owns.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ficoco.h"
#include "common.cuh"

using namespace ficoco;

namespace {

constexpr int NA_MAX_ROWS = FICOCO_NOALLOC_MAX_ROWS;     // vision tokens over the whole batch
constexpr int NA_MAX_BATCH = FICOCO_NOALLOC_MAX_BATCH;
constexpr int NA_MAX_DIM = FICOCO_NOALLOC_MAX_DIM;
constexpr int NA_CHUNK = 64;                             // rows per CTA
constexpr int NA_MAX_CHUNKS = NA_MAX_ROWS / NA_CHUNK + NA_MAX_BATCH;

// Layout of the scratch: rn[NA_MAX_ROWS] | partial[NA_MAX_CHUNKS][NA_MAX_DIM]   (floats)
constexpr size_t NA_RN_FLOATS = NA_MAX_ROWS;
constexpr size_t NA_PARTIAL_FLOATS = (size_t)NA_MAX_CHUNKS * NA_MAX_DIM;
constexpr size_t NA_SCRATCH_FLOATS = NA_RN_FLOATS + NA_PARTIAL_FLOATS;

// Every GPU that loads the library holds this array (about 4.7 MB) until the process exits.
static __device__ __align__(256) float g_noalloc_scratch[NA_SCRATCH_FLOATS];

// Device address of the array, per device ordinal, filled by the first call on that device.
constexpr int NA_MAX_DEVICES = 64;
float* g_scratch_addr[NA_MAX_DEVICES] = {nullptr};

// Pass 1.  One CTA per chunk of up to 64 vision tokens of one image:
//   rn_i = 1 / ||x_i|| (one warp per token), then partial[chunk][d] = sum_i rn_i x_id with one
//   thread per column, rows in ascending order.  Every scratch word that pass 2 reads is
//   written here first, so nothing has to be cleared between calls.
template <class T>
__global__ void __launch_bounds__(256) k_na_colsum(const T* __restrict__ tokens, int n_tokens, int n_cls,
                                                   int D, int chunks_per_img, float* __restrict__ rn,
                                                   float* __restrict__ partial) {
  constexpr int E = VecTraits<T>::E;
  __shared__ float rn_s[NA_CHUNK];
  const int img = blockIdx.x / chunks_per_img, chunk = blockIdx.x % chunks_per_img;
  const int np = n_tokens - n_cls;
  const int r0 = chunk * NA_CHUNK;
  const int nrows = min(NA_CHUNK, np - r0);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const T* base = tokens + ((size_t)img * n_tokens + n_cls + r0) * D;
  const int nvec = D / E;
  for (int r = warp; r < nrows; r += 8) {
    float ss = 0.f;
    for (int v = lane; v < nvec; v += 32) {
      float f[E];
      unpack(ldg16(base + (size_t)r * D + (size_t)v * E), f, (const T*)nullptr);
#pragma unroll
      for (int e = 0; e < E; ++e) ss = fmaf(f[e], f[e], ss);
    }
    ss = warp_sum(ss);
    if (lane == 0) {
      const float s = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
      rn_s[r] = s;
      rn[(size_t)img * np + r0 + r] = s;
    }
  }
  __syncthreads();
  float* out = partial + (size_t)blockIdx.x * D;
  for (int v = threadIdx.x; v < nvec; v += 256) {
    float acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;
    for (int r = 0; r < nrows; ++r) {
      float f[E];
      unpack(ldg16(base + (size_t)r * D + (size_t)v * E), f, (const T*)nullptr);
      const float s = rn_s[r];
#pragma unroll
      for (int e = 0; e < E; ++e) acc[e] = fmaf(f[e], s, acc[e]);
    }
#pragma unroll
    for (int e = 0; e < E; ++e) out[(size_t)v * E + e] = acc[e];
  }
}

// Pass 2.  v_i = rn_i * (x_i . sum of the image's partials) / Np, one warp per token.
template <class T>
__global__ void __launch_bounds__(256) k_na_rowdot(const T* __restrict__ tokens, int n_tokens, int n_cls,
                                                   int D, int chunks_per_img, const float* __restrict__ rn,
                                                   const float* __restrict__ partial, float* __restrict__ v_out) {
  constexpr int E = VecTraits<T>::E;
  extern __shared__ float msum[];
  const int img = blockIdx.x / chunks_per_img, chunk = blockIdx.x % chunks_per_img;
  const int np = n_tokens - n_cls;
  const int r0 = chunk * NA_CHUNK;
  const int nrows = min(NA_CHUNK, np - r0);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int c = threadIdx.x; c < D; c += 256) {
    float s = 0.f;
    for (int k = 0; k < chunks_per_img; ++k) s += partial[((size_t)img * chunks_per_img + k) * D + c];
    msum[c] = s;
  }
  __syncthreads();
  const T* base = tokens + ((size_t)img * n_tokens + n_cls + r0) * D;
  const int nvec = D / E;
  const float inv_np = 1.0f / (float)np;
  for (int r = warp; r < nrows; r += 8) {
    float dot = 0.f;
    for (int v = lane; v < nvec; v += 32) {
      float f[E];
      unpack(ldg16(base + (size_t)r * D + (size_t)v * E), f, (const T*)nullptr);
#pragma unroll
      for (int e = 0; e < E; ++e) dot = fmaf(f[e], msum[(size_t)v * E + e], dot);
    }
    dot = warp_sum(dot);
    if (lane == 0) v_out[(size_t)img * np + r0 + r] = dot * rn[(size_t)img * np + r0 + r] * inv_np;
  }
}

}  // namespace

extern "C" int ficoco_vision_redundancy_noalloc(const void* tokens, int dtype, int batch, int n_tokens,
                                                int dim, unsigned flags, float* v_out, void* cuda_stream) {
  if (!tokens || !v_out || batch < 1 || n_tokens < 1 || dim < 1) return FICOCO_ERR_INVALID_ARG;
  if (dtype != FICOCO_FP32 && dtype != FICOCO_BF16) return FICOCO_ERR_UNSUPPORTED;
  const int e = dtype == FICOCO_BF16 ? 8 : 4;
  if (dim % e != 0) return FICOCO_ERR_UNSUPPORTED;
  if (((uintptr_t)tokens & 15) || ((uintptr_t)v_out & 3)) return FICOCO_ERR_INVALID_ARG;
  const int n_cls = (flags & FICOCO_HAS_CLS) ? 1 : 0;
  const int np = n_tokens - n_cls;
  if (np < 1) return FICOCO_ERR_INVALID_ARG;
  const int chunks = (np + NA_CHUNK - 1) / NA_CHUNK;
  if (batch > NA_MAX_BATCH || dim > NA_MAX_DIM || (long long)batch * np > NA_MAX_ROWS ||
      (long long)batch * chunks > NA_MAX_CHUNKS)
    return FICOCO_ERR_STATIC_LIMIT;

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NA_MAX_DEVICES) return FICOCO_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (g_scratch_addr[dev] == nullptr) {
    // The address lookup may load the module: it must not run under stream capture.
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cs) != cudaSuccess) { cudaGetLastError(); return FICOCO_ERR_CUDA; }
    if (cs != cudaStreamCaptureStatusNone) return FICOCO_ERR_CAPTURE;
    // The array's name is only a handle on the host; the kernels need its device address.
    float* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return FICOCO_ERR_CUDA;
    }
    g_scratch_addr[dev] = p;
  }
  float* rn = g_scratch_addr[dev];
  float* partial = rn + NA_RN_FLOATS;
  const int grid = batch * chunks;
  cudaGetLastError();                       // an error left over from earlier work is not this call's
  if (dtype == FICOCO_BF16) {
    const __nv_bfloat16* t = (const __nv_bfloat16*)tokens;
    k_na_colsum<__nv_bfloat16><<<grid, 256, 0, st>>>(t, n_tokens, n_cls, dim, chunks, rn, partial);
    if (cudaGetLastError() != cudaSuccess) return FICOCO_ERR_CUDA;      // the second kernel needs the first
    k_na_rowdot<__nv_bfloat16><<<grid, 256, dim * sizeof(float), st>>>(t, n_tokens, n_cls, dim, chunks, rn,
                                                                         partial, v_out);
  } else {
    const float* t = (const float*)tokens;
    k_na_colsum<float><<<grid, 256, 0, st>>>(t, n_tokens, n_cls, dim, chunks, rn, partial);
    if (cudaGetLastError() != cudaSuccess) return FICOCO_ERR_CUDA;
    k_na_rowdot<float><<<grid, 256, dim * sizeof(float), st>>>(t, n_tokens, n_cls, dim, chunks, rn, partial,
                                                              v_out);
  }
  return cudaGetLastError() == cudaSuccess ? FICOCO_OK : FICOCO_ERR_CUDA;
}
