// Equivalent token of the no-CLS variant (appendix "Implementation of the Equivalent Token"):
//   M = mean of the key states over the heads, mu = mean of M over the patch tokens,
//   a_i = -cos(mu, M_i).
//
// One thread-block cluster of 8 CTAs per image.  CTA r owns a contiguous eighth of the image's
// patch tokens; their key rows are contiguous in memory (token-major layout), so one producer
// lane streams them with 8-row bulk copies (TMA) through an mbarrier ring while 8 consumer
// warps reduce each row over its heads.  The head-mean keys stay in shared memory, so the keys
// are read from HBM exactly once; the only exchange between the CTAs of an image is their
// partial column sums (head_dim floats each), read from the peers' shared memory between two
// cluster barriers.  Sums run in a fixed order (heads, tokens of a warp, warps, cluster ranks):
// results are bit-reproducible.
// Every mbarrier wait is bounded; a CTA whose wait runs out writes NaN for its tokens and still
// takes part in the cluster barriers.
#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "../../include/ficoco.h"
#include "async_ops.cuh"
#include "common.cuh"

namespace cg = cooperative_groups;
using namespace ficoco;

namespace {

constexpr int EQ_CLUSTER = 8;          // CTAs per image
constexpr int EQ_ROWS = 8;             // key rows per ring stage (one per consumer warp)
constexpr int EQ_WARPS = 8;            // consumer warps
constexpr int EQ_THREADS = 32 * (EQ_WARPS + 1);
constexpr int EQ_MAX_STAGE = 6;
constexpr int EQ_MAX_BATCH_RAGGED = 256;
constexpr int EQ_MAX_HEAD_DIM = 256;   // four pairs of columns per lane
constexpr size_t EQ_SMEM_LIMIT = 220 * 1024;

// first row of every image of a ragged batch (kernel parameter space; no device allocation)
struct EqOffsets {
  int row0[EQ_MAX_BATCH_RAGGED + 1];
};

// two adjacent columns of one head
__device__ __forceinline__ float2 load_key2(const float* p) { return *reinterpret_cast<const float2*>(p); }
__device__ __forceinline__ float2 load_key2(const __nv_bfloat16* p) {
  const uint32_t u = *reinterpret_cast<const uint32_t*>(p);
  return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xFFFF0000u));
}

// Dynamic shared memory: ring [nstage][EQ_ROWS][heads * dk] of T | Ms [tpc_max][dk] |
// nrm2 [tpc_max] | csum [EQ_WARPS][dk] | part [dk] | mu [dk]    (floats after the ring)
template <class T>
__global__ void __launch_bounds__(EQ_THREADS, 2) k_equivalent_token(
    const T* __restrict__ keys, int heads, int dk, int n_cls, int uniform_tokens,
    const __grid_constant__ EqOffsets offs, float* __restrict__ a_eq, int tpc_max, int nstage) {
  extern __shared__ __align__(128) unsigned char eq_raw[];
  __shared__ uint64_t full_bar[EQ_MAX_STAGE], empty_bar[EQ_MAX_STAGE];
  __shared__ float n_mu_s;
  __shared__ int failed;

  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int img = blockIdx.x / EQ_CLUSTER;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int row0 = uniform_tokens > 0 ? img * uniform_tokens : offs.row0[img];
  const int rows_img = uniform_tokens > 0 ? uniform_tokens : offs.row0[img + 1] - row0;
  const int np = rows_img - n_cls;
  const int patch0 = row0 - img * n_cls;
  const int tpc = (np + EQ_CLUSTER - 1) / EQ_CLUSTER;
  const int t_lo = min(np, rank * tpc), t_hi = min(np, t_lo + tpc);
  const int nt = t_hi - t_lo;
  const int row_elems = heads * dk;
  const int row_bytes = row_elems * (int)sizeof(T);
  const int stage_bytes = EQ_ROWS * row_bytes;

  unsigned char* ring = eq_raw;
  float* Ms = reinterpret_cast<float*>(eq_raw + (size_t)nstage * stage_bytes);
  float* nrm2 = Ms + (size_t)tpc_max * dk;
  float* csum = nrm2 + tpc_max;
  float* part = csum + EQ_WARPS * dk;
  float* mu = part + dk;

  if (tid == 0) {
    for (int s = 0; s < nstage; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], EQ_WARPS); }
    failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  const int ngroups = (nt + EQ_ROWS - 1) / EQ_ROWS;
  if (warp == EQ_WARPS) {
    // ---------------- producer: bulk copies of EQ_ROWS rows into the ring -------------------------------
    if (lane == 0) {
      const unsigned char* base =
          reinterpret_cast<const unsigned char*>(keys + (size_t)(row0 + n_cls + t_lo) * row_elems);
      bool ok = true;
      for (int g = 0; g < ngroups && ok; ++g) {
        const int s = g % nstage;
        if (g >= nstage) ok = mbar_wait(&empty_bar[s], ((g / nstage) - 1) & 1);
        if (!ok) break;
        const int rows = min(EQ_ROWS, nt - g * EQ_ROWS);
        mbar_expect_tx(&full_bar[s], (uint32_t)(rows * row_bytes));
        bulk_load(ring + (size_t)s * stage_bytes, base + (size_t)g * stage_bytes, (uint32_t)(rows * row_bytes),
                  &full_bar[s]);
      }
      if (!ok) failed = 1;
    }
  } else {
    // ---------------- consumers: head mean, squared norm, column sums --------------------------
    float col[EQ_MAX_HEAD_DIM / 32];
#pragma unroll
    for (int j = 0; j < EQ_MAX_HEAD_DIM / 32; ++j) col[j] = 0.f;
    const float inv_h = 1.0f / (float)heads;
    bool ok = true;
    for (int g = 0; g < ngroups; ++g) {
      const int s = g % nstage;
      if (ok) ok = mbar_wait(&full_bar[s], (g / nstage) & 1);
      if (ok) {
        for (int rr = warp; rr < EQ_ROWS; rr += EQ_WARPS) {
          const int t = g * EQ_ROWS + rr;
          if (t >= nt) break;
          const T* rp = reinterpret_cast<const T*>(ring + (size_t)s * stage_bytes + (size_t)rr * row_bytes);
          float ss = 0.f;
#pragma unroll
          for (int j = 0; j < EQ_MAX_HEAD_DIM / 64; ++j) {
            const int o = 2 * (lane + 32 * j);           // this lane's pair of columns
            if (o < dk) {
              // four running sums, so that the loads of four heads are in flight together
              float2 m0 = make_float2(0.f, 0.f), m1 = m0, m2 = m0, m3 = m0;
              int h = 0;
              for (; h + 4 <= heads; h += 4) {
                const float2 k0 = load_key2(rp + (h + 0) * dk + o), k1 = load_key2(rp + (h + 1) * dk + o);
                const float2 k2 = load_key2(rp + (h + 2) * dk + o), k3 = load_key2(rp + (h + 3) * dk + o);
                m0.x += k0.x; m0.y += k0.y; m1.x += k1.x; m1.y += k1.y;
                m2.x += k2.x; m2.y += k2.y; m3.x += k3.x; m3.y += k3.y;
              }
              for (; h < heads; ++h) {
                const float2 k0 = load_key2(rp + h * dk + o);
                m0.x += k0.x; m0.y += k0.y;
              }
              const float mx = ((m0.x + m1.x) + (m2.x + m3.x)) * inv_h;
              const float my = ((m0.y + m1.y) + (m2.y + m3.y)) * inv_h;
              *reinterpret_cast<float2*>(Ms + (size_t)t * dk + o) = make_float2(mx, my);
              col[2 * j] += mx;
              col[2 * j + 1] += my;
              ss = fmaf(mx, mx, fmaf(my, my, ss));
            }
          }
          ss = warp_sum(ss);
          if (lane == 0) nrm2[t] = ss;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty_bar[s]);
    }
    if (!ok) failed = 1;
#pragma unroll
    for (int j = 0; j < EQ_MAX_HEAD_DIM / 64; ++j) {
      const int o = 2 * (lane + 32 * j);
      if (o < dk) { csum[warp * dk + o] = col[2 * j]; csum[warp * dk + o + 1] = col[2 * j + 1]; }
    }
  }
  __syncthreads();
  for (int o = tid; o < dk; o += EQ_THREADS) {
    float t = 0.f;
    for (int ww = 0; ww < EQ_WARPS; ++ww) t += csum[ww * dk + o];
    part[o] = t;
  }
  cluster.sync();                          // every CTA's partial column sums are in place
  for (int o = tid; o < dk; o += EQ_THREADS) {
    float t = 0.f;
    for (int r = 0; r < EQ_CLUSTER; ++r) t += cluster.map_shared_rank(part, r)[o];
    mu[o] = t / (float)np;
  }
  __syncthreads();
  if (warp == 0) {
    float ss = 0.f;
    for (int o = lane; o < dk; o += 32) ss = fmaf(mu[o], mu[o], ss);
    ss = warp_sum(ss);
    if (lane == 0) n_mu_s = sqrtf(ss);
  }
  cluster.sync();                          // peers have read this CTA's partial: it may exit later
  const float n_mu = n_mu_s;
  const bool bad = failed != 0;
  if (warp < EQ_WARPS) {
    for (int t = warp; t < nt; t += EQ_WARPS) {
      float dot = 0.f;
      for (int o = lane; o < dk; o += 32) dot = fmaf(mu[o], Ms[(size_t)t * dk + o], dot);
      dot = warp_sum(dot);
      if (lane == 0) {
        const float n_i = sqrtf(nrm2[t]);
        float a = (n_mu > 0.f && n_i > 0.f) ? -dot / (n_mu * n_i) : 0.f;
        if (bad) a = CUDART_NAN_F;
        a_eq[patch0 + t_lo + t] = a;
      }
    }
  }
}

template <class T>
cudaError_t launch_eq(const void* keys, int batch, int uniform_tokens, const EqOffsets& offs, int heads, int dk,
                      int n_cls, float* a_eq, int tpc_max, int nstage, size_t smem, cudaStream_t st) {
  cudaError_t e = cudaFuncSetAttribute(k_equivalent_token<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)EQ_SMEM_LIMIT);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(batch * EQ_CLUSTER);
  cfg.blockDim = dim3(EQ_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = EQ_CLUSTER;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k_equivalent_token<T>, (const T*)keys, heads, dk, n_cls, uniform_tokens, offs,
                            a_eq, tpc_max, nstage);
}

}  // namespace

extern "C" int ficoco_equivalent_token(const void* keys, int dtype, int batch, int n_tokens, const int* seqlens,
                                       int heads, int head_dim, int has_cls, float* a_eq, void* cuda_stream) {
  if (!keys || !a_eq || batch < 1 || heads < 1 || head_dim < 1) return FICOCO_ERR_INVALID_ARG;
  if (dtype != FICOCO_FP32 && dtype != FICOCO_BF16) return FICOCO_ERR_UNSUPPORTED;
  const int n_cls = has_cls ? 1 : 0;
  const size_t es = dtype == FICOCO_BF16 ? 2 : 4;
  const size_t row_bytes = (size_t)heads * head_dim * es;
  if (row_bytes % 16 != 0 || ((uintptr_t)keys & 15) != 0) return FICOCO_ERR_INVALID_ARG;
  if (head_dim > EQ_MAX_HEAD_DIM || head_dim % 2 != 0) return FICOCO_ERR_UNSUPPORTED;
  EqOffsets offs;
  offs.row0[0] = 0;
  int max_np = 0;
  if (seqlens) {
    if (batch > EQ_MAX_BATCH_RAGGED) return FICOCO_ERR_UNSUPPORTED;
    long long r = 0;
    for (int b = 0; b < batch; ++b) {
      if (seqlens[b] < n_cls + 1) return FICOCO_ERR_INVALID_ARG;
      r += seqlens[b];
      if (r > INT32_MAX) return FICOCO_ERR_UNSUPPORTED;
      offs.row0[b + 1] = (int)r;
      if (seqlens[b] - n_cls > max_np) max_np = seqlens[b] - n_cls;
    }
  } else {
    if (n_tokens < n_cls + 1) return FICOCO_ERR_INVALID_ARG;
    if ((long long)batch * n_tokens > INT32_MAX) return FICOCO_ERR_UNSUPPORTED;
    max_np = n_tokens - n_cls;
  }
  const int tpc_max = (max_np + EQ_CLUSTER - 1) / EQ_CLUSTER;
  const size_t tail = ((size_t)tpc_max * head_dim + tpc_max + (EQ_WARPS + 2) * (size_t)head_dim) * sizeof(float);
  const size_t stage_bytes = (size_t)EQ_ROWS * row_bytes;
  if (tail + 2 * stage_bytes > EQ_SMEM_LIMIT) return FICOCO_ERR_UNSUPPORTED;
  // prefer a ring small enough for two CTAs per SM (an image's cluster then needs four SMs, and
  // a batch of 32 images is resident at once); otherwise the deepest ring that fits
  int nstage = 0;
  if (tail + 2 * stage_bytes <= EQ_SMEM_LIMIT / 2) nstage = (int)((EQ_SMEM_LIMIT / 2 - tail) / stage_bytes);
  else nstage = (int)((EQ_SMEM_LIMIT - tail) / stage_bytes);
  if (nstage > EQ_MAX_STAGE) nstage = EQ_MAX_STAGE;
  const size_t smem = (size_t)nstage * stage_bytes + tail;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const int uniform = seqlens ? 0 : n_tokens;
  const cudaError_t e = dtype == FICOCO_BF16
      ? launch_eq<__nv_bfloat16>(keys, batch, uniform, offs, heads, head_dim, n_cls, a_eq, tpc_max, nstage, smem, st)
      : launch_eq<float>(keys, batch, uniform, offs, heads, head_dim, n_cls, a_eq, tpc_max, nstage, smem, st);
  return e == cudaSuccess ? FICOCO_OK : FICOCO_ERR_CUDA;
}
