// Shared device-side definitions: per-image descriptors, work items, vector loads.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ficoco {

constexpr int KCAP = 16;            // longest per-token top list (targets + 1 order statistic)
constexpr int MAX_CHUNKS = 64;      // row chunks per image for the column-sum partials
constexpr int MAX_IMG_TOKENS = 8192;
constexpr unsigned STATUS_POS_RANGE = 1u;

// One image (FiCoCo-V) or sequence (FiCoCo-L) of the batch.  All offsets are in elements of
// the array they index, counted over the whole packed batch.
struct ImgDesc {
  int row0;        // first token row in `tokens`
  int n_cls;       // leading pass-through rows (CLS)
  int np;          // alive vision tokens
  int n_src;       // N^S, discarded
  int n_tgt;       // N^T, preserved
  int n_tail;      // trailing pass-through rows (text)
  int n_extra;     // 1: one additional output row after the preserved tokens ("convergent correlation" ablation)
  int gh, gw;      // original patch grid
  int patch0;      // offset in per-vision-token arrays
  int out_row0;    // first output row (also offset in kept_idx)
  int src0;        // offset in per-discarded-token arrays
  int tgt0;        // offset in per-preserved-token arrays
  int ent0;        // offset in the (target, source, weight) entry arrays
  int part0;       // offset in the partial top-list arrays
  int list_len;    // L: entries of the top list needed for tau_i (0 = no merging)
  float frac;      // interpolation weight of the quantile
  int nsplit;      // column splits of the correlate step
  int cols_per_split;
  int corr_items;  // correlate work items (CTAs) of this image
  int chunk0;      // first row chunk (column-sum partials)
  int n_chunks;
  int avg;         // 1: every alpha_ij is 1 ("average compression" ablation)
  long long attn0; // offset (floats) of this image's attention block
  long long rel0;  // offset (floats) of this image's [Np, Np] relation block (relation mode)
};

struct WorkItem {
  int img;
  int r0;      // first row (patch / source slot / output row) inside the image
  int nrows;
  int aux;     // row chunks: chunk index inside the image; correlate: column split
};

// ---------------------------------------------------------------------------------------
// 16-byte vector access, converted to fp32 lanes
// ---------------------------------------------------------------------------------------
template <class T> struct VecTraits;
template <> struct VecTraits<float> { static constexpr int E = 4; };
template <> struct VecTraits<__nv_bfloat16> { static constexpr int E = 8; };

__device__ __forceinline__ void unpack(const uint4& u, float (&f)[4], const float*) {
  f[0] = __uint_as_float(u.x); f[1] = __uint_as_float(u.y);
  f[2] = __uint_as_float(u.z); f[3] = __uint_as_float(u.w);
}
__device__ __forceinline__ void unpack(const uint4& u, float (&f)[8], const __nv_bfloat16*) {
  f[0] = __uint_as_float(u.x << 16); f[1] = __uint_as_float(u.x & 0xFFFF0000u);
  f[2] = __uint_as_float(u.y << 16); f[3] = __uint_as_float(u.y & 0xFFFF0000u);
  f[4] = __uint_as_float(u.z << 16); f[5] = __uint_as_float(u.z & 0xFFFF0000u);
  f[6] = __uint_as_float(u.w << 16); f[7] = __uint_as_float(u.w & 0xFFFF0000u);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ uint4 pack(const float (&f)[4], const float*) {
  return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
}
__device__ __forceinline__ uint4 pack(const float (&f)[8], const __nv_bfloat16*) {
  return make_uint4(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3]), pack_bf16x2(f[4], f[5]), pack_bf16x2(f[6], f[7]));
}

__device__ __forceinline__ uint4 ldg16(const void* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }
// Streaming store (st.global.cs) for the output rows.  A step's token rows, read by all three of
// its kernels, plus its output rows are about as much as L2 keeps; written as ordinary stores the
// output pushes the token rows out before the next kernel reads them again.
__device__ __forceinline__ void st_stream16(uint4* p, const uint4& v) { __stcs(p, v); }

// A token index read from an index list of the step, as a row offset inside its image: anything
// outside [0, np) (lists left behind by a step that went wrong) raises STATUS_INDEX and becomes 0,
// so that no gather leaves the image.
__device__ __forceinline__ int checked_index(int idx, int np, unsigned* status) {
  if ((unsigned)idx >= (unsigned)np) {
    atomicOr(status, 8u);
    return 0;
  }
  return idx;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

// Order-preserving map fp32 -> uint32 (larger float <=> larger key).
__device__ __forceinline__ uint32_t order_key(float s) {
  uint32_t u = __float_as_uint(s);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Barrier over the first `n` threads of the CTA (n a multiple of 32) on hardware barrier `id`;
// cta_sync(0, blockDim.x) is __syncthreads().
__device__ __forceinline__ void cta_sync(int id, int n) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory");
}

// Exclusive prefix sum of one value per thread over `nthr` threads (<= 1024, multiple of 32)
// that synchronise on barrier `bar`.  `warp_tot` is a 33-int shared scratch.  Returns the
// exclusive prefix; *total gets the total.  Contains barriers: call from all `nthr` threads.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_tot, int* total, int bar, int nthr) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = nthr >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int n = __shfl_up_sync(0xFFFFFFFFu, inc, o);
    if (lane >= o) inc += n;
  }
  cta_sync(bar, nthr);
  if (lane == 31) warp_tot[warp] = inc;
  cta_sync(bar, nthr);
  if (warp == 0) {
    int w = (lane < nwarp) ? warp_tot[lane] : 0;
    int winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int n = __shfl_up_sync(0xFFFFFFFFu, winc, o);
      if (lane >= o) winc += n;
    }
    if (lane < nwarp) warp_tot[lane] = winc - w;
    if (lane == 31) warp_tot[32] = winc;
  }
  cta_sync(bar, nthr);
  *total = warp_tot[32];
  return warp_tot[warp] + inc - v;
}

// Sorted top list (descending value, ties: lower index first).
__device__ __forceinline__ bool toplist_better(float val, int idx, float v_last, int i_last) {
  return val > v_last || (val == v_last && idx < i_last);
}
__device__ __forceinline__ void toplist_insert(float* v, int* ix, int L, float val, int idx) {
  int p = L - 1;
  while (p > 0 && toplist_better(val, idx, v[p - 1], ix[p - 1])) {
    v[p] = v[p - 1];
    ix[p] = ix[p - 1];
    --p;
  }
  v[p] = val;
  ix[p] = idx;
}

}  // namespace ficoco
