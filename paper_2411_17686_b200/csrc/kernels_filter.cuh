// Filter stage (Eq. 1, local penalty, top-N^S selection).
#pragma once
#include "async_ops.cuh"
#include "common.cuh"

namespace ficoco {

// ---------------------------------------------------------------------------------------
// Row norms.  One warp per vision token: rn_i = 1 / ||x_i||.  Used alone when the hidden
// size is too wide for the fused kernel below.
// ---------------------------------------------------------------------------------------
template <class T>
__global__ void __launch_bounds__(256) k_rownorm(const T* __restrict__ tokens, int D,
                                                 const ImgDesc* __restrict__ desc,
                                                 const WorkItem* __restrict__ work,
                                                 float* __restrict__ rn) {
  constexpr int E = VecTraits<T>::E;
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nvec = D / E;
  for (int r = warp; r < w.nrows; r += 8) {
    const T* row = tokens + (size_t)(d.row0 + d.n_cls + w.r0 + r) * D;
    float ss = 0.f;
    for (int v0 = lane; v0 < nvec; v0 += 32 * 8) {     // eight 16-byte loads in flight per lane
      uint4 u[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int v = v0 + 32 * k;
        u[k] = v < nvec ? ldg16(row + (size_t)v * E) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        float f[E];
        unpack(u[k], f, (const T*)nullptr);
#pragma unroll
        for (int e = 0; e < E; ++e) ss = fmaf(f[e], f[e], ss);
      }
    }
    ss = warp_sum(ss);
    if (lane == 0) rn[d.patch0 + w.r0 + r] = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
  }
}

// ---------------------------------------------------------------------------------------
// Column sums of the normalised tokens: partial[chunk][d] = sum_{i in chunk} rn_i x_id.
// The row mean of the cosine relation is x_hat_i . (1/N) sum_j x_hat_j, so this vector is
// all the first term of Eq. 1 needs.  One CTA per row chunk; a warp owns whole rows, each
// lane the 16-byte vectors lane, lane+32, ... of the column slab [c0, c0 + VPL*32*E).
// FUSED: the CTA also computes rn (requires the slab to cover the full row).
// Warps are folded into shared memory one after the other, so the result does not depend
// on scheduling.
// ---------------------------------------------------------------------------------------
template <class T, int VPL, bool FUSED>
__global__ void __launch_bounds__(256) k_colsum(const T* __restrict__ tokens, int D,
                                                const ImgDesc* __restrict__ desc,
                                                const WorkItem* __restrict__ work,
                                                float* __restrict__ rn,
                                                float* __restrict__ partial) {
  constexpr int E = VecTraits<T>::E;
  extern __shared__ float sm_acc[];  // VPL*32*E floats
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int slab = blockIdx.y;
  const int c0 = slab * (VPL * 32 * E);
  const int nvec = (min(D - c0, VPL * 32 * E)) / E;

  float acc[VPL][E];
#pragma unroll
  for (int k = 0; k < VPL; ++k)
#pragma unroll
    for (int e = 0; e < E; ++e) acc[k][e] = 0.f;

  const T* base = tokens + (size_t)(d.row0 + d.n_cls + w.r0) * D + c0;
  float* rn_out = rn + d.patch0 + w.r0;

  for (int r = warp; r < w.nrows; r += 16) {
    const int r2 = r + 8;
    const bool has2 = r2 < w.nrows;
    uint4 u[VPL], u2[VPL];
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
      const int v = lane + 32 * k;
      u[k] = (v < nvec) ? ldg16(base + (size_t)r * D + (size_t)v * E) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
      const int v = lane + 32 * k;
      u2[k] = (has2 && v < nvec) ? ldg16(base + (size_t)r2 * D + (size_t)v * E) : make_uint4(0, 0, 0, 0);
    }
    float s1, s2;
    if (FUSED) {
      float ss = 0.f, ss2 = 0.f;
#pragma unroll
      for (int k = 0; k < VPL; ++k) {
        float f[E];
        unpack(u[k], f, (const T*)nullptr);
#pragma unroll
        for (int e = 0; e < E; ++e) ss = fmaf(f[e], f[e], ss);
        unpack(u2[k], f, (const T*)nullptr);
#pragma unroll
        for (int e = 0; e < E; ++e) ss2 = fmaf(f[e], f[e], ss2);
      }
      ss = warp_sum(ss);
      ss2 = warp_sum(ss2);
      s1 = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
      s2 = ss2 > 0.f ? 1.0f / sqrtf(ss2) : 0.f;
      if (lane == 0) {
        rn_out[r] = s1;
        if (has2) rn_out[r2] = s2;
      }
    } else {
      s1 = rn_out[r];
      s2 = has2 ? rn_out[r2] : 0.f;
    }
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
      float f[E];
      unpack(u[k], f, (const T*)nullptr);
#pragma unroll
      for (int e = 0; e < E; ++e) acc[k][e] = fmaf(f[e], s1, acc[k][e]);
      unpack(u2[k], f, (const T*)nullptr);
#pragma unroll
      for (int e = 0; e < E; ++e) acc[k][e] = fmaf(f[e], s2, acc[k][e]);
    }
  }

  // fold the 8 warps in order
  for (int wv = 0; wv < 8; ++wv) {
    if (warp == wv) {
#pragma unroll
      for (int k = 0; k < VPL; ++k) {
        const int v = lane + 32 * k;
        float* dst = sm_acc + (size_t)v * E;
#pragma unroll
        for (int e = 0; e < E; ++e) dst[e] = (wv == 0) ? acc[k][e] : dst[e] + acc[k][e];
      }
    }
    __syncthreads();
  }
  float* out = partial + (size_t)(d.chunk0 + w.aux) * D + c0;
  for (int i = threadIdx.x; i < nvec * E; i += 256) out[i] = sm_acc[i];
}

// ---------------------------------------------------------------------------------------
// Eq. 1 (and the FiCoCo-L score): s_i = cA * v_i - (1 - cA) * a_i with
//   v_i = rn_i * (x_i . msum) / Np,   msum = the image's column sums (k_msum),
//   a_i = (1/H) sum_h attn[h, i]      (FiCoCo-L: H = M rows of the head-mean block t).
// One CTA per row chunk, one warp per token for the dot product.
// ---------------------------------------------------------------------------------------
// Column sums of every image: msum[b, c] = sum over the image's row chunks, in chunk order.
__global__ void __launch_bounds__(256) k_msum(int D, const ImgDesc* __restrict__ desc,
                                              const float* __restrict__ partial, float* __restrict__ msum) {
  const ImgDesc d = desc[blockIdx.x];
  const int c = blockIdx.y * 256 + threadIdx.x;
  if (c >= D) return;
  float s = 0.f;
  for (int k = 0; k < d.n_chunks; ++k) s += partial[(size_t)(d.chunk0 + k) * D + c];
  msum[(size_t)blockIdx.x * D + c] = s;
}

// Mean over the H attention rows of the chunk's tokens, a_i = (1/H) sum_h attn[h, i], by all 256 threads:
// warp q adds rows q, q + 8, ... for 32 tokens per lane trip (eight loads in flight), the eight partial sums
// of a token are then added in warp order.  `part` holds 8 * nrows floats.
__device__ __forceinline__ void attn_mean_rows(const float* __restrict__ a0, int H, int np, int nrows,
                                               float* part, int tid) {
  const int lane = tid & 31, warp = tid >> 5;
  for (int r = lane; r < nrows; r += 32) {
    float s = 0.f;
    for (int h0 = warp; h0 < H; h0 += 64) {
      float q[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) q[j] = h0 + 8 * j < H ? __ldg(a0 + (size_t)(h0 + 8 * j) * np + r) : 0.f;
#pragma unroll
      for (int j = 0; j < 8; ++j) s += q[j];
    }
    part[warp * nrows + r] = s;
  }
}

template <class T>
__global__ void __launch_bounds__(256) k_score(const T* __restrict__ tokens, int D,
                                               const ImgDesc* __restrict__ desc,
                                               const WorkItem* __restrict__ work,
                                               const float* __restrict__ rn,
                                               const float* __restrict__ msum_all,
                                               const float* __restrict__ attn, int H, float cA,
                                               float* __restrict__ s_raw) {
  constexpr int E = VecTraits<T>::E;
  extern __shared__ float sm[];  // msum[D], v[nrows], attention partial sums [8][nrows]
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  float* msum = sm;
  float* vrow = sm + D;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  for (int c = threadIdx.x; c < D; c += 256) msum[c] = msum_all[(size_t)w.img * D + c];
  __syncthreads();

  const int nvec = D / E;
  const float inv_np = 1.0f / (float)d.np;
  for (int r = warp; r < w.nrows; r += 8) {
    const T* row = tokens + (size_t)(d.row0 + d.n_cls + w.r0 + r) * D;
    float dot = 0.f;
    for (int v0 = lane; v0 < nvec; v0 += 32 * 8) {     // eight 16-byte loads in flight per lane
      uint4 u[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int v = v0 + 32 * k;
        u[k] = v < nvec ? ldg16(row + (size_t)v * E) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int v = v0 + 32 * k;
        if (v < nvec) {
          float f[E];
          unpack(u[k], f, (const T*)nullptr);
          const float* m = msum + (size_t)v * E;
#pragma unroll
          for (int e = 0; e < E; ++e) dot = fmaf(f[e], m[e], dot);
        }
      }
    }
    dot = warp_sum(dot);
    if (lane == 0) vrow[r] = dot * rn[d.patch0 + w.r0 + r] * inv_np;
  }
  __syncthreads();

  const float inv_h = 1.0f / (float)H;
  float* part = vrow + w.nrows;
  attn_mean_rows(attn + d.attn0 + w.r0, H, d.np, w.nrows, part, threadIdx.x);
  __syncthreads();
  for (int r = threadIdx.x; r < w.nrows; r += 256) {
    float s = 0.f;
#pragma unroll
    for (int q = 0; q < 8; ++q) s += part[q * w.nrows + r];
    s_raw[d.patch0 + w.r0 + r] = cA * vrow[r] - (1.0f - cA) * (s * inv_h);
  }
}

// ---------------------------------------------------------------------------------------
// Wide rows (more than 256 16-byte vectors: hidden 4096 in bf16): a row no longer fits one
// warp's registers, so the CTA's 256 threads own the row's column vectors (NV each) and rows
// go through in batches of RB.  A per-row sum is folded lane -> warp -> the 8 warps in order.
//   k_colsum_wide: row norms and the chunk's column sums of the normalised rows in one read;
//                  every thread keeps the sums of its own columns, so there is no fold at the end
//   k_score_wide:  Eq. 1 with the image's column sums held in registers
// ---------------------------------------------------------------------------------------
template <class T, int NV, int RB>
__device__ __forceinline__ void wide_load(const T* __restrict__ base, int D, int nvec, int r0, int nrows, int tid,
                                          uint4 (&u)[RB][NV]) {
  constexpr int E = VecTraits<T>::E;
#pragma unroll
  for (int j = 0; j < RB; ++j)
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      const int v = tid + 256 * k;
      u[j][k] = (r0 + j < nrows && v < nvec) ? ldg16(base + (size_t)(r0 + j) * D + (size_t)v * E) : make_uint4(0, 0, 0, 0);
    }
}

__device__ __forceinline__ float fold8(const float* r) {
  const float4 a = *reinterpret_cast<const float4*>(r), b = *reinterpret_cast<const float4*>(r + 4);
  return ((((((a.x + a.y) + a.z) + a.w) + b.x) + b.y) + b.z) + b.w;
}

template <class T, int NV, int RB>
__global__ void __launch_bounds__(256, 2) k_colsum_wide(const T* __restrict__ tokens, int D,
                                                     const ImgDesc* __restrict__ desc,
                                                     const WorkItem* __restrict__ work,
                                                     float* __restrict__ rn_out, float* __restrict__ partial) {
  constexpr int E = VecTraits<T>::E;
  __shared__ __align__(16) float red[2][RB][8];
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nvec = D / E;
  const T* base = tokens + (size_t)(d.row0 + d.n_cls + w.r0) * D;
  float* rn = rn_out + d.patch0 + w.r0;
  float acc[NV][E];
#pragma unroll
  for (int k = 0; k < NV; ++k)
#pragma unroll
    for (int e = 0; e < E; ++e) acc[k][e] = 0.f;

  int par = 0;
  for (int r0 = 0; r0 < w.nrows; r0 += RB, par ^= 1) {
    uint4 u[RB][NV];
    wide_load<T, NV, RB>(base, D, nvec, r0, w.nrows, tid, u);
#pragma unroll
    for (int j = 0; j < RB; ++j) {
      float ss = 0.f;
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        float f[E];
        unpack(u[j][k], f, (const T*)nullptr);
#pragma unroll
        for (int e = 0; e < E; ++e) ss = fmaf(f[e], f[e], ss);
      }
      ss = warp_sum(ss);
      if (lane == 0) red[par][j][warp] = ss;
    }
    __syncthreads();   // one barrier per batch: the next batch writes the other half of `red`
#pragma unroll
    for (int j = 0; j < RB; ++j) {
      const float tot = fold8(red[par][j]);
      const float sc = tot > 0.f ? 1.0f / sqrtf(tot) : 0.f;
      if (tid == j && r0 + j < w.nrows) rn[r0 + j] = sc;
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        float f[E];
        // unpack again rather than keep the batch's converted values in registers across the barrier
        asm volatile("" : "+r"(u[j][k].x), "+r"(u[j][k].y), "+r"(u[j][k].z), "+r"(u[j][k].w));
        unpack(u[j][k], f, (const T*)nullptr);
#pragma unroll
        for (int e = 0; e < E; ++e) acc[k][e] = fmaf(f[e], sc, acc[k][e]);
      }
    }
  }
  float* out = partial + (size_t)(d.chunk0 + w.aux) * D;
#pragma unroll
  for (int k = 0; k < NV; ++k) {
    const int v = tid + 256 * k;
    if (v < nvec) {
#pragma unroll
      for (int e = 0; e < E; e += 4)
        *reinterpret_cast<float4*>(out + (size_t)v * E + e) = make_float4(acc[k][e], acc[k][e + 1], acc[k][e + 2], acc[k][e + 3]);
    }
  }
}

template <class T, int NV, int RB>
__global__ void __launch_bounds__(256) k_score_wide(const T* __restrict__ tokens, int D,
                                                    const ImgDesc* __restrict__ desc,
                                                    const WorkItem* __restrict__ work,
                                                    const float* __restrict__ rn,
                                                    const float* __restrict__ msum_all,
                                                    const float* __restrict__ attn, int H, float cA,
                                                    float* __restrict__ s_raw) {
  constexpr int E = VecTraits<T>::E;
  extern __shared__ float vrow[];  // v[nrows], attention partial sums [8][nrows]
  __shared__ __align__(16) float red[2][RB][8];
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nvec = D / E;
  const T* base = tokens + (size_t)(d.row0 + d.n_cls + w.r0) * D;
  float m[NV][E];
#pragma unroll
  for (int k = 0; k < NV; ++k) {
    const int v = tid + 256 * k;
#pragma unroll
    for (int e = 0; e < E; e += 4) {
      const float4 q = v < nvec ? __ldg(reinterpret_cast<const float4*>(msum_all + (size_t)w.img * D + (size_t)v * E + e))
                                : make_float4(0.f, 0.f, 0.f, 0.f);
      m[k][e] = q.x; m[k][e + 1] = q.y; m[k][e + 2] = q.z; m[k][e + 3] = q.w;
    }
  }
  const float inv_np = 1.0f / (float)d.np;
  int par = 0;
  for (int r0 = 0; r0 < w.nrows; r0 += RB, par ^= 1) {
    uint4 u[RB][NV];
    wide_load<T, NV, RB>(base, D, nvec, r0, w.nrows, tid, u);
#pragma unroll
    for (int j = 0; j < RB; ++j) {
      float dot = 0.f;
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        float f[E];
        unpack(u[j][k], f, (const T*)nullptr);
#pragma unroll
        for (int e = 0; e < E; ++e) dot = fmaf(f[e], m[k][e], dot);
      }
      dot = warp_sum(dot);
      if (lane == 0) red[par][j][warp] = dot;
    }
    __syncthreads();
    if (tid < RB && r0 + tid < w.nrows)
      vrow[r0 + tid] = fold8(red[par][tid]) * rn[d.patch0 + w.r0 + r0 + tid] * inv_np;
  }
  __syncthreads();

  const float inv_h = 1.0f / (float)H;
  float* part = vrow + w.nrows;
  attn_mean_rows(attn + d.attn0 + w.r0, H, d.np, w.nrows, part, tid);
  __syncthreads();
  for (int r = tid; r < w.nrows; r += 256) {
    float s = 0.f;
#pragma unroll
    for (int q = 0; q < 8; ++q) s += part[q * w.nrows + r];
    s_raw[d.patch0 + w.r0 + r] = cA * vrow[r] - (1.0f - cA) * (s * inv_h);
  }
}

// ---------------------------------------------------------------------------------------
// FiCoCo-L: head mean of the text->vision attention, t[b, k, i] = (1/H) sum_h A[b, h, k, i].
// One CTA per (sequence, text row).
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_head_mean(const float* __restrict__ attn, int H, int M,
                                                   int N, float* __restrict__ t) {
  const int b = blockIdx.x / M, k = blockIdx.x % M;
  const float inv_h = 1.0f / (float)H;
  const float* src = attn + ((size_t)b * H * M + k) * N;
  float* dst = t + ((size_t)b * M + k) * N;
  if ((N & 3) == 0 && (reinterpret_cast<uintptr_t>(attn) & 15) == 0 && (reinterpret_cast<uintptr_t>(t) & 15) == 0) {
    // four tokens per thread, eight heads in flight, added in head order
    for (int i = threadIdx.x * 4; i < N; i += 1024) {
      float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int h0 = 0; h0 < H; h0 += 8) {
        float4 a[8];
#pragma unroll
        for (int q = 0; q < 8; ++q)
          a[q] = h0 + q < H ? __ldg(reinterpret_cast<const float4*>(src + (size_t)(h0 + q) * M * N + i))
                            : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int q = 0; q < 8; ++q) { s.x += a[q].x; s.y += a[q].y; s.z += a[q].z; s.w += a[q].w; }
      }
      *reinterpret_cast<float4*>(dst + i) = make_float4(s.x * inv_h, s.y * inv_h, s.z * inv_h, s.w * inv_h);
    }
    return;
  }
  for (int i = threadIdx.x; i < N; i += 256) {
    float s = 0.f;
    for (int h0 = 0; h0 < H; h0 += 8) {      // eight heads in flight, added in head order
      float a[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) a[q] = h0 + q < H ? __ldg(src + (size_t)(h0 + q) * M * N + i) : 0.f;
#pragma unroll
      for (int q = 0; q < 8; ++q) s += a[q];
    }
    dst[i] = s * inv_h;
  }
}

// ---------------------------------------------------------------------------------------
// Local penalty + top-N^S selection of one image by `nthr` threads (tid 0..nthr-1) that
// synchronise on hardware barrier `bar`.
//   1. every alive token bids (score key, lower index wins ties) for its window with a
//      64-bit shared-memory max; the winner's score is multiplied by `coef`;
//   2. an 8-bit-per-pass radix select over order-preserving keys finds the N^S-th largest
//      score; ties at the threshold go to the lower index;
//   3. a block scan turns the membership flags into ascending index lists S and T, the kept
//      row indices and the surviving grid positions.
// The code runs once per image, so it is kept compact (rolled loops, not inlined): a long
// unrolled body would be paid for in instruction-cache misses.
// `work` is a shared-memory area of select_work_bytes(np, windows) bytes: the scores and grid
// positions are read from global memory once and kept there with the keys and window bids.
// ---------------------------------------------------------------------------------------
__host__ __device__ inline size_t select_work_bytes(int np, int nwin) {
  return (size_t)np * 12 + 8 + (size_t)nwin * 8 + 16 + 4 * 256 * sizeof(int);
}

struct SelectShared {
  int warp_tot[33];
  uint32_t prefix;
  int remaining;
};

__device__ __noinline__ void select_image(
    const ImgDesc& d, const float* s_raw, const int* __restrict__ pos, int window, float coef,
    int penalty, float* __restrict__ s_pen, float* __restrict__ scores_out, int* __restrict__ S_idx,
    int* __restrict__ T_idx, int* __restrict__ kept_idx, int* __restrict__ pos_out,
    unsigned* __restrict__ status, unsigned char* work, SelectShared& sh, int tid, int nthr, int bar) {
  const int np = d.np;
  uint32_t* keys = reinterpret_cast<uint32_t*>(work);
  float* sc = reinterpret_cast<float*>(work + (size_t)np * 4);
  int* pp = reinterpret_cast<int*>(work + (size_t)np * 8);
  unsigned long long* win = reinterpret_cast<unsigned long long*>(work + (((size_t)np * 12 + 7) & ~(size_t)7));
  const int nwc = (d.gw + window - 1) / window;
  const int nwr = (d.gh + window - 1) / window;
  const int nwin = penalty ? nwc * nwr : 0;
  // [4][256], one histogram per digit, 16-byte aligned
  int* hist = reinterpret_cast<int*>((reinterpret_cast<uintptr_t>(win + nwin) + 15) & ~(uintptr_t)15);

  #pragma unroll 1
  for (int i = tid; i < 4 * 256; i += nthr) hist[i] = 0;
  #pragma unroll 1
  for (int i = tid; i < nwin; i += nthr) win[i] = 0ull;
  #pragma unroll 1
  for (int i0 = tid; i0 < np; i0 += 4 * nthr) {    // four tokens' loads in flight per thread
    float a[4];
    int q[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = i0 + j * nthr;
      a[j] = i < np ? __ldcg(s_raw + d.patch0 + i) : 0.f;
      q[j] = (i < np && pos) ? pos[d.patch0 + i] : i;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = i0 + j * nthr;
      if (i < np) { sc[i] = a[j]; pp[i] = q[j]; }
    }
  }
  cta_sync(bar, nthr);

  // ---- local penalty ------------------------------------------------------------------
  if (penalty) {
    #pragma unroll 1
    for (int i = tid; i < np; i += nthr) {
      const int p = pp[i];
      if (p < 0 || p >= d.gh * d.gw) { atomicOr(status, STATUS_POS_RANGE); continue; }
      const int wid = (p / d.gw / window) * nwc + (p % d.gw) / window;
      const unsigned long long bid =
          ((unsigned long long)order_key(sc[i]) << 32) | (unsigned)(0xFFFFFFFFu - (unsigned)i);
      atomicMax(&win[wid], bid);
    }
    cta_sync(bar, nthr);
  }
  #pragma unroll 1
  for (int i = tid; i < np; i += nthr) {
    float s = sc[i];
    if (penalty) {
      const int p = pp[i];
      if (p >= 0 && p < d.gh * d.gw) {
        const int wid = (p / d.gw / window) * nwc + (p % d.gw) / window;
        if ((unsigned)(win[wid] & 0xFFFFFFFFull) == 0xFFFFFFFFu - (unsigned)i) s *= coef;
      }
    }
    s_pen[d.patch0 + i] = s;
    if (scores_out) scores_out[d.patch0 + i] = s;
    keys[i] = order_key(s);
  }
  cta_sync(bar, nthr);

  // ---- radix select: key of the n_src-th largest ------------------------------------------
  // Two barriers per digit: count, then the first warp finds the digit's bin; every digit has a
  // histogram of its own, zeroed up front.
  const int k = d.n_src;
  uint32_t thr = 0;       // threshold key
  int need_eq = 0;        // how many keys equal to thr are selected (lowest indices)
  if (k > 0 && k < np) {
    const int lane = tid & 31;
    uint32_t prefix = 0, mask = 0;
    int remaining = k;
    #pragma unroll 1
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      int* h = hist + 256 * pass;
      #pragma unroll 1
      for (int i = tid; i < np; i += nthr) {
        const uint32_t key = keys[i];
        if ((key & mask) == prefix) atomicAdd(&h[(key >> shift) & 255], 1);
      }
      cta_sync(bar, nthr);
      if (tid < 32) {
        // lane l owns bins 255-8l .. 248-8l (descending); find where the running count from
        // the top reaches `remaining`
        int c[8], tot = 0;
        {
          const int4 lo = *reinterpret_cast<const int4*>(h + 248 - 8 * lane);
          const int4 hi = *reinterpret_cast<const int4*>(h + 252 - 8 * lane);
          c[0] = hi.w; c[1] = hi.z; c[2] = hi.y; c[3] = hi.x;
          c[4] = lo.w; c[5] = lo.z; c[6] = lo.y; c[7] = lo.x;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) tot += c[j];
        int inc = tot;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          int n = __shfl_up_sync(0xFFFFFFFFu, inc, o);
          if (lane >= o) inc += n;
        }
        const int before = inc - tot;
        if (before < remaining && inc >= remaining) {
          int cum = before;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            if (cum < remaining && cum + c[j] >= remaining) {
              sh.prefix = prefix | ((uint32_t)(255 - 8 * lane - j) << shift);
              sh.remaining = remaining - cum;
            }
            cum += c[j];
          }
        }
      }
      cta_sync(bar, nthr);
      prefix = sh.prefix;
      remaining = sh.remaining;
      mask |= 0xFFu << shift;
    }
    thr = prefix;
    need_eq = remaining;
  }

  // ---- ordered compaction into S and T ------------------------------------------------------
  // Each thread takes a run of consecutive tokens; one block scan over packed counts
  // (greater-than in the high half, equal in the low half) places every run.
  {
    const int ipt = (np + nthr - 1) / nthr;
    const int i_lo = min(np, tid * ipt), i_hi = min(np, i_lo + ipt);
    int n_gt = 0, n_eq = 0;
    #pragma unroll 1
    for (int i = i_lo; i < i_hi; ++i) {
      const uint32_t key = keys[i];
      if (k >= np) ++n_gt;
      else if (k > 0) { n_gt += key > thr ? 1 : 0; n_eq += key == thr ? 1 : 0; }
    }
    int tot;
    const int packed = block_exclusive_scan((n_gt << 16) | n_eq, sh.warp_tot, &tot, bar, nthr);
    int gt_before = packed >> 16, eq_before = packed & 0xFFFF;
    #pragma unroll 1
    for (int i = i_lo; i < i_hi; ++i) {
      const uint32_t key = keys[i];
      bool gt, eq;
      if (k <= 0) { gt = false; eq = false; }
      else if (k >= np) { gt = true; eq = false; }
      else { gt = key > thr; eq = key == thr; }
      const bool sel = gt || (eq && eq_before < need_eq);
      const int sel_rank = gt_before + min(eq_before, need_eq);   // selected tokens before i
      if (sel) {
        S_idx[d.src0 + sel_rank] = i;
      } else {
        const int tp = i - sel_rank;
        T_idx[d.tgt0 + tp] = i;
        kept_idx[d.out_row0 + d.n_cls + tp] = d.n_cls + i;
        if (pos_out) pos_out[d.tgt0 + tp] = pp[i];
      }
      gt_before += gt ? 1 : 0;
      eq_before += eq ? 1 : 0;
    }
  }
  #pragma unroll 1
  for (int i = tid; i < d.n_cls; i += nthr) kept_idx[d.out_row0 + i] = i;
  #pragma unroll 1
  for (int i = tid; i < d.n_tail; i += nthr)
    kept_idx[d.out_row0 + d.n_cls + d.n_tgt + d.n_extra + i] = d.n_cls + np + i;
  if (tid == 0 && d.n_extra) kept_idx[d.out_row0 + d.n_cls + d.n_tgt] = -1;
}

// ---------------------------------------------------------------------------------------
// The same step for images of up to SEL_SMALL_MAX tokens by exactly 512 threads, two tokens per
// thread held in registers, built for a short critical path (seven or eight barriers, no
// contended atomics):
//   1. scores and grid positions are loaded once; a grid-cell -> token map in shared memory lets
//      one thread per window pick the window's maximum (lower token index on equal scores) and
//      multiply it in place;
//   2. keys are made dense: key - min key, shifted so that the largest has its top bit set, so the
//      first radix digit already spreads the tokens over its 256 bins (raw fp32 keys of one
//      image share sign and exponent and would all hit one bin); every warp reads the histogram
//      and finds the digit by itself, so a pass costs one barrier; passes that could only see
//      zero bits are skipped;
//   3. membership flags become ascending positions with two ballots per warp and one 32-entry
//      table of per-warp counts.
// Only the outputs of tokens w_lo <= i < w_hi are written (plus the CLS / trailing entries of
// kept_idx when w_lo == 0), so the CTAs that scored an image can each run the selection and
// write their own slice.  select_small_prepare() zeroes the work area; a barrier (or any
// inter-CTA wait that ends in one) must separate it from select_small().
// ---------------------------------------------------------------------------------------
constexpr int SEL_SMALL_MAX = 1024;
constexpr int SEL_SMALL_THREADS = 512;

struct SelectSmallShared {
  uint32_t wmin[16], wmax[16];
  int cnt[32];
};

__host__ __device__ inline size_t select_small_bytes(int np, int cells) {
  return (size_t)np * 8 + 16 + 4 * 256 * sizeof(int) + (size_t)cells * 2 + 16;
}

struct SelectSmallWork {
  float* sc;        // [np] scores (penalised in place)
  uint32_t* nk;     // [np] dense keys
  int* hist;        // [4][256]
  short* cell;      // [gh * gw] token of every grid cell, -1 = no alive token
};
__device__ __forceinline__ SelectSmallWork select_small_layout(unsigned char* work, int np) {
  SelectSmallWork w;
  w.sc = reinterpret_cast<float*>(work);
  w.nk = reinterpret_cast<uint32_t*>(work + (size_t)np * 4);
  w.hist = reinterpret_cast<int*>((reinterpret_cast<uintptr_t>(work + (size_t)np * 8) + 15) & ~(uintptr_t)15);
  w.cell = reinterpret_cast<short*>(w.hist + 4 * 256);
  return w;
}

__device__ __forceinline__ void select_small_prepare(const ImgDesc& d, int penalty, unsigned char* work, int tid) {
  const SelectSmallWork w = select_small_layout(work, d.np);
  w.hist[tid] = 0;
  w.hist[tid + SEL_SMALL_THREADS] = 0;
  if (penalty) {
    const int cells = d.gh * d.gw;
    #pragma unroll 1
    for (int c = tid; c < cells; c += SEL_SMALL_THREADS) w.cell[c] = -1;
  }
}

__device__ __noinline__ void select_small(
    const ImgDesc& d, const float* s_raw, const int* __restrict__ pos, int window, float coef,
    int penalty, float* __restrict__ s_pen, float* __restrict__ scores_out, int* __restrict__ S_idx,
    int* __restrict__ T_idx, int* __restrict__ kept_idx, int* __restrict__ pos_out,
    unsigned* __restrict__ status, unsigned char* work, SelectSmallShared& sh, int tid, int bar,
    int w_lo, int w_hi) {
  constexpr int NT = SEL_SMALL_THREADS;
  const int np = d.np, lane = tid & 31, warp = tid >> 5;
  const SelectSmallWork wk = select_small_layout(work, np);
  const int cells = d.gh * d.gw;
  float s[2];
  int pp[2];
  bool on[2];
#pragma unroll
  for (int q = 0; q < 2; ++q) {
    const int i = tid + NT * q;
    on[q] = i < np;
    s[q] = on[q] ? __ldcg(s_raw + d.patch0 + i) : 0.f;
    pp[q] = on[q] ? (pos ? pos[d.patch0 + i] : i) : -1;
  }
#pragma unroll
  for (int q = 0; q < 2; ++q) {
    const int i = tid + NT * q;
    if (!on[q]) continue;
    wk.sc[i] = s[q];
    if (penalty) {
      if (pp[q] >= 0 && pp[q] < cells) wk.cell[pp[q]] = (short)i;
      else atomicOr(status, STATUS_POS_RANGE);
    }
  }
  cta_sync(bar, NT);

  // ---- local penalty: one thread per window ------------------------------------------------
  if (penalty) {
    const int nwc = (d.gw + window - 1) / window, nwr = (d.gh + window - 1) / window;
    #pragma unroll 1
    for (int wdx = tid; wdx < nwc * nwr; wdx += NT) {
      const int r0 = (wdx / nwc) * window, c0 = (wdx % nwc) * window;
      const int r1 = min(d.gh, r0 + window), c1 = min(d.gw, c0 + window);
      int best = -1;
      float bs = 0.f;
      #pragma unroll 1
      for (int r = r0; r < r1; ++r)
        #pragma unroll 1
        for (int c = c0; c < c1; ++c) {
          const int t = wk.cell[r * d.gw + c];
          if (t < 0) continue;
          const float v = wk.sc[t];
          if (best < 0 || v > bs || (v == bs && t < best)) { best = t; bs = v; }
        }
      if (best >= 0) wk.sc[best] = bs * coef;      // windows are disjoint: nobody else touches this token
    }
    cta_sync(bar, NT);
  }

  // ---- keys, their range, dense keys -----------------------------------------------------------
  uint32_t key[2];
  uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;
#pragma unroll
  for (int q = 0; q < 2; ++q) {
    const int i = tid + NT * q;
    if (on[q]) {
      s[q] = wk.sc[i] + 0.0f;                      // -0 and +0 are one score
      key[q] = order_key(s[q]);
      kmin = min(kmin, key[q]);
      kmax = max(kmax, key[q]);
      if (i >= w_lo && i < w_hi) {
        s_pen[d.patch0 + i] = s[q];
        if (scores_out) scores_out[d.patch0 + i] = s[q];
      }
    } else {
      key[q] = 0u;
    }
  }
  kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
  kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
  if (lane == 0) { sh.wmin[warp] = kmin; sh.wmax[warp] = kmax; }
  cta_sync(bar, NT);
  {
    const uint32_t a = sh.wmin[lane & 15], b = sh.wmax[lane & 15];
    kmin = __reduce_min_sync(0xFFFFFFFFu, a);
    kmax = __reduce_max_sync(0xFFFFFFFFu, b);
  }
  const int k = d.n_src;
  const uint32_t range = kmax - kmin;
  const int sh_l = range ? __clz(range) : 0;
  uint32_t nk[2];
#pragma unroll
  for (int q = 0; q < 2; ++q) {
    nk[q] = range ? (key[q] - kmin) << sh_l : 0u;
    if (on[q]) wk.nk[tid + NT * q] = nk[q];
  }

  // ---- radix select on the dense keys: the n_src-th largest -------------------------------------
  uint32_t thr = 0;      // threshold (dense key)
  int need_eq = 0;       // how many of the keys equal to thr are selected (lowest indices)
  int c_eq = 0;          // how many keys equal thr
  uint32_t thr_mask = 0xFFFFFFFFu;   // digits of the dense keys the passes have looked at
  if (k > 0 && k < np) {
    const int npass = range ? (32 - sh_l + 7) / 8 : 1;   // the low sh_l bits of every dense key are zero
    uint32_t prefix = 0, mask = 0;
    int remaining = k;
    #pragma unroll 1
    for (int pass = 0; pass < npass; ++pass) {
      const int shift = 24 - 8 * pass;
      int* h = wk.hist + 256 * pass;
#pragma unroll
      for (int q = 0; q < 2; ++q)
        if (on[q] && (nk[q] & mask) == prefix) atomicAdd(&h[(nk[q] >> shift) & 255], 1);
      cta_sync(bar, NT);
      // every warp: lane l owns bins 255-8l .. 248-8l (descending); find where the running count
      // from the top reaches `remaining`
      int c[8], tot = 0;
      {
        const int4 lo = *reinterpret_cast<const int4*>(h + 248 - 8 * lane);
        const int4 hi = *reinterpret_cast<const int4*>(h + 252 - 8 * lane);
        c[0] = hi.w; c[1] = hi.z; c[2] = hi.y; c[3] = hi.x;
        c[4] = lo.w; c[5] = lo.z; c[6] = lo.y; c[7] = lo.x;
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) tot += c[j];
      int inc = tot;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += n;
      }
      const int before = inc - tot;
      const bool mine = before < remaining && inc >= remaining;
      int digit = 0, rem_new = 0, ceq_new = 0;
      if (mine) {
        int cum = before;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (cum < remaining && cum + c[j] >= remaining) {
            digit = 255 - 8 * lane - j;
            rem_new = remaining - cum;
            ceq_new = c[j];
          }
          cum += c[j];
        }
      }
      const int src = __ffs(__ballot_sync(0xFFFFFFFFu, mine)) - 1;   // exactly one lane (0 < remaining <= total)
      digit = __shfl_sync(0xFFFFFFFFu, digit, src);
      remaining = __shfl_sync(0xFFFFFFFFu, rem_new, src);
      c_eq = __shfl_sync(0xFFFFFFFFu, ceq_new, src);
      prefix |= (uint32_t)digit << shift;
      mask |= 0xFFu << shift;
      if (remaining == c_eq) break;    // every key that shares these digits is selected: no need to tell them apart
    }
    thr = prefix;
    need_eq = remaining;
    thr_mask = mask;
  }

  // ---- membership ---------------------------------------------------------------------------------
  bool sel[2];
#pragma unroll
  for (int q = 0; q < 2; ++q) {
    const int i = tid + NT * q;
    if (!on[q]) sel[q] = false;
    else if (k <= 0) sel[q] = false;
    else if (k >= np) sel[q] = true;
    else if ((nk[q] & thr_mask) != thr) sel[q] = (nk[q] & thr_mask) > thr;
    else if (need_eq >= c_eq) sel[q] = true;
    else {
      // equal scores straddle the boundary: the lowest indices among them are taken
      // (all passes were made, so the mask covers every bit that is set in any key)
      int before = 0;
      #pragma unroll 1
      for (int j = 0; j < i; ++j) before += wk.nk[j] == thr ? 1 : 0;
      sel[q] = before < need_eq;
    }
  }

  // ---- ascending positions ------------------------------------------------------------------------
  const unsigned b0 = __ballot_sync(0xFFFFFFFFu, sel[0]), b1 = __ballot_sync(0xFFFFFFFFu, sel[1]);
  if (lane == 0) { sh.cnt[warp] = __popc(b0); sh.cnt[16 + warp] = __popc(b1); }
  cta_sync(bar, NT);
  {
    const int mycnt = sh.cnt[lane];
    int inc = mycnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xFFFFFFFFu, inc, o);
      if (lane >= o) inc += n;
    }
    const int excl = inc - mycnt;                 // selected tokens in the 32-token groups before group `lane`
    const unsigned lt = (1u << lane) - 1u;
    const int rank0 = __shfl_sync(0xFFFFFFFFu, excl, warp) + __popc(b0 & lt);
    const int rank1 = __shfl_sync(0xFFFFFFFFu, excl, 16 + warp) + __popc(b1 & lt);
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const int i = tid + NT * q;
      if (!on[q] || i < w_lo || i >= w_hi) continue;
      const int rank = q ? rank1 : rank0;          // selected tokens with a lower index
      if (sel[q]) {
        S_idx[d.src0 + rank] = i;
      } else {
        const int tp = i - rank;
        T_idx[d.tgt0 + tp] = i;
        kept_idx[d.out_row0 + d.n_cls + tp] = d.n_cls + i;
        if (pos_out) pos_out[d.tgt0 + tp] = pp[q];
      }
    }
  }
  if (w_lo == 0) {
    #pragma unroll 1
    for (int i = tid; i < d.n_cls; i += NT) kept_idx[d.out_row0 + i] = i;
    #pragma unroll 1
    for (int i = tid; i < d.n_tail; i += NT)
      kept_idx[d.out_row0 + d.n_cls + d.n_tgt + d.n_extra + i] = d.n_cls + np + i;
    if (tid == 0 && d.n_extra) kept_idx[d.out_row0 + d.n_cls + d.n_tgt] = -1;
  }
}

// One CTA (512 or 1024 threads) per image.
__global__ void __launch_bounds__(1024) k_select(const ImgDesc* __restrict__ desc,
                                                 const float* __restrict__ s_raw,
                                                 const int* __restrict__ pos, int window, float coef,
                                                 int penalty, float* __restrict__ s_pen,
                                                 float* __restrict__ scores_out,
                                                 int* __restrict__ S_idx, int* __restrict__ T_idx,
                                                 int* __restrict__ kept_idx, int* __restrict__ pos_out,
                                                 unsigned* __restrict__ status) {
  extern __shared__ unsigned char sm_raw[];
  __shared__ SelectShared sh;
  __shared__ SelectSmallShared shs;
  const ImgDesc d = desc[blockIdx.x];
  if (d.np <= SEL_SMALL_MAX && blockDim.x == SEL_SMALL_THREADS) {
    select_small_prepare(d, penalty, sm_raw, threadIdx.x);
    __syncthreads();
    select_small(d, s_raw, pos, window, coef, penalty, s_pen, scores_out, S_idx, T_idx, kept_idx, pos_out,
                 status, sm_raw, shs, threadIdx.x, 0, 0, d.np);
    return;
  }
  select_image(d, s_raw, pos, window, coef, penalty, s_pen, scores_out, S_idx, T_idx, kept_idx, pos_out,
               status, sm_raw, sh, threadIdx.x, (int)blockDim.x, 0);
}

}  // namespace ficoco
