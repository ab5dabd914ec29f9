// Correlate stage: C_ij for i in S, j in T, per-row top list, tau_i, J_i, alpha_ij.
#pragma once
#include <limits.h>
#include <math_constants.h>
#include "async_ops.cuh"
#include "common.cuh"

namespace ficoco {

constexpr int CBM = 64;   // source rows per CTA
constexpr int CBN = 64;   // target columns per tile
constexpr int CKC = 16;   // reduction chunk
constexpr int CPG = 4;    // reduction chunks fetched together (one group in flight ahead of the multiply)

// Four consecutive elements of a token row as fp32 (16-byte / 8-byte aligned).
__device__ __forceinline__ float4 load4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
  const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
  return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xFFFF0000u), __uint_as_float(v.y << 16),
                     __uint_as_float(v.y & 0xFFFF0000u));
}

template <int LC>
__device__ __forceinline__ void correlate_tail(
    const ImgDesc& d, const WorkItem& w, int tile, int* __restrict__ tile_done,
    const float* __restrict__ part_val,
    const int* __restrict__ part_idx, int* __restrict__ corr_cnt, float* __restrict__ tau_out,
    int* __restrict__ e_tgt, float* __restrict__ e_w, float* __restrict__ e_c, int* is_last_smem);

// ---------------------------------------------------------------------------------------
// fp32 SIMT correlate (the path for fp32 tokens, where 1e-5 relative accuracy rules out
// bf16 tensor-core products).  One CTA owns up to 64 discarded tokens of one image and one
// column split of that image's preserved tokens; it walks the split in 64-column tiles,
// forms C = gamma * rn_i rn_j (x_i . x_j) [+ (1-gamma)/M * sum_k t_ki t_kj] in registers
// (4x4 per thread) and keeps, per row, the L largest entries (value, position in T).
// The N^S x N^T matrix never leaves the SM.
// ---------------------------------------------------------------------------------------
template <class T>
__global__ void __launch_bounds__(256) k_correlate_simt(
    const T* __restrict__ tokens, int D, const ImgDesc* __restrict__ desc,
    const WorkItem* __restrict__ work, const float* __restrict__ rn,
    const int* __restrict__ S_idx, const int* __restrict__ T_idx,
    const float* __restrict__ tmean, int M, float gamma,
    float* __restrict__ part_val, int* __restrict__ part_idx, int* __restrict__ img_done,
    int* __restrict__ corr_cnt, float* __restrict__ tau_out, int* __restrict__ e_tgt,
    float* __restrict__ e_w, float* __restrict__ e_c, unsigned* __restrict__ status) {
  __shared__ int is_last;
  __shared__ __align__(16) float As[CKC][CBM + 4];
  __shared__ __align__(16) float Bs[CKC][CBN + 4];
  __shared__ float Cs[CBM][CBN + 1];
  __shared__ float lv[CBM][KCAP];
  __shared__ int li[CBM][KCAP];
  __shared__ int rowS[CBM], rowT[CBN];
  __shared__ float rnS[CBM], rnT[CBN];

  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  const int L = d.list_len;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;

  for (int i = tid; i < CBM * KCAP; i += 256) {
    (&lv[0][0])[i] = -CUDART_INF_F;
    (&li[0][0])[i] = INT_MAX;
  }
  if (tid < CBM) {
    const bool ok = tid < w.nrows;
    const int p = ok ? checked_index(S_idx[d.src0 + w.r0 + tid], d.np, status) : -1;
    rowS[tid] = p;
    rnS[tid] = ok ? rn[d.patch0 + p] : 0.f;
  }
  const int col_begin = w.aux * d.cols_per_split;
  const int col_end = min(d.n_tgt, col_begin + d.cols_per_split);
  const size_t tok0 = (size_t)(d.row0 + d.n_cls);
  const int N = d.np;

  for (int c0 = col_begin; c0 < col_end; c0 += CBN) {
    __syncthreads();
    if (tid < CBN) {
      const int c = c0 + tid;
      const bool ok = c < col_end;
      const int p = ok ? checked_index(T_idx[d.tgt0 + c], d.np, status) : -1;
      rowT[tid] = p;
      rnT[tid] = ok ? rn[d.patch0 + p] : 0.f;
    }
    __syncthreads();

    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    const int lr = tid >> 2, lq = tid & 3;
    // Operands are fetched CPG reduction chunks at a time, one group ahead of the one being
    // multiplied: a chunk per round trip to L2 made the loop pure latency (64 round trips for
    // D = 1024).
    const int pa = rowS[lr], pb = rowT[lr];
    const T* rowA = tokens + (tok0 + (pa >= 0 ? pa : 0)) * D;
    const T* rowB = tokens + (tok0 + (pb >= 0 ? pb : 0)) * D;
    auto load_group = [&](int k0, float4 (&fa)[CPG], float4 (&fb)[CPG]) {
#pragma unroll
      for (int g = 0; g < CPG; ++g) {
        const int kk = k0 + g * CKC + lq * 4;
        fa[g] = (kk < D && pa >= 0) ? load4(rowA + kk) : make_float4(0.f, 0.f, 0.f, 0.f);
        fb[g] = (kk < D && pb >= 0) ? load4(rowB + kk) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    };
    float4 ca[CPG], cb[CPG], na[CPG], nb[CPG];
    load_group(0, ca, cb);
    #pragma unroll 1
    for (int k0 = 0; k0 < D; k0 += CPG * CKC) {
      if (k0 + CPG * CKC < D) load_group(k0 + CPG * CKC, na, nb);
#pragma unroll
      for (int g = 0; g < CPG; ++g) {
        if (k0 + g * CKC < D) {
          As[lq * 4 + 0][lr] = ca[g].x; As[lq * 4 + 1][lr] = ca[g].y; As[lq * 4 + 2][lr] = ca[g].z; As[lq * 4 + 3][lr] = ca[g].w;
          Bs[lq * 4 + 0][lr] = cb[g].x; Bs[lq * 4 + 1][lr] = cb[g].y; Bs[lq * 4 + 2][lr] = cb[g].z; Bs[lq * 4 + 3][lr] = cb[g].w;
          __syncthreads();
#pragma unroll
          for (int kk = 0; kk < CKC; ++kk) {
            const float4 a = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
            const float4 b = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
              for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
          }
          __syncthreads();
        }
      }
#pragma unroll
      for (int g = 0; g < CPG; ++g) { ca[g] = na[g]; cb[g] = nb[g]; }
    }

    float cval[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) cval[i][j] = gamma * (rnS[ty * 4 + i] * rnT[tx * 4 + j]) * acc[i][j];

    if (tmean != nullptr) {
      // text-bridged term: (1-gamma)/M * sum_k t[k, i] t[k, j]
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
      const float* tb = tmean + (size_t)w.img * M * N;
      for (int k0 = 0; k0 < M; k0 += CKC) {
        for (int idx = tid; idx < CKC * CBM; idx += 256) {
          const int kk = idx / CBM, r = idx % CBM;
          const bool kin = k0 + kk < M;
          const int pa = rowS[r], pb = rowT[r];
          As[kk][r] = (kin && pa >= 0) ? __ldg(tb + (size_t)(k0 + kk) * N + pa) : 0.f;
          Bs[kk][r] = (kin && pb >= 0) ? __ldg(tb + (size_t)(k0 + kk) * N + pb) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < CKC; ++kk) {
          const float4 a = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
          const float4 b = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
          const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
          for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
      }
      const float sc = (1.0f - gamma) / (float)M;
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) cval[i][j] = fmaf(sc, acc[i][j], cval[i][j]);
    }

#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) Cs[ty * 4 + i][tx * 4 + j] = cval[i][j];
    __syncthreads();

    if (tid < w.nrows) {
      const int ncol = min(CBN, col_end - c0);
      for (int c = 0; c < ncol; ++c) {
        const float val = Cs[tid][c];
        const int idx = c0 + c;
        if (toplist_better(val, idx, lv[tid][L - 1], li[tid][L - 1]))
          toplist_insert(lv[tid], li[tid], L, val, idx);
      }
    }
  }
  __syncthreads();
  for (int i = tid; i < w.nrows * L; i += 256) {
    const int r = i / L, k = i % L;
    const size_t o = (size_t)d.part0 + ((size_t)(w.r0 + r) * d.nsplit + w.aux) * L + k;
    part_val[o] = lv[r][k];
    part_idx[o] = li[r][k] == INT_MAX ? -1 : li[r][k];
  }
  correlate_tail<KCAP>(d, w, (int)blockIdx.x - w.aux, img_done, part_val, part_idx, corr_cnt, tau_out, e_tgt, e_w, e_c, &is_last);
}

}  // namespace ficoco

namespace ficoco {

// ---------------------------------------------------------------------------------------
// One thread per discarded token: merge the column splits' partial top lists, then
//   tau_i = v[L-1] + frac * (v[L-2] - v[L-1])  (v descending: the two order statistics around
//   eps*(n-1)), J_i = { entries >= tau_i }, alpha_ij = C+_ij / sum_{J_i} C+  (Eq. 2).
// Results go to compact per-image arrays with L slots per token: e_tgt (position in T, or -1),
// e_w (alpha), e_c (the L largest C, descending).
// grid = (images, ceil(max N^S / 256)).
// ---------------------------------------------------------------------------------------
// LC: compile-time bound on the list length L of the image (lists live in registers).
template <int LC>
__device__ __forceinline__ void finalize_source(
    const ImgDesc& d, int s, const float* __restrict__ part_val, const int* __restrict__ part_idx,
    int* __restrict__ corr_cnt, float* __restrict__ tau_out, int* __restrict__ e_tgt,
    float* __restrict__ e_w, float* __restrict__ e_c) {
  const int L = d.list_len;
  const size_t o = (size_t)(d.src0 + s);
  if (L == 0) { corr_cnt[o] = 0; tau_out[o] = 0.f; return; }
  float v[LC];
  int ix[LC];
#pragma unroll
  for (int k = 0; k < LC; ++k) { v[k] = -CUDART_INF_F; ix[k] = INT_MAX; }
  const size_t pbase = (size_t)d.part0 + (size_t)s * d.nsplit * L;
  const int ne = d.nsplit * L;
#pragma unroll 1
  for (int e0 = 0; e0 < ne; e0 += 4) {
    // four entries of the partial lists in flight at a time: the insertion below is unrolled per entry,
    // and a longer body costs more in instruction fetch than the extra round trips (eight at a time:
    // +0.25 us per step on 32 x 577 tokens, +7 us on 8 x 2881; sixteen: +0.9 and +25 us)
    float pv[4];
    int pi[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const bool on = e0 + j < ne;
      pv[j] = on ? __ldcg(part_val + pbase + e0 + j) : 0.f;
      pi[j] = on ? __ldcg(part_idx + pbase + e0 + j) : -1;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float cv = pv[j];
      int ci = pi[j];
      if (ci < 0) continue;
#pragma unroll
      for (int k = 0; k < LC; ++k) {
        if (k < L && toplist_better(cv, ci, v[k], ix[k])) {
          const float tv = v[k]; const int ti = ix[k];
          v[k] = cv; ix[k] = ci; cv = tv; ci = ti;
        }
      }
    }
  }
  float vl1 = 0.f, vl2 = 0.f;
#pragma unroll
  for (int k = 0; k < LC; ++k) {
    if (k == L - 1) vl1 = v[k];
    if (k == L - 2) vl2 = v[k];
  }
  const float tau = (L >= 2) ? vl1 + d.frac * (vl2 - vl1) : vl1;
  int nj = 0;
  float den = 0.f;
  bool open = true;
#pragma unroll
  for (int k = 0; k < LC; ++k) {
    if (k < L && open) {
      if (ix[k] != INT_MAX && v[k] >= tau) { ++nj; den += fmaxf(v[k], 0.f); } else open = false;
    }
  }
  if (!d.avg && !(den > 1e-12f)) nj = 0;
  corr_cnt[o] = nj;
  tau_out[o] = tau;
  const size_t eb = (size_t)d.ent0 + (size_t)s * L;
#pragma unroll
  for (int k = 0; k < LC; ++k) {
    if (k < L) {
      e_tgt[eb + k] = k < nj ? ix[k] : -1;
      e_w[eb + k] = k < nj ? (d.avg ? 1.0f : fmaxf(v[k], 0.f) / den) : 0.f;
      e_c[eb + k] = v[k];
    }
  }
}

__global__ void __launch_bounds__(256) k_finalize_src(
    const ImgDesc* __restrict__ desc, const float* __restrict__ part_val,
    const int* __restrict__ part_idx, int* __restrict__ corr_cnt, float* __restrict__ tau_out,
    int* __restrict__ e_tgt, float* __restrict__ e_w, float* __restrict__ e_c) {
  const ImgDesc d = desc[blockIdx.x];
  const int s = blockIdx.y * 256 + threadIdx.x;
  if (s >= d.n_src) return;
  finalize_source<KCAP>(d, s, part_val, part_idx, corr_cnt, tau_out, e_tgt, e_w, e_c);
}

// Tail of a correlate CTA: once its partial lists are written it bumps the counter of its
// source tile (`tile` = index of the tile's first work item); the CTA that completes the tile
// (the last of its d.nsplit column splits) turns the partial lists of the tile's discarded
// tokens into tau_i, J_i and alpha_ij, and resets the counter.  Nobody waits: there is no
// spinning.  Call from all threads of the CTA.
template <int LC>
__device__ __forceinline__ void correlate_tail(
    const ImgDesc& d, const WorkItem& w, int tile, int* __restrict__ tile_done,
    const float* __restrict__ part_val,
    const int* __restrict__ part_idx, int* __restrict__ corr_cnt, float* __restrict__ tau_out,
    int* __restrict__ e_tgt, float* __restrict__ e_w, float* __restrict__ e_c, int* is_last_smem) {
  __syncthreads();
  if (threadIdx.x == 0) {
    // publishes this CTA's partial lists and, for the split that arrives last, observes the others'
    const int old = atom_acq_rel_add(&tile_done[tile], 1);
    const int last = old == d.nsplit - 1;
    if (last) tile_done[tile] = 0;
    *is_last_smem = last;
  }
  __syncthreads();
  if (*is_last_smem)
    for (int s = w.r0 + (int)threadIdx.x; s < w.r0 + w.nrows; s += blockDim.x)
      finalize_source<LC>(d, s, part_val, part_idx, corr_cnt, tau_out, e_tgt, e_w, e_c);
}

}  // namespace ficoco
