// Compress + compact (Eq. 2 and the last step of Algorithm 1 / 2).
#pragma once
#include "common.cuh"

namespace ficoco {

constexpr int MHUB = 4;        // source rows a lane has in flight for a hub row
constexpr int MROWS = 32;      // most output rows a CTA can take (sizes of the per-row arrays)
constexpr int MROWS_CTA = 16;  // output rows per CTA the host plans (two per warp)
constexpr int MCOPY = MROWS_CTA / 8;   // rows a warp copies in one batch
constexpr int MLIST = 1024;    // (source, alpha) entries a CTA copies to shared memory (more are read in place)
constexpr int MHEAVY = 2;      // rows with more sources than this are split into 32-vector blocks over the warps
constexpr int MVB = 4;         // 16-byte vectors a lane accumulates at a time

// acc[b][.] += sum over list entries [k0, k1) of alpha * x, for the MVB vectors v0 + 32 b of
// each row; source rows are fetched four at a time so that 4 * MVB loads are in flight per lane.
template <class T>
__device__ __forceinline__ void merge_accumulate(float (&acc)[MVB][VecTraits<T>::E], const T* pbase, int D,
                                                 const int* lsrc, const float* lw, int k0, int k1,
                                                 int v0, int nvec) {
  constexpr int E = VecTraits<T>::E;
  #pragma unroll 1
  for (int k = k0; k < k1; k += 4) {
    uint4 u[4][MVB];
    float a[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const bool on = k + j < k1;
      const T* x = pbase + (size_t)lsrc[on ? k + j : k] * D;
      a[j] = on ? lw[k + j] : 0.f;
#pragma unroll
      for (int b = 0; b < MVB; ++b) {
        const int v = v0 + 32 * b;
        u[j][b] = (on && v < nvec) ? ldg16(x + (size_t)v * E) : make_uint4(0, 0, 0, 0);
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int b = 0; b < MVB; ++b) {
        float f[E];
        unpack(u[j][b], f, (const T*)nullptr);
#pragma unroll
        for (int q = 0; q < E; ++q) acc[b][q] = fmaf(a[j], f[q], acc[b][q]);
      }
  }
}

// Compress + compact.  A CTA owns up to 32 consecutive output rows of one image (warp w: rows
// w, w + 8, w + 16, w + 24).
//   1. every row resolves its input row (CLS / preserved token / trailing text row) and, for a
//      preserved token, the bounds of its segment in the per-target entry lists that the
//      correlate step left (ordered by token index, so the fp32 sums have one fixed order and no
//      atomics touch floats); the segments of consecutive rows are contiguous, so the CTA's
//      entries are one run, copied to shared memory (read in place when there are more than MLIST);
//   2. out_j = (x_j + sum_{i in I_j} alpha_ij x_i) / (1 + sum alpha_ij), rounded once:
//      rows without sources are copied in one batch, rows with few sources are merged by their
//      own warp; hub rows are cut into blocks of 32 vectors that are dealt to the warps, every
//      lane summing the sources of its vector in list order.
template <class T>
__global__ void __launch_bounds__(256) k_merge_csr(
    const T* __restrict__ tokens, int D, const ImgDesc* __restrict__ desc,
    const WorkItem* __restrict__ work, const int* __restrict__ T_idx,
    const int* __restrict__ seg_begin, const int* __restrict__ csr_src, const float* __restrict__ csr_w,
    T* __restrict__ out, int index_before_wait, const unsigned* __restrict__ status) {
  constexpr int E = VecTraits<T>::E;
  __shared__ int cnt[MROWS], beg[MROWS + 1], srow_s[MROWS];
  __shared__ int lsrc_s[MLIST];
  __shared__ float lw_s[MLIST];
  __shared__ int heavy_rows[MROWS];
  __shared__ int n_heavy, dead;
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nvec = D / E;
  const int tp_lo = max(w.r0 - d.n_cls, 0);
  const int tp_hi = min(w.r0 + w.nrows - d.n_cls, d.n_tgt);
  const int n_tp = (d.list_len > 0 && tp_hi > tp_lo) ? tp_hi - tp_lo : 0;   // target rows that may have sources
  const T* pbase = tokens + (size_t)(d.row0 + d.n_cls) * D;

  FICOCO_PHASE(2, 0);
  if (tid < MROWS) cnt[tid] = 0;
  if (tid == 0) n_heavy = 0;
  // When the grid before this one is a correlate grid, the filter grid (which wrote T_idx) had
  // completed before this grid could start, so the row lookup may overlap that
  // grid's tail; otherwise wait first.
  if (!index_before_wait) grid_dep_wait();
  if (tid < w.nrows) {
    const int orow = w.r0 + tid;
    int srow;
    if (orow < d.n_cls) srow = orow;
    else if (orow < d.n_cls + d.n_tgt) srow = d.n_cls + T_idx[d.tgt0 + orow - d.n_cls];
    else srow = d.n_cls + d.np + (orow - d.n_cls - d.n_tgt);
    srow_s[tid] = srow;
  }
  if (index_before_wait) grid_dep_wait();
  grid_dep_launch();   // correlate is complete: the next step's filter may stream its rows under our tail
  FICOCO_PHASE(2, 1);
  // a step whose filter or correlate grid gave up has no valid index lists: write nothing
  if (tid == 0) dead = (*reinterpret_cast<const volatile unsigned*>(status) & 4u) ? 1 : 0;
  if (tid <= n_tp && n_tp > 0) beg[tid] = __ldcg(seg_begin + d.tgt0 + w.img + tp_lo + tid);
  __syncthreads();
  if (dead) return;
  const int e0 = n_tp ? beg[0] : 0;
  const int total = n_tp ? beg[n_tp] - e0 : 0;
  const bool fits = total <= MLIST;
  const int* lsrc = csr_src + d.ent0 + e0;
  const float* lw = csr_w + d.ent0 + e0;
  if (fits) {
    for (int i = tid; i < total; i += 256) {
      lsrc_s[i] = __ldcg(lsrc + i);
      lw_s[i] = __ldcg(lw + i);
    }
    lsrc = lsrc_s;
    lw = lw_s;
  }
  if (tid < n_tp) {
    const int c = beg[tid + 1] - beg[tid];
    cnt[tid] = c;
    if (c > MHEAVY) heavy_rows[atomicAdd(&n_heavy, 1)] = tid;
  }
  __syncthreads();
  FICOCO_PHASE(2, 2);

  // ---- rows without sources: plain copies, all of a warp's rows in flight together --------------
  #pragma unroll 1
  for (int v0 = lane; v0 < nvec; v0 += 32 * MVB) {
    uint4 u[MCOPY][MVB];
#pragma unroll
    for (int j = 0; j < MCOPY; ++j) {
      const int r = warp + 8 * j;
      const int orow = w.r0 + r;
      const bool is_tgt = orow >= d.n_cls && orow < d.n_cls + d.n_tgt;
      const bool copy = r < w.nrows && (!is_tgt || cnt[orow - d.n_cls - tp_lo] == 0);
      const T* src = tokens + (size_t)(d.row0 + (r < w.nrows ? srow_s[r] : 0)) * D;
#pragma unroll
      for (int b = 0; b < MVB; ++b) {
        const int v = v0 + 32 * b;
        u[j][b] = (copy && v < nvec) ? ldg16(src + (size_t)v * E) : make_uint4(0, 0, 0, 0);
      }
    }
#pragma unroll
    for (int j = 0; j < MCOPY; ++j) {
      const int r = warp + 8 * j;
      const int orow = w.r0 + r;
      const bool is_tgt = orow >= d.n_cls && orow < d.n_cls + d.n_tgt;
      const bool copy = r < w.nrows && (!is_tgt || cnt[orow - d.n_cls - tp_lo] == 0);
      T* dst = out + (size_t)(d.out_row0 + orow) * D;
#pragma unroll
      for (int b = 0; b < MVB; ++b) {
        const int v = v0 + 32 * b;
        if (copy && v < nvec) reinterpret_cast<uint4*>(dst)[v] = u[j][b];
      }
    }
  }

  FICOCO_PHASE(2, 3);
  // ---- rows with a few sources: one warp per row --------------------------------------------------
  #pragma unroll 1
  for (int r = warp; r < w.nrows; r += 8) {
    const int orow = w.r0 + r;
    T* dst = out + (size_t)(d.out_row0 + orow) * D;
    const bool is_tgt = orow >= d.n_cls && orow < d.n_cls + d.n_tgt;
    const int li = is_tgt ? orow - d.n_cls - tp_lo : 0;
    const int n = is_tgt ? cnt[li] : 0;
    const T* src = tokens + (size_t)(d.row0 + srow_s[r]) * D;
    if (n == 0) {
      continue;
    } else if (n <= MHEAVY) {
      const int b0 = beg[li] - e0;
      float wsum = 0.f;
      for (int k = 0; k < n; ++k) wsum += lw[b0 + k];
      const float inv_den = 1.0f / (1.0f + wsum);   // one division per row, then multiplies
      #pragma unroll 1
      for (int v0 = lane; v0 < nvec; v0 += 32 * MVB) {
        float acc[MVB][E];
#pragma unroll
        for (int b = 0; b < MVB; ++b) {
          const int v = v0 + 32 * b;
          unpack(v < nvec ? ldg16(src + (size_t)v * E) : make_uint4(0, 0, 0, 0), acc[b], (const T*)nullptr);
        }
        merge_accumulate<T>(acc, pbase, D, lsrc, lw, b0, b0 + n, v0, nvec);
#pragma unroll
        for (int b = 0; b < MVB; ++b) {
          const int v = v0 + 32 * b;
          if (v < nvec) {
#pragma unroll
            for (int q = 0; q < E; ++q) acc[b][q] = acc[b][q] * inv_den;
            reinterpret_cast<uint4*>(dst)[v] = pack(acc[b], (const T*)nullptr);
          }
        }
      }
    }
  }

  FICOCO_PHASE(2, 4);
  // ---- hub rows: (row, block of 32 vectors) items dealt to the warps; each lane sums all the
  // sources of its one vector in list order, MHUB source rows in flight ---------------------
  const int nh = n_heavy;
  const int nblk = (nvec + 31) / 32;
  #pragma unroll 1
  for (int it = warp; it < nh * nblk; it += 8) {
    const int li = heavy_rows[it / nblk];
    const int v = (it % nblk) * 32 + lane;
    if (v >= nvec) continue;
    const int tp = tp_lo + li;
    const int b0 = beg[li] - e0, n = cnt[li];
    const T* src = tokens + (size_t)(d.row0 + srow_s[tp + d.n_cls - w.r0]) * D;
    T* dst = out + (size_t)(d.out_row0 + d.n_cls + tp) * D;
    float wsum = 0.f;
    for (int k = 0; k < n; ++k) wsum += lw[b0 + k];
    const float inv_den = 1.0f / (1.0f + wsum);
    float acc[E];
    unpack(ldg16(src + (size_t)v * E), acc, (const T*)nullptr);
    #pragma unroll 1
    for (int k = 0; k < n; k += MHUB) {
      uint4 u[MHUB];
      float a[MHUB];
#pragma unroll
      for (int j = 0; j < MHUB; ++j) {
        const bool on = k + j < n;
        a[j] = on ? lw[b0 + k + j] : 0.f;
        u[j] = on ? ldg16(pbase + (size_t)lsrc[b0 + k + j] * D + (size_t)v * E) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int j = 0; j < MHUB; ++j) {
        float f[E];
        unpack(u[j], f, (const T*)nullptr);
#pragma unroll
        for (int q = 0; q < E; ++q) acc[q] = fmaf(a[j], f[q], acc[q]);
      }
    }
#pragma unroll
    for (int q = 0; q < E; ++q) acc[q] = acc[q] * inv_den;
    reinterpret_cast<uint4*>(dst)[v] = pack(acc, (const T*)nullptr);
  }
  FICOCO_PHASE(2, 5);
}

}  // namespace ficoco
