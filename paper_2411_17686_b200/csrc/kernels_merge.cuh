// Compress + compact (Eq. 2 and the last step of Algorithm 1 / 2).
#pragma once
#include "common.cuh"

namespace ficoco {

constexpr int MROWS = 32;   // output rows per CTA
constexpr int MCAP = 32;    // sources per target kept in shared memory

// Compress + compact, second form: no per-target lists are built in global memory.  A CTA
// owns up to 32 consecutive output rows of one image.  It scans the image's (source -> target)
// entries once, files those that hit its rows into small shared-memory lists, orders every
// list by source (so the fp32 sum has one fixed order and no atomics touch floats), then one
// warp per row forms (x_j + sum alpha_ij x_i) / (1 + sum alpha_ij) and rounds once.
// A row with more than MCAP sources takes a slower in-order rescan of the entries instead.
template <class T>
__global__ void __launch_bounds__(256) k_merge_scan(
    const T* __restrict__ tokens, int D, const ImgDesc* __restrict__ desc,
    const WorkItem* __restrict__ work, const int* __restrict__ S_idx, const int* __restrict__ T_idx,
    const int* __restrict__ e_tgt, const float* __restrict__ e_w, T* __restrict__ out) {
  constexpr int E = VecTraits<T>::E;
  __shared__ int cnt[MROWS];
  __shared__ int lsrc[MROWS][MCAP];
  __shared__ float lw[MROWS][MCAP];
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nvec = D / E;
  const int L = d.list_len;
  const int tp_lo = max(w.r0 - d.n_cls, 0);
  const int tp_hi = min(w.r0 + w.nrows - d.n_cls, d.n_tgt);
  const int n_ent = d.n_src * L;

  if (tid < MROWS) cnt[tid] = 0;
  __syncthreads();
  if (tp_hi > tp_lo) {
    for (int e = tid; e < n_ent; e += 256) {
      const int t = e_tgt[d.ent0 + e];
      if (t >= tp_lo && t < tp_hi) {
        const int slot = atomicAdd(&cnt[t - tp_lo], 1);
        if (slot < MCAP) { lsrc[t - tp_lo][slot] = e / L; lw[t - tp_lo][slot] = e_w[d.ent0 + e]; }
      }
    }
  }
  __syncthreads();

  for (int r = warp; r < w.nrows; r += 8) {
    const int orow = w.r0 + r;
    T* dst = out + (size_t)(d.out_row0 + orow) * D;
    int srow, n = 0, li = 0;
    if (orow < d.n_cls) {
      srow = orow;
    } else if (orow < d.n_cls + d.n_tgt) {
      const int tp = orow - d.n_cls;
      srow = d.n_cls + T_idx[d.tgt0 + tp];
      li = tp - tp_lo;
      n = cnt[li];
    } else {
      srow = d.n_cls + d.np + (orow - d.n_cls - d.n_tgt);
    }
    const T* src = tokens + (size_t)(d.row0 + srow) * D;
    if (n == 0) {
      for (int v = lane; v < nvec; v += 32) reinterpret_cast<uint4*>(dst)[v] = ldg16(src + (size_t)v * E);
      continue;
    }
    if (n <= MCAP) {
      // order the list by source: every lane ranks one entry
      int my_s = 0, rank = 0;
      float my_w = 0.f;
      if (lane < n) {
        my_s = lsrc[li][lane];
        my_w = lw[li][lane];
        for (int k = 0; k < n; ++k) rank += lsrc[li][k] < my_s ? 1 : 0;
      }
      __syncwarp();
      if (lane < n) { lsrc[li][rank] = my_s; lw[li][rank] = my_w; }
      __syncwarp();
      float wsum = 0.f;
      for (int k = 0; k < n; ++k) wsum += lw[li][k];
      const float den = 1.0f + wsum;
      for (int v = lane; v < nvec; v += 32) {
        float acc[E];
        unpack(ldg16(src + (size_t)v * E), acc, (const T*)nullptr);
        int k = 0;
        for (; k + 1 < n; k += 2) {
          const T* x0 = tokens + (size_t)(d.row0 + d.n_cls + S_idx[d.src0 + lsrc[li][k]]) * D;
          const T* x1 = tokens + (size_t)(d.row0 + d.n_cls + S_idx[d.src0 + lsrc[li][k + 1]]) * D;
          const uint4 u0 = ldg16(x0 + (size_t)v * E), u1 = ldg16(x1 + (size_t)v * E);
          float f[E];
          unpack(u0, f, (const T*)nullptr);
          const float a0 = lw[li][k], a1 = lw[li][k + 1];
#pragma unroll
          for (int q = 0; q < E; ++q) acc[q] = fmaf(a0, f[q], acc[q]);
          unpack(u1, f, (const T*)nullptr);
#pragma unroll
          for (int q = 0; q < E; ++q) acc[q] = fmaf(a1, f[q], acc[q]);
        }
        if (k < n) {
          const T* x0 = tokens + (size_t)(d.row0 + d.n_cls + S_idx[d.src0 + lsrc[li][k]]) * D;
          float f[E];
          unpack(ldg16(x0 + (size_t)v * E), f, (const T*)nullptr);
          const float a0 = lw[li][k];
#pragma unroll
          for (int q = 0; q < E; ++q) acc[q] = fmaf(a0, f[q], acc[q]);
        }
#pragma unroll
        for (int q = 0; q < E; ++q) acc[q] = acc[q] / den;
        reinterpret_cast<uint4*>(dst)[v] = pack(acc, (const T*)nullptr);
      }
    } else {
      // many sources: walk the entries in order (ascending source), no list
      const int tp = orow - d.n_cls;
      float wsum = 0.f;
      for (int e = 0; e < n_ent; ++e)
        if (e_tgt[d.ent0 + e] == tp) wsum += e_w[d.ent0 + e];
      const float den = 1.0f + wsum;
      for (int v = lane; v < nvec; v += 32) {
        float acc[E];
        unpack(ldg16(src + (size_t)v * E), acc, (const T*)nullptr);
        for (int e = 0; e < n_ent; ++e) {
          if (e_tgt[d.ent0 + e] != tp) continue;
          const T* x0 = tokens + (size_t)(d.row0 + d.n_cls + S_idx[d.src0 + e / L]) * D;
          float f[E];
          unpack(ldg16(x0 + (size_t)v * E), f, (const T*)nullptr);
          const float a0 = e_w[d.ent0 + e];
#pragma unroll
          for (int q = 0; q < E; ++q) acc[q] = fmaf(a0, f[q], acc[q]);
        }
#pragma unroll
        for (int q = 0; q < E; ++q) acc[q] = acc[q] / den;
        reinterpret_cast<uint4*>(dst)[v] = pack(acc, (const T*)nullptr);
      }
    }
  }
}

}  // namespace ficoco
