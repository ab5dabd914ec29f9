// Compress + compact (Eq. 2 and the last step of Algorithm 1 / 2).
#pragma once
#include "common.cuh"

namespace ficoco {

constexpr int MROWS = 8;    // output rows per CTA, one warp each
constexpr int MCAP = 64;    // sources per target kept in shared memory
constexpr int MVB = 4;      // 16-byte vectors a lane accumulates at a time

// Compress + compact.  No per-target lists are built in global memory.  A CTA owns up to 8
// consecutive output rows of one image.  It scans the image's (source -> target) entries once,
// files those that hit its rows into small shared-memory lists (token index, alpha), orders
// every list by token index (so the fp32 sum has one fixed order and no atomics touch floats),
// then one warp per row forms (x_j + sum alpha_ij x_i) / (1 + sum alpha_ij) and rounds once.
// Source rows are fetched two at a time, MVB vectors per lane each, to keep loads in flight.
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
        if (slot < MCAP) {
          lsrc[t - tp_lo][slot] = S_idx[d.src0 + e / L];
          lw[t - tp_lo][slot] = e_w[d.ent0 + e];
        }
      }
    }
  }
  __syncthreads();

  const int r = warp;
  if (r >= w.nrows) return;
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
  const T* pbase = tokens + (size_t)(d.row0 + d.n_cls) * D;
  if (n == 0) {
    for (int v = lane; v < nvec; v += 32) reinterpret_cast<uint4*>(dst)[v] = ldg16(src + (size_t)v * E);
    return;
  }
  if (n <= MCAP) {
    // order the list by token index: lanes rank entries lane and lane + 32
    int s0 = 0, s1 = 0, r0 = 0, r1 = 0;
    float w0 = 0.f, w1 = 0.f;
    const bool h0 = lane < n, h1 = lane + 32 < n;
    if (h0) { s0 = lsrc[li][lane]; w0 = lw[li][lane]; }
    if (h1) { s1 = lsrc[li][lane + 32]; w1 = lw[li][lane + 32]; }
    for (int k = 0; k < n; ++k) {
      const int sk = lsrc[li][k];
      r0 += (h0 && sk < s0) ? 1 : 0;
      r1 += (h1 && sk < s1) ? 1 : 0;
    }
    __syncwarp();
    if (h0) { lsrc[li][r0] = s0; lw[li][r0] = w0; }
    if (h1) { lsrc[li][r1] = s1; lw[li][r1] = w1; }
    __syncwarp();
    float wsum = 0.f;
    for (int k = 0; k < n; ++k) wsum += lw[li][k];
    const float den = 1.0f + wsum;
    for (int v0 = lane; v0 < nvec; v0 += 32 * MVB) {
      float acc[MVB][E];
#pragma unroll
      for (int b = 0; b < MVB; ++b) {
        const int v = v0 + 32 * b;
        if (v < nvec) unpack(ldg16(src + (size_t)v * E), acc[b], (const T*)nullptr);
      }
      int k = 0;
      for (; k + 1 < n; k += 2) {
        const T* x0 = pbase + (size_t)lsrc[li][k] * D;
        const T* x1 = pbase + (size_t)lsrc[li][k + 1] * D;
        const float a0 = lw[li][k], a1 = lw[li][k + 1];
        uint4 u0[MVB], u1[MVB];
#pragma unroll
        for (int b = 0; b < MVB; ++b) {
          const int v = v0 + 32 * b;
          u0[b] = v < nvec ? ldg16(x0 + (size_t)v * E) : make_uint4(0, 0, 0, 0);
          u1[b] = v < nvec ? ldg16(x1 + (size_t)v * E) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int b = 0; b < MVB; ++b) {
          float f[E];
          unpack(u0[b], f, (const T*)nullptr);
#pragma unroll
          for (int q = 0; q < E; ++q) acc[b][q] = fmaf(a0, f[q], acc[b][q]);
          unpack(u1[b], f, (const T*)nullptr);
#pragma unroll
          for (int q = 0; q < E; ++q) acc[b][q] = fmaf(a1, f[q], acc[b][q]);
        }
      }
      if (k < n) {
        const T* x0 = pbase + (size_t)lsrc[li][k] * D;
        const float a0 = lw[li][k];
#pragma unroll
        for (int b = 0; b < MVB; ++b) {
          const int v = v0 + 32 * b;
          if (v < nvec) {
            float f[E];
            unpack(ldg16(x0 + (size_t)v * E), f, (const T*)nullptr);
#pragma unroll
            for (int q = 0; q < E; ++q) acc[b][q] = fmaf(a0, f[q], acc[b][q]);
          }
        }
      }
#pragma unroll
      for (int b = 0; b < MVB; ++b) {
        const int v = v0 + 32 * b;
        if (v < nvec) {
#pragma unroll
          for (int q = 0; q < E; ++q) acc[b][q] = acc[b][q] / den;
          reinterpret_cast<uint4*>(dst)[v] = pack(acc[b], (const T*)nullptr);
        }
      }
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
        const T* x0 = pbase + (size_t)S_idx[d.src0 + e / L] * D;
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

}  // namespace ficoco
