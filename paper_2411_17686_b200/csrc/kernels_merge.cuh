// Compress + compact (Eq. 2 and the last step of Algorithm 1 / 2).
#pragma once
#include "common.cuh"

namespace ficoco {

// One warp per output row, 16-byte vectors per lane, coalesced reads and writes.
//   CLS / text rows        : copied
//   preserved row j, I_j={}: copied bit for bit
//   preserved row j        : (x_j + sum_{i in I_j} alpha_ij x_i) / (1 + sum alpha_ij), fp32
//                            accumulation in ascending source order, one rounding.
// The per-target segments are sorted by source, so the sum has one fixed order and there
// are no floating-point atomics.
template <class T>
__global__ void __launch_bounds__(256) k_merge_compact(
    const T* __restrict__ tokens, int D, const ImgDesc* __restrict__ desc,
    const WorkItem* __restrict__ work, const int* __restrict__ S_idx,
    const int* __restrict__ T_idx, const int* __restrict__ seg_off,
    const int* __restrict__ seg_src, const float* __restrict__ seg_w, T* __restrict__ out) {
  constexpr int E = VecTraits<T>::E;
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nvec = D / E;

  for (int r = warp; r < w.nrows; r += 8) {
    const int orow = w.r0 + r;
    T* dst = out + (size_t)(d.out_row0 + orow) * D;
    int srow, e0 = 0, e1 = 0;
    if (orow < d.n_cls) {
      srow = orow;
    } else if (orow < d.n_cls + d.n_tgt) {
      const int tp = orow - d.n_cls;
      srow = d.n_cls + T_idx[d.tgt0 + tp];
      e0 = seg_off[d.tgt0 + w.img + tp];
      e1 = seg_off[d.tgt0 + w.img + tp + 1];
    } else {
      srow = d.n_cls + d.np + (orow - d.n_cls - d.n_tgt);
    }
    const T* src = tokens + (size_t)(d.row0 + srow) * D;
    if (e0 == e1) {
      for (int v = lane; v < nvec; v += 32)
        reinterpret_cast<uint4*>(dst)[v] = ldg16(src + (size_t)v * E);
      continue;
    }
    float wsum = 0.f;
    for (int e = e0; e < e1; ++e) wsum += seg_w[e];
    const float den = 1.0f + wsum;
    for (int v = lane; v < nvec; v += 32) {
      float acc[E];
      unpack(ldg16(src + (size_t)v * E), acc, (const T*)nullptr);
      for (int e = e0; e < e1; ++e) {
        const float a = seg_w[e];
        const T* xi = tokens + (size_t)(d.row0 + d.n_cls + S_idx[d.src0 + seg_src[e]]) * D;
        float f[E];
        unpack(ldg16(xi + (size_t)v * E), f, (const T*)nullptr);
#pragma unroll
        for (int k = 0; k < E; ++k) acc[k] = fmaf(a, f[k], acc[k]);
      }
#pragma unroll
      for (int k = 0; k < E; ++k) acc[k] = acc[k] / den;
      reinterpret_cast<uint4*>(dst)[v] = pack(acc, (const T*)nullptr);
    }
  }
}

}  // namespace ficoco
