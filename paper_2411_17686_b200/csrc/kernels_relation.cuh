// Reduce step driven by a caller-supplied relation matrix: the paper's own formulation, in
// which every token-token quantity is read from the self-attention map A^v (Eq. 1 first term,
// and C = A^v in Sec. "Correlation-based Information Recycling") instead of from the cosine
// similarity of the hidden states.  `rel` holds, image after image, one fp32 [Np, Np] block
// over the alive patch tokens (row = query token, no CLS row or column).
#pragma once
#include <limits.h>
#include <math_constants.h>
#include "common.cuh"
#include "kernels_correlate.cuh"

namespace ficoco {

constexpr int RCOLS = 64;   // columns summed together in the by-column mode

// s_i = cA * v_i - (1 - cA) * mean_h attn[h, i] for one row chunk of one image, with
//   by_column == 0:  v_i = (1/Np) sum_j A[i, j]   (Eq. 1 as printed: row i of the map)
//   by_column == 1:  v_i = (1/Np) sum_j A[j, i]   (the attention token i receives)
// Row mode: one warp per row, four partial sums per lane.  Column mode: 64 columns x 4 row
// phases per pass, two partial sums per thread, phases added in a fixed order.
__global__ void __launch_bounds__(256) k_score_rel(const float* __restrict__ rel,
                                                   const ImgDesc* __restrict__ desc,
                                                   const WorkItem* __restrict__ work,
                                                   const float* __restrict__ attn, int H, float cA,
                                                   int by_column, float* __restrict__ s_raw) {
  extern __shared__ float vrow[];            // [rows of the largest chunk]
  __shared__ float red[4][RCOLS];
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  const int np = d.np;
  const float* A = rel + d.rel0;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float inv_np = 1.0f / (float)np;
  if (!by_column) {
    for (int r = warp; r < w.nrows; r += 8) {
      const float* row = A + (size_t)(w.r0 + r) * np;
      float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
      int j = lane;
      for (; j + 96 < np; j += 128) {
        s0 += __ldg(row + j); s1 += __ldg(row + j + 32); s2 += __ldg(row + j + 64); s3 += __ldg(row + j + 96);
      }
      for (; j < np; j += 32) s0 += __ldg(row + j);
      const float s = warp_sum((s0 + s1) + (s2 + s3));
      if (lane == 0) vrow[r] = s * inv_np;
    }
  } else {
    const int tx = tid & (RCOLS - 1), ty = tid / RCOLS;
    for (int c0 = 0; c0 < w.nrows; c0 += RCOLS) {
      const int c = c0 + tx;
      float s0 = 0.f, s1 = 0.f;
      if (c < w.nrows) {
        const float* col = A + w.r0 + c;
        int j = ty;
        for (; j + 4 < np; j += 8) { s0 += __ldg(col + (size_t)j * np); s1 += __ldg(col + (size_t)(j + 4) * np); }
        for (; j < np; j += 4) s0 += __ldg(col + (size_t)j * np);
      }
      red[ty][tx] = s0 + s1;
      __syncthreads();
      if (ty == 0 && c < w.nrows) vrow[c] = ((red[0][tx] + red[1][tx]) + (red[2][tx] + red[3][tx])) * inv_np;
      __syncthreads();
    }
  }
  __syncthreads();
  const float inv_h = 1.0f / (float)H;
  for (int r = tid; r < w.nrows; r += 256) {
    const float* a = attn + d.attn0 + w.r0 + r;
    float s = 0.f;
    for (int h = 0; h < H; ++h) s += __ldg(a + (size_t)h * np);
    s_raw[d.patch0 + w.r0 + r] = cA * vrow[r] - (1.0f - cA) * (s * inv_h);
  }
}

// C_ij = A[S_i, T_j]: a CTA owns up to 64 discarded tokens and one column split of the image's
// preserved tokens, gathers the entries 64 columns at a time into shared memory and keeps the L
// largest per row (value, position in T) exactly as the fp32 correlate kernel does; the partial
// lists and the tail (tau_i, J_i, alpha_ij by the last split of the tile) are shared with it.
__global__ void __launch_bounds__(256) k_correlate_rel(
    const float* __restrict__ rel, const ImgDesc* __restrict__ desc, const WorkItem* __restrict__ work,
    const int* __restrict__ S_idx, const int* __restrict__ T_idx,
    float* __restrict__ part_val, int* __restrict__ part_idx, int* __restrict__ tile_done,
    int* __restrict__ corr_cnt, float* __restrict__ tau_out, int* __restrict__ e_tgt,
    float* __restrict__ e_w, float* __restrict__ e_c) {
  __shared__ int is_last;
  __shared__ float Cs[CBM][CBN + 1];
  __shared__ float lv[CBM][KCAP];
  __shared__ int li[CBM][KCAP];
  __shared__ int rowS[CBM], rowT[CBN];
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  const int L = d.list_len, np = d.np;
  const int tid = threadIdx.x;
  const float* A = rel + d.rel0;
  for (int i = tid; i < CBM * KCAP; i += 256) {
    (&lv[0][0])[i] = -CUDART_INF_F;
    (&li[0][0])[i] = INT_MAX;
  }
  if (tid < CBM) rowS[tid] = tid < w.nrows ? S_idx[d.src0 + w.r0 + tid] : 0;
  const int col_begin = w.aux * d.cols_per_split;
  const int col_end = min(d.n_tgt, col_begin + d.cols_per_split);
  for (int c0 = col_begin; c0 < col_end; c0 += CBN) {
    __syncthreads();
    const int ncol = min(CBN, col_end - c0);
    if (tid < CBN) rowT[tid] = tid < ncol ? T_idx[d.tgt0 + c0 + tid] : 0;
    __syncthreads();
    for (int i = tid; i < w.nrows * CBN; i += 256) {
      const int r = i / CBN, c = i % CBN;
      Cs[r][c] = c < ncol ? __ldg(A + (size_t)rowS[r] * np + rowT[c]) : 0.f;
    }
    __syncthreads();
    if (tid < w.nrows) {
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
  correlate_tail<KCAP>(d, w, (int)blockIdx.x - w.aux, tile_done, part_val, part_idx, corr_cnt, tau_out,
                       e_tgt, e_w, e_c, &is_last);
}

}  // namespace ficoco
