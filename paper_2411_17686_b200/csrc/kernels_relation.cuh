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
constexpr int RINF = 12;    // 16-byte loads a thread has in flight in the by-column mode

// s_i = cA * v_i - (1 - cA) * mean_h attn[h, i] for one row chunk of one image, with
//   by_column == 0:  v_i = (1/Np) sum_j A[i, j]   (Eq. 1 as printed: row i of the map)
//   by_column == 1:  v_i = (1/Np) sum_j A[j, i]   (the attention token i receives)
// Row mode: a few rows per warp at a time, partial sums per row and lane.  Column mode: 64
// columns per pass, the rows dealt to row phases with eight rows in flight per thread, phases
// added in a fixed order.  Blocks whose rows start on 16-byte boundaries (Np a multiple of four)
// are read with 16-byte loads.
__global__ void __launch_bounds__(256) k_score_rel(const float* __restrict__ rel,
                                                   const ImgDesc* __restrict__ desc,
                                                   const WorkItem* __restrict__ work,
                                                   const float* __restrict__ attn, int H, float cA,
                                                   int by_column, float* __restrict__ s_raw) {
  extern __shared__ float vrow[];            // [rows of the largest chunk]
  __shared__ float red[4][RCOLS];
  __shared__ float4 red4[16][16];
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  const int np = d.np;
  const float* A = rel + d.rel0;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float inv_np = 1.0f / (float)np;
  // 16-byte loads when every row of the block starts on a 16-byte boundary
  const bool vec = (np & 3) == 0 && (reinterpret_cast<uintptr_t>(A) & 15) == 0;
  if (!by_column) {
    if (vec) {
      // four rows per warp at a time, two 16-byte loads per row and lane in flight
      const int nv = np >> 2;
      for (int r = 4 * warp; r < w.nrows; r += 32) {
        float s[4] = {0.f, 0.f, 0.f, 0.f};
        for (int j0 = lane; j0 < nv; j0 += 64) {
          float4 a[4][2];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float4* row = reinterpret_cast<const float4*>(A + (size_t)(w.r0 + min(r + i, w.nrows - 1)) * np);
#pragma unroll
            for (int q = 0; q < 2; ++q) {
              const int j = j0 + 32 * q;
              a[i][q] = j < nv ? __ldg(row + j) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
          }
#pragma unroll
          for (int i = 0; i < 4; ++i)
            s[i] += ((a[i][0].x + a[i][0].y) + (a[i][0].z + a[i][0].w)) + ((a[i][1].x + a[i][1].y) + (a[i][1].z + a[i][1].w));
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float t = warp_sum(s[i]);
          if (lane == 0 && r + i < w.nrows) vrow[r + i] = t * inv_np;
        }
      }
    } else {
    // two rows per warp at a time, four partial sums per row and lane
    for (int r = 2 * warp; r < w.nrows; r += 16) {
      const bool two = r + 1 < w.nrows;
      const float* row0 = A + (size_t)(w.r0 + r) * np;
      const float* row1 = two ? row0 + np : row0;
      float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
      for (int j0 = lane; j0 < np; j0 += 128) {
        float a[2][4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int j = j0 + 32 * q;
          a[0][q] = j < np ? __ldg(row0 + j) : 0.f;
          a[1][q] = j < np ? __ldg(row1 + j) : 0.f;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) { s[0][q] += a[0][q]; s[1][q] += a[1][q]; }
      }
      const float t0 = warp_sum((s[0][0] + s[0][1]) + (s[0][2] + s[0][3]));
      const float t1 = warp_sum((s[1][0] + s[1][1]) + (s[1][2] + s[1][3]));
      if (lane == 0) {
        vrow[r] = t0 * inv_np;
        if (two) vrow[r + 1] = t1 * inv_np;
      }
    }
    }
  } else if (vec && (w.r0 & 3) == 0) {
    // 16 groups of four columns x 16 row phases per pass, RINF rows in flight per thread
    const int tx = tid & 15, ty = tid >> 4;
    for (int c0 = 0; c0 < w.nrows; c0 += RCOLS) {
      const int c = c0 + 4 * tx;
      float4 s4 = make_float4(0.f, 0.f, 0.f, 0.f);
      if (c < w.nrows) {     // w.r0 + c + 3 < np because both are multiples of four
        const float* col = A + w.r0 + c;
        for (int j0 = ty; j0 < np; j0 += 16 * RINF) {
          float4 a[RINF];
#pragma unroll
          for (int q = 0; q < RINF; ++q) {
            const int j = j0 + 16 * q;
            a[q] = j < np ? __ldg(reinterpret_cast<const float4*>(col + (size_t)j * np)) : make_float4(0.f, 0.f, 0.f, 0.f);
          }
#pragma unroll
          for (int q = 0; q < RINF; ++q) { s4.x += a[q].x; s4.y += a[q].y; s4.z += a[q].z; s4.w += a[q].w; }
        }
      }
      red4[ty][tx] = s4;
      __syncthreads();
      if (tid < RCOLS && c0 + tid < w.nrows) {
        float t = 0.f;
#pragma unroll
        for (int k = 0; k < 16; ++k) t += reinterpret_cast<const float*>(&red4[k][tid >> 2])[tid & 3];
        vrow[c0 + tid] = t * inv_np;
      }
      __syncthreads();
    }
  } else {
    const int tx = tid & (RCOLS - 1), ty = tid / RCOLS;
    for (int c0 = 0; c0 < w.nrows; c0 += RCOLS) {
      const int c = c0 + tx;
      float s8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      if (c < w.nrows) {
        const float* col = A + w.r0 + c;
        for (int j0 = ty; j0 < np; j0 += 32) {     // rows j0, j0 + 4, ..., j0 + 28 in flight
          float a[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const int j = j0 + 4 * q;
            a[q] = j < np ? __ldg(col + (size_t)j * np) : 0.f;
          }
#pragma unroll
          for (int q = 0; q < 8; ++q) s8[q] += a[q];
        }
      }
      red[ty][tx] = ((s8[0] + s8[1]) + (s8[2] + s8[3])) + ((s8[4] + s8[5]) + (s8[6] + s8[7]));
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

// C_ij = A[S_i, T_j].  A CTA owns a few discarded tokens of one image and one column split of
// the image's preserved tokens, whose token indices it first copies to shared memory; a warp then
// takes one discarded token at a time.  Its lanes walk the split's columns, eight gathers from the
// token's row of the map in flight per lane, each lane keeping the LC largest entries it saw
// (value, position in T) in registers; the warp then draws the L largest of the 32 lists one by
// one (a shuffle tournament over the lists' heads).  The partial lists and the tail (tau_i, J_i,
// alpha_ij by the last split of the tile) are those of the fp32 correlate kernel.
constexpr int RGATHER = 8;   // gathers a lane has in flight

template <int LC>
__global__ void __launch_bounds__(256, LC <= 4 ? 4 : 2) k_correlate_rel(
    const float* __restrict__ rel, const ImgDesc* __restrict__ desc, const WorkItem* __restrict__ work,
    const int* __restrict__ S_idx, const int* __restrict__ T_idx,
    float* __restrict__ part_val, int* __restrict__ part_idx, int* __restrict__ tile_done,
    int* __restrict__ corr_cnt, float* __restrict__ tau_out, int* __restrict__ e_tgt,
    float* __restrict__ e_w, float* __restrict__ e_c, unsigned* __restrict__ status) {
  extern __shared__ int tcol[];              // token index of every column of the split
  __shared__ int is_last;
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  const int L = d.list_len, np = d.np;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const float* A = rel + d.rel0;
  const int col_begin = w.aux * d.cols_per_split;
  const int ncol = min(d.n_tgt, col_begin + d.cols_per_split) - col_begin;
  // the rows of this warp (two at most with the planned tiles of 16) are looked up while the
  // column indices arrive
  const int r_first = warp < w.nrows ? checked_index(S_idx[d.src0 + w.r0 + warp], np, status) : 0;
  for (int c = threadIdx.x; c < ncol; c += 256) tcol[c] = checked_index(T_idx[d.tgt0 + col_begin + c], np, status);
  __syncthreads();
  #pragma unroll 1
  for (int r = warp; r < w.nrows; r += 8) {
    const float* row = A + (size_t)(r == warp ? r_first : checked_index(S_idx[d.src0 + w.r0 + r], np, status)) * np;
    float v[LC];
    int ix[LC];
#pragma unroll
    for (int k = 0; k < LC; ++k) { v[k] = -CUDART_INF_F; ix[k] = INT_MAX; }
    #pragma unroll 1
    for (int c0 = lane; c0 < ncol; c0 += 32 * RGATHER) {
      float a[RGATHER];
#pragma unroll
      for (int q = 0; q < RGATHER; ++q) {
        const int c = c0 + 32 * q;
        a[q] = c < ncol ? __ldg(row + tcol[c]) : -CUDART_INF_F;
      }
#pragma unroll
      for (int q = 0; q < RGATHER; ++q) {
        float cv = a[q];
        int ci = col_begin + c0 + 32 * q;
        if (c0 + 32 * q >= ncol) continue;
#pragma unroll
        for (int k = 0; k < LC; ++k) {     // sorted insertion: the displaced entry moves down
          if (toplist_better(cv, ci, v[k], ix[k])) {
            const float tv = v[k]; const int ti = ix[k];
            v[k] = cv; ix[k] = ci; cv = tv; ci = ti;
          }
        }
      }
    }
    // the L best of the warp, best first
    const size_t o = (size_t)d.part0 + ((size_t)(w.r0 + r) * d.nsplit + w.aux) * L;
    #pragma unroll 1
    for (int k = 0; k < L; ++k) {
      float bv = v[0];
      int bi = ix[0];
#pragma unroll
      for (int m = 16; m >= 1; m >>= 1) {
        const float ov = __shfl_xor_sync(0xFFFFFFFFu, bv, m);
        const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, m);
        if (toplist_better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
      }
      if (bi != INT_MAX && bi == ix[0]) {   // the winner's owner pops its head
#pragma unroll
        for (int q = 0; q + 1 < LC; ++q) { v[q] = v[q + 1]; ix[q] = ix[q + 1]; }
        v[LC - 1] = -CUDART_INF_F; ix[LC - 1] = INT_MAX;
      }
      if (lane == 0) {
        part_val[o + k] = bv;
        part_idx[o + k] = bi == INT_MAX ? -1 : bi;
      }
    }
  }
  correlate_tail<LC>(d, w, (int)blockIdx.x - w.aux, tile_done, part_val, part_idx, corr_cnt, tau_out,
                     e_tgt, e_w, e_c, &is_last);
}

}  // namespace ficoco
