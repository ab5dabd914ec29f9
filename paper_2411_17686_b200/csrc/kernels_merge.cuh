// Compress + compact (Eq. 2 and the last step of Algorithm 1 / 2).
#pragma once
#include "async_ops.cuh"
#include "common.cuh"

namespace ficoco {

constexpr int MHUB = 4;        // source rows a lane has in flight for a hub row
constexpr int MROWS = 32;      // most output rows a CTA can take (sizes of the per-row arrays)
constexpr int MROWS_CTA = 16;  // output rows per CTA the host plans (two per warp); 24 when that saves a wave
constexpr int MCOPY = MROWS_CTA / 8;   // rows a warp copies in one batch
constexpr int MLIST = 1024;    // (source, alpha) entries a CTA can hold in shared memory
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

// Compress + compact.  No per-target lists are built in global memory.  A CTA owns up to 32
// consecutive output rows of one image (warp w: rows w, w + 8, w + 16, w + 24).
//   1. every warp resolves the input row of its output rows (L1 prefetches of the rows were tried:
//      they never produced L1 hits and cost 1.7 us per step, so there are none);
//   2. meanwhile the CTA scans the image's (source -> target) entries twice (count, then fill)
//      to file those that hit its rows into per-row lists in shared memory (token index,
//      alpha), and orders every list by token index so that the
//      fp32 sums have one fixed order and no atomics touch floats;
//   3. out_j = (x_j + sum_{i in I_j} alpha_ij x_i) / (1 + sum alpha_ij), rounded once:
//      rows with few sources by their own warp; hub rows are cut into blocks of 32 vectors that
//      are dealt to the warps, every lane summing the sources of its vector in list order.
// If the CTA's rows receive more than MLIST sources in total, a slow in-order rescan is used.
// MINB (resident CTAs per SM the registers are capped for): 4 fills the SMs better when the merge
// grid runs between ordinary grids; 3 (no spills, fewer and shorter waves of CTAs draining) is
// faster when the next step's persistent filter grid is waiting for every SM to drain.
template <class T, int MINB>
__global__ void __launch_bounds__(256, MINB) k_merge_scan(
    const T* __restrict__ tokens, int D, const ImgDesc* __restrict__ desc,
    const WorkItem* __restrict__ work, const int* __restrict__ S_idx, const int* __restrict__ T_idx,
    const int* __restrict__ e_tgt, const float* __restrict__ e_w, T* __restrict__ out,
    int index_before_wait, unsigned* __restrict__ status, int* __restrict__ filter_cnt, int n_filter_cnt) {
  constexpr int E = VecTraits<T>::E;
  __shared__ int cnt[MROWS], beg[MROWS + 1], cur[MROWS], srow_s[MROWS];
  __shared__ int lsrc[MLIST];
  __shared__ float lw[MLIST];
  __shared__ int tsrc[MLIST];
  __shared__ float tw[MLIST];
  __shared__ int heavy_rows[MROWS];
  __shared__ int n_heavy, dead;
  FICOCO_PHASE_BEGIN(2);
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nvec = D / E;
  const int L = d.list_len;
  const int tp_lo = max(w.r0 - d.n_cls, 0);
  const int tp_hi = min(w.r0 + w.nrows - d.n_cls, d.n_tgt);
  const int n_ent = d.n_src * L;
  const T* pbase = tokens + (size_t)(d.row0 + d.n_cls) * D;

  if (tid < MROWS) { cnt[tid] = 0; cur[tid] = 0; }
  if (tid == 0) n_heavy = 0;
  // When the grid before this one is a correlate grid, the filter grid (which wrote T_idx) had
  // completed before this grid could start, so the row lookup may overlap that
  // grid's tail; otherwise wait first.
  if (!index_before_wait) grid_dep_wait();
  // input row of every output row (CLS / preserved token / trailing text row)
  #pragma unroll 1
  for (int r = warp; r < w.nrows; r += 8) {
    const int orow = w.r0 + r;
    int srow;
    if (orow < d.n_cls) srow = orow;
    else if (orow < d.n_cls + d.n_tgt) srow = d.n_cls + checked_index(T_idx[d.tgt0 + orow - d.n_cls], d.np, status);
    else if (orow < d.n_cls + d.n_tgt + d.n_extra) srow = -1;     // the additional token: written by k_convergent_token
    else srow = d.n_cls + d.np + (orow - d.n_cls - d.n_tgt - d.n_extra);
    if (lane == 0) srow_s[r] = srow;
  }
  if (index_before_wait) grid_dep_wait();
  // The filter grid of this step is complete: its per-image counters are cleared for whichever launch
  // uses that set next (launches replayed from graphs need not alternate between the two sets).  The
  // stores are fenced and the CTA synchronised before it releases the dependent grid.
  if (filter_cnt != nullptr && blockIdx.x == 0) {
    for (int i = tid; i < n_filter_cnt; i += 256) filter_cnt[i] = 0;
    __threadfence();
    __syncthreads();
  }
  grid_dep_launch();   // correlate is complete: the next step's filter may stream its rows under our tail
  FICOCO_PHASE(2, 1);
  // a step whose filter or correlate grid gave up has no valid index lists: write nothing
  if (tid == 0) dead = (*reinterpret_cast<const volatile unsigned*>(status) & STATUS_TIMEOUT) ? 1 : 0;
  __syncthreads();
  if (dead) return;
  // file the entries that hit this CTA's rows.  Up to 1024 entries per image every thread looks
  // at no more than four, keeps its matches in registers and needs one pass; larger images
  // take a counting pass and a filling pass.
  const bool one_pass = n_ent <= 4 * 256;
  int st_row[4], st_slot[4], st_src[4];
  float st_w[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) st_row[i] = -1;
  if (tp_hi > tp_lo) {
    if (one_pass) {
      int t4[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        // target, source and weight are fetched together: a source fetched only for the matches
        // would add a second round trip to L2
        const int e = tid + 256 * i;
        const bool on = e < n_ent;
        t4[i] = on ? e_tgt[d.ent0 + e] : -1;
        st_src[i] = on ? checked_index(S_idx[d.src0 + e / L], d.np, status) : 0;
        st_w[i] = on ? e_w[d.ent0 + e] : 0.f;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int t = t4[i];
        if (t >= tp_lo && t < tp_hi) {
          st_row[i] = t - tp_lo;
          st_slot[i] = atomicAdd(&cnt[t - tp_lo], 1);
        }
      }
    } else {
      for (int e = tid; e < n_ent; e += 256) {
        const int t = e_tgt[d.ent0 + e];
        if (t >= tp_lo && t < tp_hi) atomicAdd(&cnt[t - tp_lo], 1);
      }
    }
  }
  __syncthreads();
  if (warp == 0) {
    // exclusive scan of the 32 counts
    const int c = cnt[lane];
    int inc = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xFFFFFFFFu, inc, o);
      if (lane >= o) inc += n;
    }
    beg[lane] = inc - c;
    if (lane == 31) beg[MROWS] = inc;
    if (c > MHEAVY) heavy_rows[atomicAdd(&n_heavy, 1)] = lane;
  }
  __syncthreads();
  const int total = beg[MROWS];
  const bool fits = total <= MLIST;
  if (fits && total > 0) {
    if (one_pass) {
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (st_row[i] >= 0) {
          const int slot = beg[st_row[i]] + st_slot[i];
          tsrc[slot] = st_src[i];
          tw[slot] = st_w[i];
        }
    } else {
      for (int e = tid; e < n_ent; e += 256) {
        const int t = e_tgt[d.ent0 + e];
        if (t >= tp_lo && t < tp_hi) {
          const int slot = beg[t - tp_lo] + atomicAdd(&cur[t - tp_lo], 1);
          const int si = checked_index(S_idx[d.src0 + e / L], d.np, status);
          tsrc[slot] = si;
          tw[slot] = e_w[d.ent0 + e];
        }
      }
    }
    __syncthreads();
    // order every list by token index (rank of each entry inside its row)
    for (int i = tid; i < total; i += 256) {
      int r = 0;
      while (i >= beg[r + 1]) ++r;
      const int my = tsrc[i];
      int rank = 0;
      for (int k = beg[r]; k < beg[r + 1]; ++k) rank += tsrc[k] < my ? 1 : 0;
      lsrc[beg[r] + rank] = my;
      lw[beg[r] + rank] = tw[i];
    }
  }
  __syncthreads();

  FICOCO_PHASE(2, 2);
  // ---- rows without sources: plain copies, all of a warp's rows in flight together --------------
  #pragma unroll 1
  for (int j0 = 0; 8 * j0 < w.nrows; j0 += MCOPY)
  #pragma unroll 1
  for (int v0 = lane; v0 < nvec; v0 += 32 * MVB) {
    uint4 u[MCOPY][MVB];
#pragma unroll
    for (int j = 0; j < MCOPY; ++j) {
      const int r = warp + 8 * (j0 + j);
      const int orow = w.r0 + r;
      const bool is_tgt = orow >= d.n_cls && orow < d.n_cls + d.n_tgt;
      const bool copy = r < w.nrows && srow_s[r < w.nrows ? r : 0] >= 0 && (!is_tgt || cnt[orow - d.n_cls - tp_lo] == 0);
      const T* src = tokens + (size_t)(d.row0 + (copy ? srow_s[r] : 0)) * D;
#pragma unroll
      for (int b = 0; b < MVB; ++b) {
        const int v = v0 + 32 * b;
        u[j][b] = (copy && v < nvec) ? ldg16(src + (size_t)v * E) : make_uint4(0, 0, 0, 0);
      }
    }
#pragma unroll
    for (int j = 0; j < MCOPY; ++j) {
      const int r = warp + 8 * (j0 + j);
      const int orow = w.r0 + r;
      const bool is_tgt = orow >= d.n_cls && orow < d.n_cls + d.n_tgt;
      const bool copy = r < w.nrows && srow_s[r < w.nrows ? r : 0] >= 0 && (!is_tgt || cnt[orow - d.n_cls - tp_lo] == 0);
      T* dst = out + (size_t)(d.out_row0 + orow) * D;
#pragma unroll
      for (int b = 0; b < MVB; ++b) {
        const int v = v0 + 32 * b;
        if (copy && v < nvec) st_stream16(reinterpret_cast<uint4*>(dst) + v, u[j][b]);
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
    } else if (fits && n <= MHEAVY) {
      const int b0 = beg[li];
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
            st_stream16(reinterpret_cast<uint4*>(dst) + v, pack(acc[b], (const T*)nullptr));
          }
        }
      }
    } else if (!fits) {
      // too many sources for shared memory: walk the entries in order (ascending source)
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
          const T* x0 = pbase + (size_t)checked_index(S_idx[d.src0 + e / L], d.np, status) * D;
          float f[E];
          unpack(ldg16(x0 + (size_t)v * E), f, (const T*)nullptr);
          const float a0 = e_w[d.ent0 + e];
#pragma unroll
          for (int q = 0; q < E; ++q) acc[q] = fmaf(a0, f[q], acc[q]);
        }
#pragma unroll
        for (int q = 0; q < E; ++q) acc[q] = acc[q] / den;
        st_stream16(reinterpret_cast<uint4*>(dst) + v, pack(acc, (const T*)nullptr));
      }
    }
  }
  if (!fits) return;

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
    const int b0 = beg[li], n = cnt[li];
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
    st_stream16(reinterpret_cast<uint4*>(dst) + v, pack(acc, (const T*)nullptr));
  }
  FICOCO_PHASE(2, 5);
}

// Ablation "convergent correlation" (Sec. "Correlation-based Information Recycling": all discarded
// tokens merge into one additional token): the plain mean of an image's discarded rows, written
// behind the image's preserved rows.  One CTA per image; warp w sums the discarded rows w, w + 8,
// ... in ascending order, the eight partial sums are added in warp order (fp32, fixed order),
// scaled by 1 / N^S and rounded once.  Columns are processed in slabs of 128 vectors.
template <class T>
__global__ void __launch_bounds__(256) k_convergent_token(
    const T* __restrict__ tokens, int D, const ImgDesc* __restrict__ desc, const int* __restrict__ S_idx,
    T* __restrict__ out, const unsigned* __restrict__ status) {
  constexpr int E = VecTraits<T>::E;
  __shared__ float part[8][128 * E];
  const ImgDesc d = desc[blockIdx.x];
  if (!d.n_extra || (*status & STATUS_TIMEOUT)) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nvec = D / E;
  const T* pbase = tokens + (size_t)(d.row0 + d.n_cls) * D;
  T* dst = out + (size_t)(d.out_row0 + d.n_cls + d.n_tgt) * D;
  const float inv = 1.0f / (float)d.n_src;
  #pragma unroll 1
  for (int c0 = 0; c0 < nvec; c0 += 128) {
    float acc[4][E];
#pragma unroll
    for (int k = 0; k < 4; ++k)
#pragma unroll
      for (int q = 0; q < E; ++q) acc[k][q] = 0.f;
    #pragma unroll 1
    for (int s = warp; s < d.n_src; s += 8) {
      const T* row = pbase + (size_t)S_idx[d.src0 + s] * D;
      uint4 u[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int v = c0 + lane + 32 * k;
        u[k] = v < nvec ? ldg16(row + (size_t)v * E) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float f[E];
        unpack(u[k], f, (const T*)nullptr);
#pragma unroll
        for (int q = 0; q < E; ++q) acc[k][q] += f[q];
      }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k)
#pragma unroll
      for (int q = 0; q < E; ++q) part[warp][(lane + 32 * k) * E + q] = acc[k][q];
    __syncthreads();
    if (tid < 128 && c0 + tid < nvec) {
      float o[E];
#pragma unroll
      for (int q = 0; q < E; ++q) {
        float t = 0.f;
#pragma unroll
        for (int wv = 0; wv < 8; ++wv) t += part[wv][tid * E + q];
        o[q] = t * inv;
      }
      reinterpret_cast<uint4*>(dst)[c0 + tid] = pack(o, (const T*)nullptr);
    }
    __syncthreads();
  }
}

}  // namespace ficoco
