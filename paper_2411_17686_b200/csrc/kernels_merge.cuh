// Compress + compact (Eq. 2 and the last step of Algorithm 1 / 2).
#pragma once
#include "async_ops.cuh"
#include "common.cuh"

namespace ficoco {

constexpr int MROWS = 32;      // most output rows a CTA can take (sizes of the per-row arrays)
constexpr int MROWS_CTA = 16;  // output rows per CTA the host plans (two per warp)
constexpr int MCOPY = 3;       // rows a warp copies in one batch (covers CTAs of up to 24 rows)
constexpr int MLIST = 2048;    // entries of hub rows a CTA can order in shared memory
constexpr int MHUBS = 256;     // hub rows a CTA can keep track of (each has more than REC_INLINE entries)
constexpr int MMAP = 2048;      // preserved tokens per image up to which the image's hub rows are shared by its CTAs
constexpr int MVB = 4;         // 16-byte vectors a lane accumulates at a time
constexpr int MHUB = 8;        // source rows a lane has in flight on a hub row

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
// w, w + 8, ...).
//   1. every row resolves its input row (CLS / preserved token / trailing text row);
//   2. one pass over the records of the image's preserved tokens (how many discarded tokens are
//      merged into each and the first REC_INLINE of them): the short lists of the CTA's own rows
//      are ordered in registers, and every row of the image with more entries (a "hub" row) is
//      registered with its inline entries; the rest of a hub row's entries come from the image's
//      overflow pool.  Every list is ordered by token index, so that the fp32 sums of Eq. 2 have
//      one fixed order and no atomics touch floats;
//   3. out_j = (x_j + sum_{i in I_j} alpha_ij x_i) / (1 + sum alpha_ij), rounded once: rows
//      without sources are copied in one batch, rows with up to REC_INLINE sources are merged by
//      their own warp (both while the pool entries are in flight);
//   4. hub rows hold most of the source traffic and sit in few CTAs, so they are shared: every
//      (hub row, block of 32 vectors) item belongs to the CTA of the image that its number
//      (position * blocks + block) modulo the image's CTAs names.  A warp takes an item, every
//      lane summing the sources of its vector in list order, MHUB source rows in flight.  The
//      lists are built redundantly by the image's CTAs, but nothing is exchanged between CTAs
//      and nobody waits.
// When an image has more preserved tokens, hub rows or hub entries than fit (MMAP / MHUBS /
// MLIST), a CTA merges only the hub rows among its own rows, and if even those do not fit it
// walks the image's entry arrays in order (slow, degenerate inputs only).
template <class T>
__global__ void __launch_bounds__(256, 3) k_merge_rec(
    const T* __restrict__ tokens, int D, const ImgDesc* __restrict__ desc,
    const WorkItem* __restrict__ work, const int* __restrict__ S_idx, const int* __restrict__ T_idx,
    const int* __restrict__ e_tgt, const float* __restrict__ e_w, const TgtRec* __restrict__ rec,
    const int* __restrict__ pool_cnt, const PoolEnt* __restrict__ pool, T* __restrict__ out,
    int index_before_wait, const unsigned* __restrict__ status, int rows_per_cta) {
  constexpr int E = VecTraits<T>::E;
  __shared__ int cnt[MROWS], srow_s[MROWS];
  __shared__ int lsrc_l[MROWS][8];                  // own rows with up to REC_INLINE sources, ordered
  __shared__ float lw_l[MROWS][8];
  __shared__ int hsrc[MLIST], tsrc[MLIST];          // hub rows: ordered entries / as they arrived
  __shared__ float hw[MLIST], tw[MLIST];
  __shared__ short hmap[MMAP];                      // preserved token (minus scan_lo) -> hub slot, -1 = none
  __shared__ int hub_t[MHUBS], hub_srow[MHUBS], hoff[MHUBS], hlen[MHUBS], hcur[MHUBS];
  __shared__ float hub_inv[MHUBS];
  __shared__ int n_hub_s, hub_total_s, overflow_s, dead;
  FICOCO_PHASE(2, 0);
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nvec = D / E;
  const int L = d.list_len;
  const T* pbase = tokens + (size_t)(d.row0 + d.n_cls) * D;
  const int tp_lo = max(w.r0 - d.n_cls, 0);                         // own preserved tokens: [tp_lo, tp_hi)
  const int tp_hi = max(tp_lo, min(w.r0 + w.nrows - d.n_cls, d.n_tgt));

  // When the grid before this one is a correlate grid, the filter grid (which wrote T_idx) had
  // completed before this grid could start, so the row lookup may overlap that
  // grid's tail; otherwise wait first.
  if (!index_before_wait) grid_dep_wait();
  int my_srow = 0;
  if (tid < w.nrows) {
    const int orow = w.r0 + tid;
    if (orow < d.n_cls) my_srow = orow;
    else if (orow < d.n_cls + d.n_tgt) my_srow = d.n_cls + T_idx[d.tgt0 + orow - d.n_cls];
    else my_srow = d.n_cls + d.np + (orow - d.n_cls - d.n_tgt);
  }
  // The token rows do not stay in L2 from the kernels before (the step's working set is larger than
  // what L2 keeps of it), and this grid is resident well before the correlate grid ends: ask L2
  // for the rows this CTA will copy or merge into, and for its share of the image's discarded rows
  // (every discarded row is merged somewhere), so that the reads below find them on chip.
  if (tid < w.nrows) srow_s[tid] = my_srow;
  __syncthreads();
  {
    const int lines = (D * (int)sizeof(T) + 127) / 128;          // 128-byte lines per row
    #pragma unroll 1
    for (int r = warp; r < w.nrows; r += 8) {
      const char* row = reinterpret_cast<const char*>(tokens + (size_t)(d.row0 + srow_s[r]) * D);
      for (int l = lane; l < lines; l += 32) asm volatile("prefetch.global.L2 [%0];" ::"l"(row + (size_t)l * 128));
    }
    if (index_before_wait && L > 0) {                            // S_idx is final: the filter grid has completed
      const int nct0 = (d.n_cls + d.n_tgt + d.n_tail + rows_per_cta - 1) / rows_per_cta;
      const int per = (d.n_src + nct0 - 1) / nct0;
      const int s_end = min(d.n_src, (w.aux + 1) * per);
      #pragma unroll 1
      for (int sidx = w.aux * per + warp; sidx < s_end; sidx += 8) {
        const char* row = reinterpret_cast<const char*>(pbase + (size_t)S_idx[d.src0 + sidx] * D);
        for (int l = lane; l < lines; l += 32) asm volatile("prefetch.global.L2 [%0];" ::"l"(row + (size_t)l * 128));
      }
    }
  }
  if (tid < MROWS) cnt[tid] = 0;
  if (tid == 0) { n_hub_s = 0; hub_total_s = 0; overflow_s = 0; }
  bool shared_hubs = L > 0 && d.n_tgt <= MMAP;
  int scan_lo = shared_hubs ? 0 : tp_lo, scan_hi = shared_hubs ? d.n_tgt : tp_hi;
  for (int i = tid; i < scan_hi - scan_lo; i += 256) hmap[i] = -1;
  if (index_before_wait) grid_dep_wait();
  grid_dep_launch();   // correlate is complete: the next step's filter may stream its rows under our tail
  FICOCO_PHASE(2, 1);
  // a step whose filter or correlate grid gave up has no valid index lists: write nothing
  if (tid == 0) dead = (*reinterpret_cast<const volatile unsigned*>(status) & STATUS_TIMEOUT) ? 1 : 0;
  const int np_ent = L > 0 ? __ldcg(pool_cnt + w.img) : 0;
  __syncthreads();
  if (dead) return;
  // ---- one pass over the records: own rows' short lists, hub rows of the scanned range ----------
  #pragma unroll 1
  for (int pass = 0; pass < 2; ++pass) {
    if (L > 0) {
      #pragma unroll 1
      for (int t0 = scan_lo + tid; t0 < scan_hi; t0 += 2 * 256) {      // two records in flight per thread
        uint4 q[2][4];
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
          for (int k = 0; k < 4; ++k)
            q[j][k] = t0 + 256 * j < scan_hi
                          ? __ldcg(reinterpret_cast<const uint4*>(rec + d.tgt0 + t0 + 256 * j) + k)
                          : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int t = t0 + 256 * j;
          if (t >= scan_hi) continue;
          const int c = (int)q[j][0].x;
          const int es[REC_INLINE] = {(int)q[j][0].z, (int)q[j][1].x, (int)q[j][1].z, (int)q[j][2].x,
                                      (int)q[j][2].z, (int)q[j][3].x, (int)q[j][3].z};
          const uint32_t ew[REC_INLINE] = {q[j][0].w, q[j][1].y, q[j][1].w, q[j][2].y, q[j][2].w, q[j][3].y, q[j][3].w};
          const bool own = t >= tp_lo && t < tp_hi;
          const int r = t + d.n_cls - w.r0;                              // own row index
          if (own) cnt[r] = c;
          if (c > REC_INLINE) {
            const int slot = atomicAdd(&n_hub_s, 1);
            const int off = atomicAdd(&hub_total_s, c);
            if (slot < MHUBS && off + c <= MLIST) {
              hub_t[slot] = t; hoff[slot] = off; hlen[slot] = c; hcur[slot] = off + REC_INLINE;
              hmap[t - scan_lo] = (short)slot;
#pragma unroll
              for (int k = 0; k < REC_INLINE; ++k) { tsrc[off + k] = es[k]; tw[off + k] = __uint_as_float(ew[k]); }
            } else {
              overflow_s = 1;
            }
          } else if (own) {
#pragma unroll
            for (int k = 0; k < REC_INLINE; ++k) {
              if (k < c) {
                int rank = 0;
#pragma unroll
                for (int m = 0; m < REC_INLINE; ++m) rank += (m < c && es[m] < es[k]) ? 1 : 0;
                lsrc_l[r][rank] = es[k];
                lw_l[r][rank] = __uint_as_float(ew[k]);
              }
            }
          }
        }
      }
    }
    __syncthreads();
    if (!overflow_s || !shared_hubs) break;
    // the image's hub rows do not fit: this CTA looks after the hub rows among its own rows only
    __syncthreads();
    shared_hubs = false;
    scan_lo = tp_lo;
    scan_hi = tp_hi;
    if (tid == 0) { n_hub_s = 0; hub_total_s = 0; overflow_s = 0; }
    for (int i = tid; i < tp_hi - tp_lo; i += 256) hmap[i] = -1;
    __syncthreads();
  }
  const bool fits = overflow_s == 0;
  const int n_hub = fits ? n_hub_s : 0;
  // the rest of the hub rows' entries (overflow pool) and their input rows: in flight during the copies
  uint4 pe[2];
#pragma unroll
  for (int j = 0; j < 2; ++j)
    pe[j] = (n_hub > 0 && tid + 256 * j < np_ent)
                ? __ldcg(reinterpret_cast<const uint4*>(pool + (size_t)d.ent0 + tid + 256 * j))
                : make_uint4(0xFFFFFFFFu, 0, 0, 0);
  const int hub_in = tid < n_hub ? T_idx[d.tgt0 + hub_t[tid]] : 0;
  FICOCO_PHASE(2, 2);

  // ---- rows without sources: plain copies, all of a warp's rows in flight together --------------
  #pragma unroll 1
  for (int v0 = lane; v0 < nvec; v0 += 32 * MVB) {
    uint4 u[MCOPY][MVB];
#pragma unroll
    for (int j = 0; j < MCOPY; ++j) {
      const int r = warp + 8 * j;
      const bool copy = r < w.nrows && cnt[r] == 0;
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
      const bool copy = r < w.nrows && cnt[r] == 0;
      T* dst = out + (size_t)(d.out_row0 + w.r0 + r) * D;
#pragma unroll
      for (int b = 0; b < MVB; ++b) {
        const int v = v0 + 32 * b;
        if (copy && v < nvec) reinterpret_cast<uint4*>(dst)[v] = u[j][b];
      }
    }
  }
  #pragma unroll 1
  for (int r = warp + 8 * MCOPY; r < w.nrows; r += 8) {      // rows past the batch (more than 16 rows per CTA)
    if (cnt[r] != 0) continue;
    const T* src = tokens + (size_t)(d.row0 + srow_s[r]) * D;
    T* dst = out + (size_t)(d.out_row0 + w.r0 + r) * D;
    for (int v = lane; v < nvec; v += 32) reinterpret_cast<uint4*>(dst)[v] = ldg16(src + (size_t)v * E);
  }
  FICOCO_PHASE(2, 3);

  // ---- rows with a few sources: one warp per row --------------------------------------------------
  #pragma unroll 1
  for (int r = warp; r < w.nrows; r += 8) {
    const int n = cnt[r];
    if (n == 0 || n > REC_INLINE) continue;
    T* dst = out + (size_t)(d.out_row0 + w.r0 + r) * D;
    const T* src = tokens + (size_t)(d.row0 + srow_s[r]) * D;
    float wsum = 0.f;
    for (int k = 0; k < n; ++k) wsum += lw_l[r][k];
    const float inv_den = 1.0f / (1.0f + wsum);   // one division per row, then multiplies
    #pragma unroll 1
    for (int v0 = lane; v0 < nvec; v0 += 32 * MVB) {
      float acc[MVB][E];
#pragma unroll
      for (int b = 0; b < MVB; ++b) {
        const int v = v0 + 32 * b;
        unpack(v < nvec ? ldg16(src + (size_t)v * E) : make_uint4(0, 0, 0, 0), acc[b], (const T*)nullptr);
      }
      merge_accumulate<T>(acc, pbase, D, lsrc_l[r], lw_l[r], 0, n, v0, nvec);
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
  FICOCO_PHASE(2, 4);

  if (!fits) {
    // too many entries for shared memory: every own hub row walks the image's entries in order
    // (ascending token index)
    const int n_ent = d.n_src * L;
    #pragma unroll 1
    for (int r = warp; r < w.nrows; r += 8) {
      if (cnt[r] <= REC_INLINE) continue;
      const int tp = w.r0 + r - d.n_cls;
      const T* src = tokens + (size_t)(d.row0 + srow_s[r]) * D;
      T* dst = out + (size_t)(d.out_row0 + w.r0 + r) * D;
      float wsum = 0.f;
      for (int e = 0; e < n_ent; ++e)
        if (e_tgt[d.ent0 + e] == tp) wsum += e_w[d.ent0 + e];
      const float inv_den = 1.0f / (1.0f + wsum);
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
        for (int q = 0; q < E; ++q) acc[q] = acc[q] * inv_den;
        reinterpret_cast<uint4*>(dst)[v] = pack(acc, (const T*)nullptr);
      }
    }
    FICOCO_PHASE(2, 5);
    return;
  }
  if (n_hub == 0) { FICOCO_PHASE(2, 5); return; }

  // ---- hub rows: finish the lists (pool entries), order them, weights ---------------------------
  {
    const int span = scan_hi - scan_lo;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int t = (int)pe[j].x - scan_lo;
      if (tid + 256 * j < np_ent && t >= 0 && t < span && hmap[t] >= 0) {
        const int slot = atomicAdd(&hcur[hmap[t]], 1);
        tsrc[slot] = (int)pe[j].y;
        tw[slot] = __uint_as_float(pe[j].z);
      }
    }
    #pragma unroll 1
    for (int e = tid + 512; e < np_ent; e += 256) {
      const uint4 u = __ldcg(reinterpret_cast<const uint4*>(pool + (size_t)d.ent0 + e));
      const int t = (int)u.x - scan_lo;
      if (t >= 0 && t < span && hmap[t] >= 0) {
        const int slot = atomicAdd(&hcur[hmap[t]], 1);
        tsrc[slot] = (int)u.y;
        tw[slot] = __uint_as_float(u.z);
      }
    }
    if (tid < n_hub) hub_srow[tid] = d.n_cls + hub_in;
  }
  __syncthreads();
  #pragma unroll 1
  for (int h = warp; h < n_hub; h += 8) {
    const int off = hoff[h], n = hlen[h];
    for (int k = lane; k < n; k += 32) {
      const int my = tsrc[off + k];
      int rank = 0;
      for (int m = 0; m < n; ++m) rank += tsrc[off + m] < my ? 1 : 0;
      hsrc[off + rank] = my;
      hw[off + rank] = tw[off + k];
    }
    __syncwarp();
    // 1 / (1 + sum alpha), the sum in a fixed order: lane l adds entries l, l + 32, ...; then a shuffle tree
    float wsum = 0.f;
    for (int k = lane; k < n; k += 32) wsum += hw[off + k];
    wsum = warp_sum(wsum);
    if (lane == 0) hub_inv[h] = 1.0f / (1.0f + wsum);
  }
  __syncthreads();

  // ---- this CTA's share of the (hub row, block of 32 vectors) items ------------------------------
  const int nblk = (nvec + 31) / 32;
  int nct = 1, me = 0;                              // CTAs of the image that share its hub rows, this one's index
  if (shared_hubs) {
    nct = (d.n_cls + d.n_tgt + d.n_tail + rows_per_cta - 1) / rows_per_cta;
    me = w.aux;
  }
  #pragma unroll 1
  for (int h = warp; h < n_hub; h += 8) {
    const int b0 = hoff[h], n = hlen[h];
    // blocks with (position * nblk + block) % nct == me
    int blk0 = (me - (int)(((long long)hub_t[h] * nblk) % nct)) % nct;
    if (blk0 < 0) blk0 += nct;
    #pragma unroll 1
    for (int blk = blk0; blk < nblk; blk += nct) {
      const int v = blk * 32 + lane;
      if (v >= nvec) continue;
      // the target row's vector travels with the first sources
      const uint4 xt = ldg16(tokens + (size_t)(d.row0 + hub_srow[h]) * D + (size_t)v * E);
      float acc[E];
#pragma unroll
      for (int q = 0; q < E; ++q) acc[q] = 0.f;
      #pragma unroll 1
      for (int k0 = 0; k0 < n; k0 += MHUB) {
        uint4 u[MHUB];
        float a[MHUB];
#pragma unroll
        for (int j = 0; j < MHUB; ++j) {
          const bool on = k0 + j < n;
          a[j] = on ? hw[b0 + k0 + j] : 0.f;
          u[j] = on ? ldg16(pbase + (size_t)hsrc[b0 + k0 + j] * D + (size_t)v * E) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int j = 0; j < MHUB; ++j) {
          float f[E];
          unpack(u[j], f, (const T*)nullptr);
#pragma unroll
          for (int q = 0; q < E; ++q) acc[q] = fmaf(a[j], f[q], acc[q]);
        }
      }
      T* dst = out + (size_t)(d.out_row0 + d.n_cls + hub_t[h]) * D;
      float x[E];
      unpack(xt, x, (const T*)nullptr);
      const float inv_den = hub_inv[h];
#pragma unroll
      for (int q = 0; q < E; ++q) acc[q] = (x[q] + acc[q]) * inv_den;
      reinterpret_cast<uint4*>(dst)[v] = pack(acc, (const T*)nullptr);
    }
  }
  FICOCO_PHASE(2, 5);
}

}  // namespace ficoco
