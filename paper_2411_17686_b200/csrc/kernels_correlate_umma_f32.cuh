// Correlate stage for fp32 tokens on the 5th-generation tensor cores (FiCoCo-V).
//
// The tensor cores multiply bf16.  An fp32 value x is the sum of three bf16 terms,
//   h = bf16(x),  m = bf16(x - h),  l = bf16(x - h - m)        (x - h and x - h - m are exact in fp32),
// which together hold its 24 significant bits, and a product of two such sums is, up to terms
// below 2^-24 of it,
//   x y = h h' + h m' + m h' + m m' + h l' + l h'.
// The producers load fp32 token rows, split them in registers and write three K-major,
// 128B-swizzled bf16 tiles per operand.  The three column tiles [h' | m' | l'] lie back to back, so one
// MMA multiplies an A tile with several of them at once; per k-step the MMA warp issues
//   h x [h' | m' | l']  (N = 3 n),   m x [h' | m']  (N = 2 n),   l x [h']  (N = n)
// into three accumulator regions of their own (6 n TMEM columns): three independent accumulation
// chains instead of one chain of six small MMAs, which is what bounded the first version (a
// tcgen05.mma that accumulates into the columns of the one before it waits for it).  The epilogue adds
// the six partial products of an entry, smallest terms first; everything after that (cosines,
// top-L lists, threshold, alpha weights) is the code of the bf16 kernel.
//
// One CTA: up to 128 discarded tokens x up to 64 preserved tokens of one image, two stages of
// 64 hidden elements; thread (row r mod 32, 16-byte chunk c) of the 256 producers handles chunk c of
// rows r, r + 32, ... of both operands and keeps the next k-block's loads in flight while it
// converts the current one (a third register buffer spilled and was slower).  Every wait is bounded as in the bf16 kernel.
#pragma once
#include "kernels_correlate_umma.cuh"

namespace ficoco {

constexpr int UF_COLS = 64;      // preserved tokens per CTA (two rows per producer thread)
constexpr int UF_STAGES = 2;
constexpr int UF_AR = UM / 32;       // A rows per producer thread
constexpr int UF_BR = UF_COLS / 32;  // B rows per producer thread

// eight fp32 values -> the same eight as three bf16 terms (16 bytes each, element 0 in the low half)
__device__ __forceinline__ void split3(const float4& a, const float4& b, uint4& h, uint4& m, uint4& l) {
  const float x[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
  uint32_t hh[4], mm[4], ll[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const __nv_bfloat162 h2 = __floats2bfloat162_rn(x[2 * j], x[2 * j + 1]);
    const float2 hf = __bfloat1622float2(h2);
    const float r0 = x[2 * j] - hf.x, r1 = x[2 * j + 1] - hf.y;
    const __nv_bfloat162 m2 = __floats2bfloat162_rn(r0, r1);
    const float2 mf = __bfloat1622float2(m2);
    const __nv_bfloat162 l2 = __floats2bfloat162_rn(r0 - mf.x, r1 - mf.y);
    hh[j] = *reinterpret_cast<const uint32_t*>(&h2);
    mm[j] = *reinterpret_cast<const uint32_t*>(&m2);
    ll[j] = *reinterpret_cast<const uint32_t*>(&l2);
  }
  h = make_uint4(hh[0], hh[1], hh[2], hh[3]);
  m = make_uint4(mm[0], mm[1], mm[2], mm[3]);
  l = make_uint4(ll[0], ll[1], ll[2], ll[3]);
}

__device__ __forceinline__ void st_shared16(uint32_t addr, const uint4& v) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// Top-L of one accumulator row over the columns [c_lo, c_hi) (multiples of 16), the entry of column c
// being the sum of the six partial products at TMEM columns c + {5, 2, 4, 3, 1, 0} * nb (l h', h l',
// m m', m h', h m', h h').  Same list discipline as epilogue_scan().  Warp-collective (tcgen05.ld).
template <int LCAP>
__device__ __forceinline__ void epilogue_scan_split(uint32_t tmem_lane, int nb, int c_lo, int c_hi, int ncols,
                                                    int col_begin, float rs, const float* rnT, bool row_valid, int L,
                                                    float (&v)[LCAP], int (&ix)[LCAP]) {
#pragma unroll
  for (int k = 0; k < LCAP; ++k) { v[k] = -CUDART_INF_F; ix[k] = INT_MAX; }
  const int cmax = row_valid ? min(ncols, c_hi) : 0;
#pragma unroll 1
  for (int c0 = c_lo; c0 < c_hi; c0 += 16) {
    float a[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) a[j] = 0.f;
#pragma unroll 1
    for (int q = 0; q < 6; ++q) {
      const int blk = q == 0 ? 5 : q == 1 ? 2 : q == 2 ? 4 : q == 3 ? 3 : q == 4 ? 1 : 0;
      uint32_t r[16];
      tmem_ld16(tmem_lane + (uint32_t)(blk * nb + c0), r);
#pragma unroll
      for (int j = 0; j < 16; ++j) a[j] += __uint_as_float(r[j]);
    }
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const int c = c0 + j;
      float cv = (rs * rnT[c]) * a[j];
      if (!(c < cmax)) cv = -CUDART_INF_F;
      int ci = col_begin + c;
      bool ins = false;
#pragma unroll
      for (int k = 0; k < LCAP; ++k) {
        if (k < L) {
          const bool p = ins || cv > v[k];
          const float tv = v[k];
          const int ti = ix[k];
          v[k] = p ? cv : tv;
          ix[k] = p ? ci : ti;
          cv = p ? tv : cv;
          ci = p ? ti : ci;
          ins = p;
        }
      }
    }
  }
}

// Dynamic shared memory: [1024-aligned] two stages of [A_h | A_m | A_l | B_h | B_m | B_l]; an A tile has
// a_bytes (valid rows rounded up to 8, x 128 B), a B tile b_bytes (columns rounded to 16, x 128 B).  An
// MMA reads 128 A rows: rows past a tile alias the tiles behind it (or the slack the host adds behind
// the last stage) and only feed accumulator rows that are never read.
template <int LCAP>
__global__ void __launch_bounds__(UTHREADS, 1) k_correlate_umma_f32(
    const float* __restrict__ tokens, int D, const ImgDesc* __restrict__ desc,
    const WorkItem* __restrict__ work, const float* __restrict__ rn,
    const int* __restrict__ S_idx, const int* __restrict__ T_idx,
    float* __restrict__ part_val, int* __restrict__ part_idx, unsigned* __restrict__ status,
    int a_bytes, int b_bytes, int tmem_cols, int* __restrict__ img_done, int* __restrict__ corr_cnt,
    float* __restrict__ tau_out, int* __restrict__ e_tgt, float* __restrict__ e_w, float* __restrict__ e_c,
    unsigned long long wait_ns) {
  extern __shared__ unsigned char uf_raw[];
  __shared__ uint64_t full_bar[UF_STAGES], empty_bar[UF_STAGES], acc_bar;
  __shared__ uint32_t tmem_base_s;
  __shared__ int rowS[UM], rowT[UF_COLS];
  __shared__ float rnT[UF_COLS];
  __shared__ int failed, acc_committed, is_last, dead;

  FICOCO_PHASE_BEGIN(3);
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  const int L = d.list_len;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int col_begin = w.aux * d.cols_per_split;
  const int ncols = min(d.n_tgt, col_begin + d.cols_per_split) - col_begin;   // 1..64
  const int n_pad = (ncols + 15) & ~15;
  const int nb = b_bytes / 128;               // rows of a column tile: every CTA multiplies all of them
  const int nkb = D / UKB;
  const int stage_bytes = 3 * (a_bytes + b_bytes);
  const uint32_t ring = (smem_u32(uf_raw) + 1023u) & ~1023u;

  if (tid == 0) {
    for (int s = 0; s < UF_STAGES; ++s) { mbar_init(&full_bar[s], 8); mbar_init(&empty_bar[s], 1); }
    mbar_init(&acc_bar, 1);
    failed = 0;
    acc_committed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&tmem_base_s)), "r"((uint32_t)tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  FICOCO_PHASE(3, 1);
  grid_dep_wait();
  grid_dep_launch();
  FICOCO_PHASE(3, 2);
  // A filter grid that gave up left no valid index lists: do nothing but give the TMEM back.
  if (tid == 0) dead = (*reinterpret_cast<const volatile unsigned*>(status) & STATUS_TIMEOUT) ? 1 : 0;
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (dead) {
    if (warp == 4)
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base_s), "r"((uint32_t)tmem_cols)
                   : "memory");
    return;
  }
  if (tid < UM) rowS[tid] = tid < w.nrows ? checked_index(S_idx[d.src0 + w.r0 + tid], d.np, status) : -1;
  if (tid >= UM && tid < UM + UF_COLS) {
    const int c = tid - UM;
    const int p = c < ncols ? checked_index(T_idx[d.tgt0 + col_begin + c], d.np, status) : -1;
    rowT[c] = p;
    rnT[c] = p >= 0 ? rn[d.patch0 + p] : 0.f;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  FICOCO_PHASE(3, 3);

  if (warp != 4) {
    // ---------------- producers: load fp32, split, store three bf16 tiles per operand -------------
    const int pt = warp < 4 ? tid : tid - 32;
    const int chunk = pt & 7;
    const int rsub = pt >> 3;           // 0..31
    size_t offA[UF_AR], offB[UF_BR];
    uint32_t onA = 0, onB = 0;
#pragma unroll
    for (int i = 0; i < UF_AR; ++i) {
      const int r = rsub + 32 * i;
      const bool on = r < w.nrows;
      offA[i] = on ? (size_t)rowS[r] * (size_t)D : 0;
      onA |= on ? 1u << i : 0u;
    }
#pragma unroll
    for (int i = 0; i < UF_BR; ++i) {
      const int r = rsub + 32 * i;
      const bool on = r < ncols;
      offB[i] = on ? (size_t)rowT[r] * (size_t)D : 0;
      onB |= on ? 1u << i : 0u;
    }
    const uint32_t dsw = (uint32_t)((rsub >> 3) * 1024 + (rsub & 7) * 128 + ((chunk ^ (rsub & 7)) << 4));
    const float* tbase = tokens + (size_t)(d.row0 + d.n_cls) * D + chunk * 8;
    bool ok = true;
    float4 bufA[UF_AR + UF_BR][2], bufB[UF_AR + UF_BR][2];
    auto load = [&](float4 (&buf)[UF_AR + UF_BR][2], int kb) {
      const float* src = tbase + (size_t)kb * UKB;
#pragma unroll
      for (int i = 0; i < UF_AR; ++i)
        if (onA >> i & 1u) {
          buf[i][0] = __ldg(reinterpret_cast<const float4*>(src + offA[i]));
          buf[i][1] = __ldg(reinterpret_cast<const float4*>(src + offA[i]) + 1);
        }
#pragma unroll
      for (int i = 0; i < UF_BR; ++i)
        if (onB >> i & 1u) {
          buf[UF_AR + i][0] = __ldg(reinterpret_cast<const float4*>(src + offB[i]));
          buf[UF_AR + i][1] = __ldg(reinterpret_cast<const float4*>(src + offB[i]) + 1);
        }
    };
    auto store = [&](const float4 (&buf)[UF_AR + UF_BR][2], int kb) {
      const int s = kb % UF_STAGES;
      if (kb >= UF_STAGES && ok) ok = mbar_wait(&empty_bar[s], ((kb / UF_STAGES) - 1) & 1, wait_ns);
      if (ok) {
        const uint32_t a0 = ring + (uint32_t)s * stage_bytes + dsw;
        const uint32_t b0 = a0 + 3u * (uint32_t)a_bytes;
#pragma unroll
        for (int i = 0; i < UF_AR; ++i)
          if (onA >> i & 1u) {
            uint4 h, m, l;
            split3(buf[i][0], buf[i][1], h, m, l);
            st_shared16(a0 + i * 4096, h);
            st_shared16(a0 + (uint32_t)a_bytes + i * 4096, m);
            st_shared16(a0 + 2u * (uint32_t)a_bytes + i * 4096, l);
          }
#pragma unroll
        for (int i = 0; i < UF_BR; ++i)
          if (onB >> i & 1u) {
            uint4 h, m, l;
            split3(buf[UF_AR + i][0], buf[UF_AR + i][1], h, m, l);
            st_shared16(b0 + i * 4096, h);
            st_shared16(b0 + (uint32_t)b_bytes + i * 4096, m);
            st_shared16(b0 + 2u * (uint32_t)b_bytes + i * 4096, l);
          }
      }
      fence_proxy_async();          // the tiles were written through the generic proxy, the MMA reads them through the async proxy
      __syncwarp();
      if (lane == 0) mbar_arrive(&full_bar[s]);
    };
    load(bufA, 0);
    for (int kb = 0; kb < nkb; kb += 2) {
      if (kb + 1 < nkb) load(bufB, kb + 1);
      store(bufA, kb);
      if (kb + 1 < nkb) {
        if (kb + 2 < nkb) load(bufA, kb + 2);
        store(bufB, kb + 1);
      }
    }
    FICOCO_PHASE(3, 4);
    if (!ok) { atomicOr(status, STATUS_TIMEOUT); failed = 1; }
    bool acc_ok = ok && mbar_wait(&acc_bar, 0, wait_ns);
    FICOCO_PHASE(3, 5);
    if (!acc_ok) { atomicOr(status, STATUS_TIMEOUT); failed = 1; }
    acc_ok = __all_sync(0xFFFFFFFFu, acc_ok);          // tcgen05.ld below is warp-collective
    tc_fence_after();
    const int c_mid = ((n_pad / 16 + 1) / 2) * 16;
    float* hv = reinterpret_cast<float*>(uf_raw + (ring - smem_u32(uf_raw)));   // the operand ring is idle now
    int* hi = reinterpret_cast<int*>(hv + UM * LCAP);
    if (warp < 4) {
      // ---------------- epilogue: lane = accumulator row; lower half of the columns ----------------
      const int row = tid;
      const bool row_valid = row < w.nrows;
      const float rs = row_valid ? rn[d.patch0 + rowS[row]] : 0.f;
      float v[LCAP];
      int ix[LCAP];
      if (acc_ok && warp * 32 < w.nrows)
        epilogue_scan_split<LCAP>(tmem_base + ((uint32_t)(warp * 32) << 16), nb, 0, c_mid, ncols, col_begin, rs, rnT,
                                  row_valid, L, v, ix);
      else {
#pragma unroll
        for (int k = 0; k < LCAP; ++k) { v[k] = -CUDART_INF_F; ix[k] = INT_MAX; }
      }
      cta_sync(1, 256);                                // the helpers' lists are in shared memory
      #pragma unroll 1                                 // rolled: the body is a full insertion
      for (int e = 0; e < L; ++e) {
        {
          float cv = hv[tid * LCAP + e];
          int ci = hi[tid * LCAP + e];
          if (ci != INT_MAX) {
            bool shift = false;
#pragma unroll
            for (int k = 0; k < LCAP; ++k)
              if (k < L && (shift || toplist_better(cv, ci, v[k], ix[k]))) {
                const float tv = v[k]; const int ti = ix[k];
                v[k] = cv; ix[k] = ci; cv = tv; ci = ti;
                shift = true;
              }
          }
        }
      }
      if (row_valid) {
        const size_t o = (size_t)d.part0 + ((size_t)(w.r0 + row) * d.nsplit + w.aux) * L;
#pragma unroll
        for (int k = 0; k < LCAP; ++k)
          if (k < L) {
            part_val[o + k] = v[k];
            part_idx[o + k] = ix[k] == INT_MAX ? -1 : ix[k];
          }
      }
    } else {
      // ---------------- epilogue helpers: upper half of the columns of the same TMEM lanes ---------
      const int grp = warp & 3;
      const int lrow = grp * 32 + lane;
      const bool row_valid = lrow < w.nrows;
      const float rs = row_valid ? rn[d.patch0 + rowS[lrow]] : 0.f;
      float v[LCAP];
      int ix[LCAP];
      if (acc_ok && grp * 32 < w.nrows)
        epilogue_scan_split<LCAP>(tmem_base + ((uint32_t)(grp * 32) << 16), nb, c_mid, n_pad, ncols, col_begin, rs, rnT,
                                  row_valid, L, v, ix);
      else {
#pragma unroll
        for (int k = 0; k < LCAP; ++k) { v[k] = -CUDART_INF_F; ix[k] = INT_MAX; }
      }
#pragma unroll
      for (int k = 0; k < LCAP; ++k) { hv[lrow * LCAP + k] = v[k]; hi[lrow * LCAP + k] = ix[k]; }
      cta_sync(1, 256);
    }
  } else {
    // ---------------- MMA issuer (one lane): six products per k-step, smallest terms first ---------
    if (lane == 0) {
      const uint32_t id3 = umma_idesc_bf16(3 * nb), id2 = umma_idesc_bf16(2 * nb), id1 = umma_idesc_bf16(nb);
      bool ok = true;
      for (int kb = 0; kb < nkb && ok; ++kb) {
        const int s = kb % UF_STAGES;
        ok = mbar_wait(&full_bar[s], (kb / UF_STAGES) & 1, wait_ns);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a0 = ring + (uint32_t)s * stage_bytes;
        const uint64_t ah = umma_smem_desc(a0), am = umma_smem_desc(a0 + (uint32_t)a_bytes),
                       al = umma_smem_desc(a0 + 2u * (uint32_t)a_bytes);
        const uint64_t bh = umma_smem_desc(a0 + 3u * (uint32_t)a_bytes);   // [h' | m' | l'] start here
#pragma unroll
        for (int k4 = 0; k4 < UKB / 16; ++k4) {
          const uint64_t o = (uint64_t)(k4 * 2);
          const uint32_t acc = (kb > 0 || k4 > 0) ? 1u : 0u;
          umma_bf16(tmem_base, ah + o, bh + o, id3, acc);                       // h h' | h m' | h l'
          umma_bf16(tmem_base + (uint32_t)(3 * nb), am + o, bh + o, id2, acc);  // m h' | m m'
          umma_bf16(tmem_base + (uint32_t)(5 * nb), al + o, bh + o, id1, acc);  // l h'
        }
        umma_commit(&empty_bar[s]);      // frees the stage once these MMAs have read it
      }
      if (ok) { umma_commit(&acc_bar); acc_committed = 1; }   // accumulator complete
      else { atomicOr(status, STATUS_TIMEOUT); failed = 1; }
    }
    __syncwarp();
  }

  FICOCO_PHASE(3, 6);
  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    if (failed) {
      // MMAs may still be in flight: give them a bounded time to drain before freeing TMEM
      if (lane == 0) {
        if (!acc_committed) umma_commit(&acc_bar);
        mbar_wait(&acc_bar, 0, wait_ns);
      }
      __syncwarp();
    }
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)tmem_cols)
                 : "memory");
  }
  correlate_tail<LCAP>(d, w, (int)blockIdx.x - w.aux, img_done, part_val, part_idx, corr_cnt, tau_out, e_tgt, e_w, e_c,
                       &is_last);
  FICOCO_PHASE(3, 7);
}

}  // namespace ficoco
