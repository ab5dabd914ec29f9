// Correlate stage on the 5th-generation tensor cores (bf16 tokens; FiCoCo-V, and FiCoCo-L with its
// text-bridged term added in the epilogue).
//
// One CTA owns a tile of discarded tokens (rows of the accumulator, one TMEM lane each) and
// one column split (<= 256 preserved tokens) of one image.  A tile has up to 128 rows, or up
// to 256 as two sub-tiles that share the gathered column tile and accumulate in adjacent TMEM
// column ranges:
//   warps 0-3, 5-8  gather the token rows with 16-byte cp.async into a ring of 128B-swizzled,
//              K-major shared-memory tiles (64 bf16 of the hidden dimension per stage);
//   warp  4    allocates TMEM and issues tcgen05.mma (M = 128, N = columns rounded to 16,
//              K = 16 per instruction, fp32 accumulation of exact bf16 products), one per
//              sub-tile and k-step;
//   warps 0-3, 5-8  afterwards read TMEM lanes back with tcgen05.ld (warps 0-3 the lower half
//              of the columns, warps 5-8 the upper half of the same lanes), scale by
//              rn_i * rn_j to cosines and keep each row's L <= LCAP largest entries in registers.
// Rows / columns past the valid range are never loaded: their shared memory is garbage that
// only reaches accumulator rows / columns the epilogue ignores.
// Every wait is bounded; on a timeout the CTA raises STATUS_TIMEOUT, drains its copies,
// frees its TMEM and returns.
#pragma once
#include <limits.h>
#include <math_constants.h>
#include "async_ops.cuh"
#include "common.cuh"
#include "kernels_correlate.cuh"

namespace ficoco {

constexpr int UM = 128;          // accumulator rows per MMA (one TMEM lane each)
constexpr int UM_SUB = 2;        // row sub-tiles per CTA: up to 256 discarded tokens share one gathered column tile
constexpr int UN_MAX = 256;      // accumulator columns per CTA
constexpr int UKB = 64;          // bf16 elements per k-block (one 128-byte swizzle row)
constexpr int UTHREADS = 288;    // warps 0-3 and 5-8 gather + epilogue, warp 4 MMA
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// K-major, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);   // start address, 16-byte units
  d |= (uint64_t)1 << 16;                      // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;            // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                      // descriptor version for sm_100
  d |= (uint64_t)2 << 61;                      // SWIZZLE_128B
  return d;
}
// kind::f16 instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t umma_idesc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(UM >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
               ::"r"(smem_u32(bar)) : "memory");
}
// 32 consecutive accumulator columns of this thread's TMEM lane; completes at tmem_ld_wait().
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// 16 consecutive accumulator columns of this thread's TMEM lane; completes at tmem_ld_wait().
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}

// Top-L of one accumulator row over the columns [c_lo, c_hi) (multiples of 16).  The code is
// kept small on purpose (a rolled loop over 16-column TMEM loads): it runs once per CTA, so a
// long unrolled body would be paid for in instruction-cache misses.  Insertion is branch-free:
// once a value is placed the rest of the list shifts down; '>' keeps the lower column first
// among equal values because columns arrive in ascending order.
// v / ix: descending list, -inf / INT_MAX in empty slots.  Warp-collective (tcgen05.ld).
// FiCoCo-L adds the text-bridged term: tS (this row's text->vision weights, element k at
// tS[k * s_stride]) and tT ([M][t_stride], one row per text token over the CTA's columns) sit in
// shared memory; C = gamma * cosine + t_scale * sum_k tS_k tT_kc.  tT == nullptr: FiCoCo-V.
template <int LCAP>
__device__ __forceinline__ void epilogue_scan(uint32_t tmem_lane, int c_lo, int c_hi, int ncols, int col_begin,
                                              float rs, const float* rnT, bool row_valid, int L,
                                              float (&v)[LCAP], int (&ix)[LCAP], const float* tS, int s_stride,
                                              const float* tT, int t_stride, int M, float gamma, float t_scale) {
#pragma unroll
  for (int k = 0; k < LCAP; ++k) { v[k] = -CUDART_INF_F; ix[k] = INT_MAX; }
  const int cmax = row_valid ? min(ncols, c_hi) : 0;
#pragma unroll 1
  for (int c0 = c_lo; c0 < c_hi; c0 += 16) {
    uint32_t r[16];
    tmem_ld16_issue(tmem_lane + (uint32_t)c0, r);
    float tx[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) tx[j] = 0.f;
    if (tT != nullptr) {
      #pragma unroll 1
      for (int k = 0; k < M; ++k) {
        const float a = tS[(size_t)k * s_stride];
        const float4* q = reinterpret_cast<const float4*>(tT + (size_t)k * t_stride + c0);
#pragma unroll
        for (int j4 = 0; j4 < 4; ++j4) {
          const float4 t4 = q[j4];
          tx[4 * j4 + 0] = fmaf(a, t4.x, tx[4 * j4 + 0]);
          tx[4 * j4 + 1] = fmaf(a, t4.y, tx[4 * j4 + 1]);
          tx[4 * j4 + 2] = fmaf(a, t4.z, tx[4 * j4 + 2]);
          tx[4 * j4 + 3] = fmaf(a, t4.w, tx[4 * j4 + 3]);
        }
      }
    }
    tmem_ld_wait();
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const int c = c0 + j;
      float cv = gamma * ((rs * rnT[c]) * __uint_as_float(r[j])) + t_scale * tx[j];
      if (!(c < cmax)) cv = -CUDART_INF_F;           // also drops NaN-free padding columns
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

// Dynamic shared memory: [1024-aligned] ring of NSTAGE stages, each an A tile (a_bytes: the
// valid source rows rounded up to 8, x 128 B) followed by a B tile (column rows x 128 B).  An
// MMA always reads 128 A rows; rows past a_bytes alias the B tile (or the slack the host adds
// behind the ring) and only feed accumulator rows that are never read.
template <int NSTAGE, int LCAP>
__global__ void __launch_bounds__(UTHREADS, 2) k_correlate_umma(
    const __nv_bfloat16* __restrict__ tokens, int D, const ImgDesc* __restrict__ desc,
    const WorkItem* __restrict__ work, const float* __restrict__ rn,
    const int* __restrict__ S_idx, const int* __restrict__ T_idx,
    float* __restrict__ part_val, int* __restrict__ part_idx, unsigned* __restrict__ status,
    int stage_bytes, int a_bytes, int tmem_cols, int* __restrict__ img_done, int* __restrict__ corr_cnt,
    float* __restrict__ tau_out, int* __restrict__ e_tgt, float* __restrict__ e_w, float* __restrict__ e_c,
    const float* __restrict__ tmean, int M, int NV, float gamma, unsigned long long wait_ns) {
  extern __shared__ unsigned char um_raw[];
  __shared__ uint64_t full_bar[NSTAGE], empty_bar[NSTAGE], acc_bar;
  __shared__ uint32_t tmem_base_s;
  __shared__ int rowS[UM * UM_SUB], rowT[UN_MAX];
  __shared__ float rnT[UN_MAX];
  __shared__ int failed, acc_committed, is_last, dead;

  FICOCO_PHASE_BEGIN(1);
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  const int L = d.list_len;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int col_begin = w.aux * d.cols_per_split;
  const int ncols = min(d.n_tgt, col_begin + d.cols_per_split) - col_begin;   // 1..256
  const int n_pad = (ncols + 15) & ~15;
  const int nkb = D / UKB;
  const int nsub = (w.nrows + UM - 1) / UM;       // 1 or 2; sub-tile s accumulates in TMEM columns [s * n_pad, (s + 1) * n_pad)
  const uint32_t ring = (smem_u32(um_raw) + 1023u) & ~1023u;

  if (tid == 0) {
    for (int s = 0; s < NSTAGE; ++s) { mbar_init(&full_bar[s], 8); mbar_init(&empty_bar[s], 1); }
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
  // Everything above touches only launch-constant plan data and this CTA's own resources, so it
  // may run while the filter grid is still finishing; the index lists and norms it wrote are
  // read below.  The dependent (merge) grid is released only after this wait, so by the time
  // any of its blocks starts, the filter grid is complete as well.
  FICOCO_PHASE(1, 1);
  grid_dep_wait();
  grid_dep_launch();
  FICOCO_PHASE(1, 2);
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
  if (tid < UM * UM_SUB) rowS[tid] = tid < w.nrows ? checked_index(S_idx[d.src0 + w.r0 + tid], d.np, status) : -1;
  for (int c = tid; c < UN_MAX; c += UTHREADS) {
    const int p = c < ncols ? checked_index(T_idx[d.tgt0 + col_begin + c], d.np, status) : -1;
    rowT[c] = p;
    rnT[c] = p >= 0 ? rn[d.patch0 + p] : 0.f;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  FICOCO_PHASE(1, 3);

  if (warp != 4) {
    // ---------------- producers (all eight epilogue warps): gather rows, 16 bytes per copy -------
    // Thread pt copies chunk (pt & 7) of rows (pt >> 3) + 32 i of the A tile and of the B tile.
    // Row offsets stay in registers and the swizzled destination advances by a constant
    // (32 rows = 4 KB), so a copy costs an add and the cp.async itself.
    const int pt = warp < 4 ? tid : tid - 32;
    const int chunk = pt & 7;
    const int rsub = pt >> 3;           // 0..31
    uint32_t offA[UM * UM_SUB / 32], offB[UN_MAX / 32];
    uint32_t onA = 0, onB = 0;
#pragma unroll
    for (int i = 0; i < UM * UM_SUB / 32; ++i) {
      const int r = rsub + 32 * i;
      const bool on = r < w.nrows;
      offA[i] = on ? (uint32_t)rowS[r] * (uint32_t)D : 0u;
      onA |= on ? 1u << i : 0u;
    }
#pragma unroll
    for (int i = 0; i < UN_MAX / 32; ++i) {
      const int r = rsub + 32 * i;
      const bool on = r < ncols;
      offB[i] = on ? (uint32_t)rowT[r] * (uint32_t)D : 0u;
      onB |= on ? 1u << i : 0u;
    }
    const uint32_t dsw = (uint32_t)((rsub >> 3) * 1024 + (rsub & 7) * 128 + ((chunk ^ (rsub & 7)) << 4));
    const __nv_bfloat16* tbase = tokens + (size_t)(d.row0 + d.n_cls) * D + chunk * 8;
    bool ok = true;
    // a stage is published LAG iterations after its copies were issued; LAG < NSTAGE - 1 leaves
    // the MMA a full iteration to drain a stage before the producer needs it again
    constexpr int LAG = NSTAGE >= 3 ? NSTAGE - 2 : 1;
    for (int kb = 0; kb < nkb + LAG; ++kb) {
      if (kb < nkb) {
        const int s = kb % NSTAGE;
        if (kb >= NSTAGE && ok) ok = mbar_wait(&empty_bar[s], ((kb / NSTAGE) - 1) & 1, wait_ns);
        if (ok) {
          const uint32_t a0 = ring + (uint32_t)s * stage_bytes + dsw;
          const uint32_t b0 = a0 + (uint32_t)a_bytes;
          const __nv_bfloat16* src = tbase + (size_t)kb * UKB;
#pragma unroll
          for (int i = 0; i < UM * UM_SUB / 32; ++i)
            if (onA >> i & 1u) cp_async16(a0 + i * 4096, src + offA[i]);
#pragma unroll
          for (int i = 0; i < UN_MAX / 32; ++i)
            if (onB >> i & 1u) cp_async16(b0 + i * 4096, src + offB[i]);
        }
      }
      cp_async_commit();
      // the group committed LAG iterations ago has landed: publish that stage
      const int done = kb - LAG;
      if (done >= 0) {
        cp_async_wait<LAG>();
        fence_proxy_async();
        // one arrival per producer warp: 256 arrivals per stage queue up on the barrier word
        __syncwarp();
        if (lane == 0) mbar_arrive(&full_bar[done % NSTAGE]);
      }
    }
    cp_async_wait<0>();
    FICOCO_PHASE(1, 4);
    if (!ok) { atomicOr(status, STATUS_TIMEOUT); failed = 1; }
    bool acc_ok = ok && mbar_wait(&acc_bar, 0, wait_ns);
    FICOCO_PHASE(1, 5);
    if (!acc_ok) { atomicOr(status, STATUS_TIMEOUT); failed = 1; }
    acc_ok = __all_sync(0xFFFFFFFFu, acc_ok);          // tcgen05.ld below is warp-collective
    tc_fence_after();
    // FiCoCo-L: the head-mean text->vision weights of this tile's columns and rows go into the idle
    // ring, behind the area the two epilogue halves use to hand over their lists
    const int rows_pad = nsub * UM;
    float* tT = nullptr;
    float* tSb = nullptr;
    const float t_scale = tmean != nullptr ? (1.0f - gamma) / (float)M : 0.f;
    if (tmean != nullptr) {
      tT = reinterpret_cast<float*>(um_raw + (ring - smem_u32(um_raw)) + (size_t)UM * LCAP * 8);
      tSb = tT + (size_t)M * n_pad;
      const float* tb = tmean + (size_t)w.img * M * NV;
      // eight gathers in flight per thread (one at a time cost a round trip each: 13 us per CTA)
      #pragma unroll 1
      for (int i0 = pt; i0 < M * n_pad; i0 += 8 * 256) {
        float q[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int i = i0 + 256 * j;
          const int k = i / n_pad, cc = i - k * n_pad;
          q[j] = (i < M * n_pad && cc < ncols) ? __ldg(tb + (size_t)k * NV + rowT[cc]) : 0.f;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (i0 + 256 * j < M * n_pad) tT[i0 + 256 * j] = q[j];
      }
      #pragma unroll 1
      for (int i0 = pt; i0 < M * rows_pad; i0 += 8 * 256) {
        float q[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int i = i0 + 256 * j;
          const int k = i / rows_pad, rr = i - k * rows_pad;
          q[j] = (i < M * rows_pad && rr < w.nrows) ? __ldg(tb + (size_t)k * NV + rowS[rr]) : 0.f;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (i0 + 256 * j < M * rows_pad) tSb[i0 + 256 * j] = q[j];
      }
      cta_sync(1, 256);
    }
    if (warp < 4) {
    // ---------------- epilogue: lane = accumulator row ---------------------------------------
    // this warp scans the lower half of the columns, its helper warp (same TMEM lanes) the
    // upper half; the helper's list comes back through the (now idle) operand ring
    const int c_mid = ((n_pad / 16 + 1) / 2) * 16;
    #pragma unroll 1
    for (int sub = 0; sub < nsub; ++sub) {
      const int row = sub * UM + tid;                  // TMEM lane == accumulator row of the sub-tile
      const bool row_valid = row < w.nrows;
      const float rs = row_valid ? rn[d.patch0 + rowS[row]] : 0.f;
      float v[LCAP];
      int ix[LCAP];
      if (acc_ok && sub * UM + warp * 32 < w.nrows)
        epilogue_scan<LCAP>(tmem_base + (uint32_t)(sub * n_pad) + ((uint32_t)(warp * 32) << 16), 0, c_mid, ncols,
                            col_begin, rs, rnT, row_valid, L, v, ix, tSb + row, rows_pad, tT, n_pad, M, gamma,
                            t_scale);
      else {
#pragma unroll
        for (int k = 0; k < LCAP; ++k) { v[k] = -CUDART_INF_F; ix[k] = INT_MAX; }
      }
      cta_sync(1, 256);                                // helper lists of this sub-tile are in shared memory
      {
        const float* hv = reinterpret_cast<const float*>(um_raw + (ring - smem_u32(um_raw)));
        const int* hi = reinterpret_cast<const int*>(hv + UM * LCAP);
        #pragma unroll 1                               // rolled: the body is a full insertion
        for (int e = 0; e < L; ++e) {
          {
            float cv = hv[tid * LCAP + e];
            int ci = hi[tid * LCAP + e];
            bool shift = ci == INT_MAX;                // empty helper slot: nothing to insert
            if (!shift) {
              shift = false;
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
      if (sub + 1 < nsub) cta_sync(1, 256);            // the helpers may reuse the hand-over area
    }
    } else {
    // ---------------- epilogue helpers: upper half of the columns --------------------------------
    const int grp = warp & 3;                          // TMEM lanes this warp may read
    const int c_mid = ((n_pad / 16 + 1) / 2) * 16;
    float* hv = reinterpret_cast<float*>(um_raw + (ring - smem_u32(um_raw)));
    int* hi = reinterpret_cast<int*>(hv + UM * LCAP);
    #pragma unroll 1
    for (int sub = 0; sub < nsub; ++sub) {
      const int lrow = grp * 32 + lane;
      const int row = sub * UM + lrow;
      const bool row_valid = row < w.nrows;
      const float rs = row_valid ? rn[d.patch0 + rowS[row]] : 0.f;
      float v[LCAP];
      int ix[LCAP];
      if (acc_ok && sub * UM + grp * 32 < w.nrows)
        epilogue_scan<LCAP>(tmem_base + (uint32_t)(sub * n_pad) + ((uint32_t)(grp * 32) << 16), c_mid, n_pad, ncols,
                            col_begin, rs, rnT, row_valid, L, v, ix, tSb + row, rows_pad, tT, n_pad, M, gamma,
                            t_scale);
      else {
#pragma unroll
        for (int k = 0; k < LCAP; ++k) { v[k] = -CUDART_INF_F; ix[k] = INT_MAX; }
      }
#pragma unroll
      for (int k = 0; k < LCAP; ++k) { hv[lrow * LCAP + k] = v[k]; hi[lrow * LCAP + k] = ix[k]; }
      cta_sync(1, 256);
      if (sub + 1 < nsub) cta_sync(1, 256);
    }
    }
  } else {
    // ---------------- MMA issuer (one lane) ---------------------------------------------------
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(n_pad);
      bool ok = true;
      for (int kb = 0; kb < nkb && ok; ++kb) {
        const int s = kb % NSTAGE;
        ok = mbar_wait(&full_bar[s], (kb / NSTAGE) & 1, wait_ns);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a0 = ring + (uint32_t)s * stage_bytes;
        const uint64_t ad = umma_smem_desc(a0), bd = umma_smem_desc(a0 + (uint32_t)a_bytes);
#pragma unroll
        for (int k4 = 0; k4 < UKB / 16; ++k4) {
          umma_bf16(tmem_base, ad + (uint64_t)(k4 * 2), bd + (uint64_t)(k4 * 2), idesc,
                    (kb > 0 || k4 > 0) ? 1u : 0u);
          // second row sub-tile: A rows 128.. (UM * 128 bytes further, in 16-byte units), same B
          if (nsub > 1)
            umma_bf16(tmem_base + (uint32_t)n_pad, ad + (uint64_t)(UM * 128 / 16) + (uint64_t)(k4 * 2),
                      bd + (uint64_t)(k4 * 2), idesc, (kb > 0 || k4 > 0) ? 1u : 0u);
        }
        umma_commit(&empty_bar[s]);      // frees the stage once these MMAs have read it
      }
      if (ok) { umma_commit(&acc_bar); acc_committed = 1; }   // accumulator complete
      else { atomicOr(status, STATUS_TIMEOUT); failed = 1; }
    }
    __syncwarp();
  }

  FICOCO_PHASE(1, 6);
  tc_fence_before();
  __syncthreads();
  FICOCO_PHASE(1, 7);
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
  FICOCO_PHASE(1, 8);
}

}  // namespace ficoco
