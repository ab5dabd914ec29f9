// Filter stage as one persistent kernel (Eq. 1, local penalty, top-N^S selection).
//
// Launched cooperatively with one CTA per SM at most, so all CTAs are co-resident.  Every CTA
// owns a fixed list of "pieces" (consecutive patch rows of one image).  Warp 8 streams the
// rows of its pieces, 8 rows per stage, into a shared-memory ring with bulk copies (TMA);
// the 8 consumer warps take one row each per stage.
//   pass 1  rn_i = 1/||x_i||, column sums of the normalised rows -> one partial per piece;
//           the piece's image counter is bumped;
//   pass 2  (rows streamed again, now from L2) once all pieces of the image are in:
//           v_i = rn_i (x_i . sum of partials) / Np,  s_i = cA v_i - (1 - cA) a_i;
//           the CTA that finishes the last piece of an image runs the local penalty and the
//           radix select for that image and resets the image's counters.
// The only inter-CTA waits are the bounded polls of the per-image counter between the passes.
#pragma once
#include "async_ops.cuh"
#include "common.cuh"
#include "kernels_filter.cuh"

namespace ficoco {

constexpr int FROWS = 8;          // rows per ring stage == consumer warps
constexpr int F_NCONS = 256;      // consumer threads
constexpr int F_THREADS = 288;    // + one producer warp
constexpr int F_MAXSTAGE = 16;
constexpr int F_MAXWON = 32;      // pieces per CTA (and therefore selections it can win)
constexpr int F_POLL_LIMIT = 1 << 20;

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.b32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

template <class T, int VPL>
__global__ void __launch_bounds__(F_THREADS, 1) k_filter_fused(
    const T* __restrict__ tokens, int D, const ImgDesc* __restrict__ desc,
    const WorkItem* __restrict__ pieces, const int* __restrict__ cta_first,
    float* __restrict__ rn, float* __restrict__ partial, const float* __restrict__ attn, int H, float cA,
    float* __restrict__ s_raw, int* __restrict__ cnt, int B,
    const int* __restrict__ pos, int window, float coef, int penalty, float* __restrict__ s_pen,
    float* __restrict__ scores_out, int* __restrict__ S_idx, int* __restrict__ T_idx,
    int* __restrict__ kept_idx, int* __restrict__ pos_out, unsigned* __restrict__ status,
    int nstage, int max_piece) {
  constexpr int E = VecTraits<T>::E;
  extern __shared__ __align__(128) unsigned char fs_raw[];
  __shared__ uint64_t full_bar[F_MAXSTAGE], empty_bar[F_MAXSTAGE];
  __shared__ SelectShared sel_sh;
  __shared__ int won[F_MAXWON];
  __shared__ int nwon, failed;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int row_bytes = D * (int)sizeof(T);
  const int stage_bytes = FROWS * row_bytes;
  const int nvec = D / E;
  unsigned char* ring = fs_raw;
  float* fold = reinterpret_cast<float*>(fs_raw + (size_t)nstage * stage_bytes);   // [8][D], msum aliases fold[0]
  float* a_s = fold + (size_t)FROWS * D;                                           // [max_piece]
  const int p_begin = cta_first[blockIdx.x], p_end = cta_first[blockIdx.x + 1];

  if (tid == 0) {
    for (int s = 0; s < nstage; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], FROWS); }
    nwon = 0;
    failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp == FROWS) {
    // ------------------------------- producer ---------------------------------------------
    if (lane == 0) {
      int seq = 0;
      bool ok = true;
      for (int pass = 0; pass < 2 && ok; ++pass)
        for (int pi = p_begin; pi < p_end && ok; ++pi) {
          const WorkItem w = pieces[pi];
          const ImgDesc d = desc[w.img];
          const unsigned char* base =
              reinterpret_cast<const unsigned char*>(tokens + (size_t)(d.row0 + d.n_cls + w.r0) * D);
          for (int g = 0; g * FROWS < w.nrows && ok; ++g, ++seq) {
            const int s = seq % nstage;
            if (seq >= nstage) ok = mbar_wait(&empty_bar[s], ((seq / nstage) - 1) & 1);
            if (!ok) break;
            const int rows = min(FROWS, w.nrows - g * FROWS);
            mbar_expect_tx(&full_bar[s], (uint32_t)(rows * row_bytes));
            bulk_load(ring + (size_t)s * stage_bytes, base + (size_t)g * stage_bytes,
                      (uint32_t)(rows * row_bytes), &full_bar[s]);
          }
        }
      if (!ok) { atomicOr(status, STATUS_TIMEOUT); failed = 1; }
    }
    return;
  }

  // --------------------------------- consumers ----------------------------------------------
  int seq = 0;
  bool ok = true;
  // pass 1: norms and column sums
  for (int pi = p_begin; pi < p_end; ++pi) {
    const WorkItem w = pieces[pi];
    const ImgDesc d = desc[w.img];
    float acc[VPL][E];
#pragma unroll
    for (int k = 0; k < VPL; ++k)
#pragma unroll
      for (int e = 0; e < E; ++e) acc[k][e] = 0.f;
    for (int g = 0; g * FROWS < w.nrows; ++g, ++seq) {
      const int s = seq % nstage;
      if (ok) ok = mbar_wait(&full_bar[s], (seq / nstage) & 1);
      const int r = g * FROWS + warp;
      if (r < w.nrows) {
        const unsigned char* rp = ring + (size_t)s * stage_bytes + (size_t)warp * row_bytes;
        uint4 u[VPL];
        float ss = 0.f;
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
          const int v = lane + 32 * k;
          u[k] = v < nvec ? *reinterpret_cast<const uint4*>(rp + (size_t)v * 16) : make_uint4(0, 0, 0, 0);
          float f[E];
          unpack(u[k], f, (const T*)nullptr);
#pragma unroll
          for (int e = 0; e < E; ++e) ss = fmaf(f[e], f[e], ss);
        }
        ss = warp_sum(ss);
        const float s1 = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
        if (lane == 0) rn[d.patch0 + w.r0 + r] = s1;
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
          float f[E];
          unpack(u[k], f, (const T*)nullptr);
#pragma unroll
          for (int e = 0; e < E; ++e) acc[k][e] = fmaf(f[e], s1, acc[k][e]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty_bar[s]);
    }
    // fold the 8 warps in a fixed order -> partial of this piece
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
      const int v = lane + 32 * k;
      if (v < nvec) {
#pragma unroll
        for (int e = 0; e < E; ++e) fold[(size_t)warp * D + (size_t)v * E + e] = acc[k][e];
      }
    }
    cta_sync(1, F_NCONS);
    float* pout = partial + (size_t)(d.chunk0 + w.aux) * D;
    for (int c = tid; c < D; c += F_NCONS) {
      float t = 0.f;
#pragma unroll
      for (int ww = 0; ww < FROWS; ++ww) t += fold[(size_t)ww * D + c];
      pout[c] = t;
    }
    __threadfence();
    cta_sync(1, F_NCONS);
    if (tid == 0) atomicAdd(&cnt[w.img], 1);
  }

  // pass 2: scores
  for (int pi = p_begin; pi < p_end; ++pi) {
    const WorkItem w = pieces[pi];
    const ImgDesc d = desc[w.img];
    if (tid == 0) {
      bool in = false;
      for (int it = 0; it < F_POLL_LIMIT && !in; ++it) {
        in = ld_acquire(&cnt[w.img]) >= d.n_chunks;
        if (!in) __nanosleep(64);
      }
      if (!in) { atomicOr(status, STATUS_TIMEOUT); failed = 1; }
    }
    cta_sync(1, F_NCONS);
    float* msum = fold;
    for (int c = tid; c < D; c += F_NCONS) {
      float t = 0.f;
      for (int k = 0; k < d.n_chunks; ++k) t += __ldcg(partial + (size_t)(d.chunk0 + k) * D + c);
      msum[c] = t;
    }
    const float inv_h = 1.0f / (float)H;
    for (int r = tid; r < w.nrows; r += F_NCONS) {
      const float* a = attn + d.attn0 + w.r0 + r;
      float t = 0.f;
      for (int h = 0; h < H; ++h) t += __ldg(a + (size_t)h * d.np);
      a_s[r] = t * inv_h;
    }
    cta_sync(1, F_NCONS);
    const float inv_np = 1.0f / (float)d.np;
    for (int g = 0; g * FROWS < w.nrows; ++g, ++seq) {
      const int s = seq % nstage;
      if (ok) ok = mbar_wait(&full_bar[s], (seq / nstage) & 1);
      const int r = g * FROWS + warp;
      if (r < w.nrows) {
        const unsigned char* rp = ring + (size_t)s * stage_bytes + (size_t)warp * row_bytes;
        float dot = 0.f;
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
          const int v = lane + 32 * k;
          if (v < nvec) {
            float f[E];
            unpack(*reinterpret_cast<const uint4*>(rp + (size_t)v * 16), f, (const T*)nullptr);
            const float* m = msum + (size_t)v * E;
#pragma unroll
            for (int e = 0; e < E; ++e) dot = fmaf(f[e], m[e], dot);
          }
        }
        dot = warp_sum(dot);
        if (lane == 0) {
          const float v_i = dot * __ldcg(rn + d.patch0 + w.r0 + r) * inv_np;
          s_raw[d.patch0 + w.r0 + r] = cA * v_i - (1.0f - cA) * a_s[r];
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty_bar[s]);
    }
    __threadfence();
    cta_sync(1, F_NCONS);
    if (tid == 0) {
      const int old = atomicAdd(&cnt[B + w.img], 1);
      if (old == d.n_chunks - 1 && nwon < F_MAXWON) won[nwon++] = w.img;
      __threadfence();
    }
  }
  if (!ok && lane == 0) { atomicOr(status, STATUS_TIMEOUT); failed = 1; }
  cta_sync(1, F_NCONS);

  // selections this CTA won (the ring is idle now and serves as work area)
  if (failed) return;
  const int nw = nwon;
  for (int k = 0; k < nw; ++k) {
    const int img = won[k];
    const ImgDesc d = desc[img];
    uint32_t* keys = reinterpret_cast<uint32_t*>(ring);
    unsigned long long* win = reinterpret_cast<unsigned long long*>(ring + (((size_t)d.np * 4 + 7) & ~(size_t)7));
    select_image(d, s_raw, pos, window, coef, penalty, s_pen, scores_out, S_idx, T_idx, kept_idx, pos_out,
                 status, keys, win, sel_sh, tid, F_NCONS, 1);
    cta_sync(1, F_NCONS);
    if (tid == 0) { cnt[img] = 0; cnt[B + img] = 0; }
  }
}

}  // namespace ficoco
