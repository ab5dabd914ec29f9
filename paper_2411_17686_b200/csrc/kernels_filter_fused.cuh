// Filter stage as one persistent kernel (Eq. 1, local penalty, top-N^S selection).
//
// Launched cooperatively with one CTA per SM at most, so all CTAs are co-resident.  Every CTA
// owns a fixed list of "pieces" (consecutive patch rows of one image).  Warp 16 streams the
// rows of its pieces, 16 rows (one bulk copy) per stage, into a shared-memory ring (TMA);
// the 16 consumer warps take one row each per stage.
//   pass 1  rn_i = 1/||x_i||, column sums of the normalised rows -> one partial per piece;
//           the piece's image counter is bumped;
//   pass 2  (rows read again, now L2-resident, with plain 16-byte loads, three rows in flight
//           per warp) once all pieces of the image are in:
//           v_i = rn_i (x_i . sum of partials) / Np,  s_i = cA v_i - (1 - cA) a_i;
//   select  images of up to 1024 tokens: every CTA that scored a piece waits until all of the
//           image's scores are in, runs the (short) selection on the whole image and writes the
//           outputs of its own tokens; larger images: the CTA that finishes the last piece runs
//           the selection alone.
// The inter-CTA waits are polls of per-image counters, bounded by elapsed time (wait_ns).  The
// counters exist twice; a launch uses the set of its parity and zeroes the other one, so a step
// that gave up half-way cannot leave counts behind for the step after the next.  The set a launch
// used is cleared by the merge grid of the same step (which runs once the filter grid is complete
// and before a later filter grid can start), so launches replayed from CUDA graphs, whose
// parities are fixed at capture, find their set clean in whatever order they run.
#pragma once
#include "async_ops.cuh"
#include "common.cuh"
#include "kernels_filter.cuh"

namespace ficoco {

constexpr int FWARPS = 16;        // consumer warps
constexpr int FROWS = 16;         // rows per ring stage (one 16-row bulk copy), one per consumer warp
constexpr int FFOLD = 8;          // rows of the fold buffer (warps w and w + 8 share a row)
constexpr int F_NCONS = 512;      // consumer threads
constexpr int F_THREADS = 544;    // + one producer warp
constexpr int F_MAXSTAGE = 16;
constexpr int F_MAXWON = 32;      // pieces per CTA (and therefore selections it can win)
static_assert(F_NCONS == SEL_SMALL_THREADS, "the short selection is written for the consumer threads");

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.b32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Poll until *p >= need.  Gives up after limit_ns, or at once when another CTA has already
// raised STATUS_TIMEOUT (its pieces will never arrive).  One thread calls this.
__device__ __forceinline__ bool poll_count(const int* p, int need, unsigned long long limit_ns,
                                           const unsigned* status) {
  unsigned long long t0 = 0;
  for (;;) {
    if (ld_acquire(p) >= need) return true;
    const unsigned long long t = global_ns();
    if (t0 == 0) t0 = t;
    else if (t - t0 > limit_ns) return false;
    if (*reinterpret_cast<const volatile unsigned*>(status) & STATUS_TIMEOUT) return false;
    __nanosleep(32);
  }
}

// The mean direction m (one float per column) is kept in shared memory so that a warp reads it
// without bank conflicts: with 8 columns per 16-byte vector, floats 0-3 of vector v live in plane
// A at 4v and floats 4-7 in plane B at 4(nvec + v); with 4 columns per vector there is one plane.
template <int E>
__device__ __forceinline__ int msum_slot(int c, int nvec) {
  const int v = c / E, e = c % E;
  return (e < 4 ? 0 : 4 * nvec) + 4 * v + (e & 3);
}

// Dot products of R rows (16-byte vectors u[r][k], vector lane + 32k of the row) with m, summed
// over the warp.  m is read once for all R rows.
template <class T, int VPL, int R>
__device__ __forceinline__ void score_rows(const uint4 (&u)[R][VPL], const float* msum, int nvec, int lane,
                                           float (&dot)[R]) {
  constexpr int E = VecTraits<T>::E;
#pragma unroll
  for (int r = 0; r < R; ++r) dot[r] = 0.f;
#pragma unroll
  for (int k = 0; k < VPL; ++k) {
    const int v = lane + 32 * k;
    const int vv = v < nvec ? v : 0;
    float m[E];
    const float4 ma = *reinterpret_cast<const float4*>(msum + 4 * vv);
    m[0] = ma.x; m[1] = ma.y; m[2] = ma.z; m[3] = ma.w;
    if (E == 8) {
      const float4 mb = *reinterpret_cast<const float4*>(msum + 4 * (nvec + vv));
      m[E - 4] = mb.x; m[E - 3] = mb.y; m[E - 2] = mb.z; m[E - 1] = mb.w;
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float f[E];
      unpack(u[r][k], f, (const T*)nullptr);
      float t = 0.f;
#pragma unroll
      for (int e = 0; e < E; ++e) t = fmaf(f[e], m[e], t);
      dot[r] += t;
    }
  }
#pragma unroll
  for (int r = 0; r < R; ++r) dot[r] = warp_sum(dot[r]);
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
    int nstage, int max_piece, int parity, int set_stride, unsigned long long wait_ns, int dbg_extra_arrivals,
    int dep_wait_first) {
  constexpr int E = VecTraits<T>::E;
  constexpr int F_P2B = VPL <= 4 ? 2 : 1;   // rows a warp scores together in pass 2 (and has in flight from L2)
  extern __shared__ __align__(128) unsigned char fs_raw[];
  __shared__ uint64_t full_bar[F_MAXSTAGE], empty_bar[F_MAXSTAGE];
  __shared__ SelectShared sel_sh;
  __shared__ SelectSmallShared sel_small_sh;
  // All CTAs of this grid are co-resident, so the next grid may be staged right away: its blocks
  // take over SMs as blocks of this grid exit and park until this grid has completed.
  grid_dep_launch();
  FICOCO_PHASE_BEGIN(0);
  __shared__ int won[F_MAXWON];
  __shared__ int nwon, failed;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int row_bytes = D * (int)sizeof(T);
  const int stage_bytes = FROWS * row_bytes;
  const int nvec = D / E;
  unsigned char* ring = fs_raw;
  float* fold = reinterpret_cast<float*>(fs_raw + (size_t)nstage * stage_bytes);   // [FFOLD][D], msum aliases fold[0]
  float* a_s = fold + (size_t)FFOLD * D;                                            // [max_piece]
  const int p_begin = cta_first[blockIdx.x], p_end = cta_first[blockIdx.x + 1];
  // counters of this launch: [0, B) pieces through pass 1, [B, 2B) pieces scored ([2B, 3B) unused).
  // The other set belongs to the launch before and the one after: it is zeroed here for the latter
  // (the launch before is complete: the correlate grid between the two waited for it).
  {
    // (the sets lie set_stride apart whatever the batch of this launch, so that launches of
    // different plans find and clear each other's counters)
    int* other = cnt + (parity ? 0 : set_stride);
    if (blockIdx.x == 0)
      for (int i = tid; i < set_stride; i += F_THREADS) other[i] = 0;
    cnt += parity ? set_stride : 0;
  }

  if (tid == 0) {
    for (int s = 0; s < nstage; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], FWARPS); }
    nwon = 0;
    failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // A step fed from the outputs of the step before it on the stream (a progressive schedule) is
  // still launched early, so that its blocks are in place and set up when that step ends, but
  // must not touch the tokens before then.
  if (dep_wait_first) grid_dep_wait();

  if (warp == FWARPS) {
    // ------------------------------- producer (pass 1 only) -------------------------------
    if (lane == 0) {
      int seq = 0;
      bool ok = true;
      for (int pi = p_begin; pi < p_end && ok; ++pi) {
        const WorkItem w = pieces[pi];
        const ImgDesc d = desc[w.img];
        const unsigned char* base =
            reinterpret_cast<const unsigned char*>(tokens + (size_t)(d.row0 + d.n_cls + w.r0) * D);
        for (int g = 0; g * FROWS < w.nrows && ok; ++g, ++seq) {
          const int s = seq % nstage;
          if (seq >= nstage) ok = mbar_wait(&empty_bar[s], ((seq / nstage) - 1) & 1, wait_ns);
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
  FICOCO_PHASE(0, 1);
  int seq = 0;
  bool ok = true;
  // The attention term of the first piece's rows depends on nothing this kernel computes: it is
  // fetched now, while the ring fills, instead of between the two passes.
  if (p_begin < p_end) {
    const WorkItem w = pieces[p_begin];
    const ImgDesc d = desc[w.img];
    const float inv_h = 1.0f / (float)H;
    for (int r = tid; r < w.nrows; r += F_NCONS) {
      const float* a = attn + d.attn0 + w.r0 + r;
      float t = 0.f;
      for (int h = 0; h < H; ++h) t += __ldg(a + (size_t)h * d.np);
      a_s[r] = t * inv_h;
    }
  }
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
      if (ok) ok = mbar_wait(&full_bar[s], (seq / nstage) & 1, wait_ns);
      const int r = g * FROWS + warp;
      if (r < w.nrows) {
        const unsigned char* rp = ring + (size_t)s * stage_bytes + (size_t)warp * row_bytes;
        uint4 u[VPL];
        float ssk[VPL];
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
          const int v = lane + 32 * k;
          u[k] = v < nvec ? *reinterpret_cast<const uint4*>(rp + (size_t)v * 16) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
          float f[E];
          unpack(u[k], f, (const T*)nullptr);
          float t = 0.f;
#pragma unroll
          for (int e = 0; e < E; ++e) t = fmaf(f[e], f[e], t);
          ssk[k] = t;
        }
        float ss = 0.f;
#pragma unroll
        for (int k = 0; k < VPL; ++k) ss += ssk[k];
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
    // fold the 16 warps in a fixed order -> partial of this piece: warps 0-7 store, warps 8-15
    // add into the row of warp - 8, then the 8 rows are summed per column
    if (warp < FFOLD) {
#pragma unroll
      for (int k = 0; k < VPL; ++k) {
        const int v = lane + 32 * k;
        if (v < nvec) {
          float4* dst = reinterpret_cast<float4*>(fold + (size_t)warp * D + (size_t)v * E);
          dst[0] = make_float4(acc[k][0], acc[k][1], acc[k][2], acc[k][3]);
          if (E == 8) dst[1] = make_float4(acc[k][E - 4], acc[k][E - 3], acc[k][E - 2], acc[k][E - 1]);
        }
      }
    }
    cta_sync(1, F_NCONS);
    if (warp >= FFOLD) {
#pragma unroll
      for (int k = 0; k < VPL; ++k) {
        const int v = lane + 32 * k;
        if (v < nvec) {
          float4* dst = reinterpret_cast<float4*>(fold + (size_t)(warp - FFOLD) * D + (size_t)v * E);
          float4 x = dst[0];
          x.x += acc[k][0]; x.y += acc[k][1]; x.z += acc[k][2]; x.w += acc[k][3];
          dst[0] = x;
          if (E == 8) {
            float4 y = dst[1];
            y.x += acc[k][E - 4]; y.y += acc[k][E - 3]; y.z += acc[k][E - 2]; y.w += acc[k][E - 1];
            dst[1] = y;
          }
        }
      }
    }
    cta_sync(1, F_NCONS);
    float* pout = partial + (size_t)(d.chunk0 + w.aux) * D;
    for (int c = tid; c < D; c += F_NCONS) {
      float t = 0.f;
#pragma unroll
      for (int ww = 0; ww < FFOLD; ++ww) t += fold[(size_t)ww * D + c];
      pout[c] = t;
    }
    cta_sync(1, F_NCONS);
    if (tid == 0) red_release_add(&cnt[w.img], 1);   // pairs with the ld.acquire poll of pass 2
  }
  if (!ok && lane == 0) { atomicOr(status, STATUS_TIMEOUT); failed = 1; }
  FICOCO_PHASE(0, 2);

  // pass 2: scores.  The last `nstage` row groups of pass 1 are still in the ring and are read
  // from there (only when every wait of pass 1 succeeded); the older ones are L2-resident and
  // are read with plain loads.
  const int first_kept = ok ? seq - nstage : seq;   // groups numbered >= this are in shared memory
  int seq2 = 0;
  for (int pi = p_begin; pi < p_end; ++pi) {
    const WorkItem w = pieces[pi];
    const ImgDesc d = desc[w.img];
    const int seq_piece = seq2;                     // number of this piece's first group
    seq2 += (w.nrows + FROWS - 1) / FROWS;
    if (tid == 0 && !poll_count(&cnt[w.img], d.n_chunks + dbg_extra_arrivals, wait_ns, status)) {
      atomicOr(status, STATUS_TIMEOUT);
      failed = 1;
    }
    if (pi == p_begin) FICOCO_PHASE(0, 3);
    const float inv_h = 1.0f / (float)H;
    for (int r = tid; pi > p_begin && r < w.nrows; r += F_NCONS) {     // attention term of a further piece
      const float* a = attn + d.attn0 + w.r0 + r;
      float t = 0.f;
      for (int h = 0; h < H; ++h) t += __ldg(a + (size_t)h * d.np);
      a_s[r] = t * inv_h;
    }
    cta_sync(1, F_NCONS);
    float* msum = fold;
    for (int c = tid; c < D; c += F_NCONS) {
      float t = 0.f;
      for (int k0 = 0; k0 < d.n_chunks; k0 += 8) {
        float q[8];
#pragma unroll
        for (int k = 0; k < 8; ++k)
          q[k] = k0 + k < d.n_chunks ? __ldcg(partial + (size_t)(d.chunk0 + k0 + k) * D + c) : 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) t += q[k];
      }
      msum[msum_slot<E>(c, nvec)] = t;
    }
    cta_sync(1, F_NCONS);
    if (pi == p_begin) FICOCO_PHASE(0, 4);
    const float inv_np = 1.0f / (float)d.np;
    const T* base = tokens + (size_t)(d.row0 + d.n_cls + w.r0) * D;
    // This warp owns line `warp` of every 16-row group of the piece.  Groups numbered below
    // g_res were overwritten in the ring and come from L2; the others are still in shared memory.
    const int G = (w.nrows + FROWS - 1) / FROWS;
    const int g_res = min(G, max(0, first_kept - seq_piece));
    // norms of the warp's rows, lane l holding the one of group l
    const int row_l = lane * FROWS + warp;
    const float rn_l = (lane < G && row_l < w.nrows) ? __ldcg(rn + d.patch0 + w.r0 + row_l) : 0.f;
    auto finish_row = [&](int g, float dot) {      // dot already summed over the warp
      const int r = g * FROWS + warp;
      const float rnv = g < 32 ? __shfl_sync(0xFFFFFFFFu, rn_l, g) : __ldcg(rn + d.patch0 + w.r0 + r);
      if (lane == 0 && r < w.nrows)
        s_raw[d.patch0 + w.r0 + r] = cA * (dot * rnv * inv_np) - (1.0f - cA) * a_s[r];
    };
    uint4 ub[F_P2B][VPL];
    auto load_batch = [&](int g0) {
#pragma unroll
      for (int jb = 0; jb < F_P2B; ++jb) {
        const int r = (g0 + jb) * FROWS + warp;
        const bool on = g0 + jb < g_res && r < w.nrows;
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
          const int v = lane + 32 * k;
          ub[jb][k] = (on && v < nvec) ? ldg16(base + (size_t)r * D + (size_t)v * E) : make_uint4(0, 0, 0, 0);
        }
      }
    };
    load_batch(0);
    // the rows in the ring are scored while the first batch from L2 is in flight
    #pragma unroll 1
    for (int g0 = g_res; g0 < G; g0 += F_P2B) {
      uint4 us[F_P2B][VPL];
#pragma unroll
      for (int jb = 0; jb < F_P2B; ++jb) {
        const int g = g0 + jb;
        const bool on = g < G && g * FROWS + warp < w.nrows;
        const unsigned char* rp =
            ring + (size_t)((seq_piece + g) % nstage) * stage_bytes + (size_t)warp * row_bytes;
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
          const int v = lane + 32 * k;
          us[jb][k] = (on && v < nvec) ? *reinterpret_cast<const uint4*>(rp + (size_t)v * 16) : make_uint4(0, 0, 0, 0);
        }
      }
      float dot[F_P2B];
      score_rows<T, VPL, F_P2B>(us, msum, nvec, lane, dot);
#pragma unroll
      for (int jb = 0; jb < F_P2B; ++jb)
        if (g0 + jb < G) finish_row(g0 + jb, dot[jb]);
    }
    #pragma unroll 1
    for (int g0 = 0; g0 < g_res; g0 += F_P2B) {
      float dot[F_P2B];
      score_rows<T, VPL, F_P2B>(ub, msum, nvec, lane, dot);
#pragma unroll
      for (int jb = 0; jb < F_P2B; ++jb)
        if (g0 + jb < g_res) finish_row(g0 + jb, dot[jb]);
      if (g0 + F_P2B < g_res) load_batch(g0 + F_P2B);
    }
    cta_sync(1, F_NCONS);
    if (tid == 0) {
      // release this piece's scores, and (for the CTA that arrives last) acquire everyone else's
      const int old = atom_acq_rel_add(&cnt[B + w.img], 1);
      if (d.np > SEL_SMALL_MAX && old == d.n_chunks - 1 && nwon < F_MAXWON) won[nwon++] = w.img;
    }
  }
  cta_sync(1, F_NCONS);

  FICOCO_PHASE(0, 5);
  if (failed) return;
  // Up to here the kernel wrote only scratch that no grid but a filter or correlate grid reads,
  // and those of the step before were complete before this grid could start.  The index lists
  // and outputs written below are read by the merge grid of the step before: wait for it.
  grid_dep_wait();
  FICOCO_PHASE(0, 6);
  // selections (the ring is idle now and serves as work area), image by image over this CTA's pieces
  int pi = p_begin;
  #pragma unroll 1
  while (pi < p_end) {
    const WorkItem w0 = pieces[pi];
    const ImgDesc d = desc[w0.img];
    int pj = pi, hi = w0.r0;
    while (pj < p_end && pieces[pj].img == w0.img) { hi = pieces[pj].r0 + pieces[pj].nrows; ++pj; }
    if (d.np <= SEL_SMALL_MAX) {
      select_small_prepare(d, penalty, ring, tid);
      if (tid == 0 && !poll_count(&cnt[B + w0.img], d.n_chunks, wait_ns, status)) {
        atomicOr(status, STATUS_TIMEOUT);
        failed = 1;
      }
      cta_sync(1, F_NCONS);
      if (failed) return;
      FICOCO_PHASE(0, 7);
      select_small(d, s_raw, pos, window, coef, penalty, s_pen, scores_out, S_idx, T_idx, kept_idx, pos_out,
                   status, ring, sel_small_sh, tid, 1, w0.r0, hi);
      // (the counters are not reset here: the next launch zeroes this launch's set, see the top)
      if (pj < p_end) cta_sync(1, F_NCONS);     // the work area is reused by the next image
    } else {
      bool mine = false;
      for (int k = 0; k < nwon; ++k) mine = mine || won[k] == w0.img;
      if (mine) {
        select_image(d, s_raw, pos, window, coef, penalty, s_pen, scores_out, S_idx, T_idx, kept_idx, pos_out,
                     status, ring, sel_sh, tid, F_NCONS, 1);
        if (pj < p_end) cta_sync(1, F_NCONS);
      }
    }
    pi = pj;
  }
  FICOCO_PHASE(0, 8);
}

}  // namespace ficoco
