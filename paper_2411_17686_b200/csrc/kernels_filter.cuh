// Filter stage (Eq. 1, local penalty, top-N^S selection).
#pragma once
#include "common.cuh"

namespace ficoco {

// ---------------------------------------------------------------------------------------
// Row norms.  One warp per vision token: rn_i = 1 / ||x_i||.  Used alone when the hidden
// size is too wide for the fused kernel below.
// ---------------------------------------------------------------------------------------
template <class T>
__global__ void __launch_bounds__(256) k_rownorm(const T* __restrict__ tokens, int D,
                                                 const ImgDesc* __restrict__ desc,
                                                 const WorkItem* __restrict__ work,
                                                 float* __restrict__ rn) {
  constexpr int E = VecTraits<T>::E;
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nvec = D / E;
  for (int r = warp; r < w.nrows; r += 8) {
    const T* row = tokens + (size_t)(d.row0 + d.n_cls + w.r0 + r) * D;
    float ss = 0.f;
    for (int v0 = lane; v0 < nvec; v0 += 32 * 8) {     // eight 16-byte loads in flight per lane
      uint4 u[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int v = v0 + 32 * k;
        u[k] = v < nvec ? ldg16(row + (size_t)v * E) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        float f[E];
        unpack(u[k], f, (const T*)nullptr);
#pragma unroll
        for (int e = 0; e < E; ++e) ss = fmaf(f[e], f[e], ss);
      }
    }
    ss = warp_sum(ss);
    if (lane == 0) rn[d.patch0 + w.r0 + r] = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
  }
}

// ---------------------------------------------------------------------------------------
// Column sums of the normalised tokens: partial[chunk][d] = sum_{i in chunk} rn_i x_id.
// The row mean of the cosine relation is x_hat_i . (1/N) sum_j x_hat_j, so this vector is
// all the first term of Eq. 1 needs.  One CTA per row chunk; a warp owns whole rows, each
// lane the 16-byte vectors lane, lane+32, ... of the column slab [c0, c0 + VPL*32*E).
// FUSED: the CTA also computes rn (requires the slab to cover the full row).
// Warps are folded into shared memory one after the other, so the result does not depend
// on scheduling.
// ---------------------------------------------------------------------------------------
template <class T, int VPL, bool FUSED>
__global__ void __launch_bounds__(256) k_colsum(const T* __restrict__ tokens, int D,
                                                const ImgDesc* __restrict__ desc,
                                                const WorkItem* __restrict__ work,
                                                float* __restrict__ rn,
                                                float* __restrict__ partial) {
  constexpr int E = VecTraits<T>::E;
  extern __shared__ float sm_acc[];  // VPL*32*E floats
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int slab = blockIdx.y;
  const int c0 = slab * (VPL * 32 * E);
  const int nvec = (min(D - c0, VPL * 32 * E)) / E;

  float acc[VPL][E];
#pragma unroll
  for (int k = 0; k < VPL; ++k)
#pragma unroll
    for (int e = 0; e < E; ++e) acc[k][e] = 0.f;

  const T* base = tokens + (size_t)(d.row0 + d.n_cls + w.r0) * D + c0;
  float* rn_out = rn + d.patch0 + w.r0;

  for (int r = warp; r < w.nrows; r += 16) {
    const int r2 = r + 8;
    const bool has2 = r2 < w.nrows;
    uint4 u[VPL], u2[VPL];
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
      const int v = lane + 32 * k;
      u[k] = (v < nvec) ? ldg16(base + (size_t)r * D + (size_t)v * E) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
      const int v = lane + 32 * k;
      u2[k] = (has2 && v < nvec) ? ldg16(base + (size_t)r2 * D + (size_t)v * E) : make_uint4(0, 0, 0, 0);
    }
    float s1, s2;
    if (FUSED) {
      float ss = 0.f, ss2 = 0.f;
#pragma unroll
      for (int k = 0; k < VPL; ++k) {
        float f[E];
        unpack(u[k], f, (const T*)nullptr);
#pragma unroll
        for (int e = 0; e < E; ++e) ss = fmaf(f[e], f[e], ss);
        unpack(u2[k], f, (const T*)nullptr);
#pragma unroll
        for (int e = 0; e < E; ++e) ss2 = fmaf(f[e], f[e], ss2);
      }
      ss = warp_sum(ss);
      ss2 = warp_sum(ss2);
      s1 = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
      s2 = ss2 > 0.f ? 1.0f / sqrtf(ss2) : 0.f;
      if (lane == 0) {
        rn_out[r] = s1;
        if (has2) rn_out[r2] = s2;
      }
    } else {
      s1 = rn_out[r];
      s2 = has2 ? rn_out[r2] : 0.f;
    }
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
      float f[E];
      unpack(u[k], f, (const T*)nullptr);
#pragma unroll
      for (int e = 0; e < E; ++e) acc[k][e] = fmaf(f[e], s1, acc[k][e]);
      unpack(u2[k], f, (const T*)nullptr);
#pragma unroll
      for (int e = 0; e < E; ++e) acc[k][e] = fmaf(f[e], s2, acc[k][e]);
    }
  }

  // fold the 8 warps in order
  for (int wv = 0; wv < 8; ++wv) {
    if (warp == wv) {
#pragma unroll
      for (int k = 0; k < VPL; ++k) {
        const int v = lane + 32 * k;
        float* dst = sm_acc + (size_t)v * E;
#pragma unroll
        for (int e = 0; e < E; ++e) dst[e] = (wv == 0) ? acc[k][e] : dst[e] + acc[k][e];
      }
    }
    __syncthreads();
  }
  float* out = partial + (size_t)(d.chunk0 + w.aux) * D + c0;
  for (int i = threadIdx.x; i < nvec * E; i += 256) out[i] = sm_acc[i];
}

// ---------------------------------------------------------------------------------------
// Eq. 1 (and the FiCoCo-L score): s_i = cA * v_i - (1 - cA) * a_i with
//   v_i = rn_i * (x_i . msum) / Np,   msum = sum of the image's column-sum partials,
//   a_i = (1/H) sum_h attn[h, i]      (FiCoCo-L: H = M rows of the head-mean block t).
// One CTA per row chunk, one warp per token for the dot product.
// ---------------------------------------------------------------------------------------
template <class T>
__global__ void __launch_bounds__(256) k_score(const T* __restrict__ tokens, int D,
                                               const ImgDesc* __restrict__ desc,
                                               const WorkItem* __restrict__ work,
                                               const float* __restrict__ rn,
                                               const float* __restrict__ partial,
                                               const float* __restrict__ attn, int H, float cA,
                                               float* __restrict__ s_raw) {
  constexpr int E = VecTraits<T>::E;
  extern __shared__ float sm[];  // msum[D], v[nrows]
  const WorkItem w = work[blockIdx.x];
  const ImgDesc d = desc[w.img];
  float* msum = sm;
  float* vrow = sm + D;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  for (int c = threadIdx.x; c < D; c += 256) {
    float s = 0.f;
    for (int k = 0; k < d.n_chunks; ++k) s += partial[(size_t)(d.chunk0 + k) * D + c];
    msum[c] = s;
  }
  __syncthreads();

  const int nvec = D / E;
  const float inv_np = 1.0f / (float)d.np;
  for (int r = warp; r < w.nrows; r += 8) {
    const T* row = tokens + (size_t)(d.row0 + d.n_cls + w.r0 + r) * D;
    float dot = 0.f;
    for (int v0 = lane; v0 < nvec; v0 += 32 * 8) {     // eight 16-byte loads in flight per lane
      uint4 u[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int v = v0 + 32 * k;
        u[k] = v < nvec ? ldg16(row + (size_t)v * E) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int v = v0 + 32 * k;
        if (v < nvec) {
          float f[E];
          unpack(u[k], f, (const T*)nullptr);
          const float* m = msum + (size_t)v * E;
#pragma unroll
          for (int e = 0; e < E; ++e) dot = fmaf(f[e], m[e], dot);
        }
      }
    }
    dot = warp_sum(dot);
    if (lane == 0) vrow[r] = dot * rn[d.patch0 + w.r0 + r] * inv_np;
  }
  __syncthreads();

  const float inv_h = 1.0f / (float)H;
  for (int r = threadIdx.x; r < w.nrows; r += 256) {
    const float* a = attn + d.attn0 + w.r0 + r;
    float s = 0.f;
    for (int h = 0; h < H; ++h) s += __ldg(a + (size_t)h * d.np);
    s_raw[d.patch0 + w.r0 + r] = cA * vrow[r] - (1.0f - cA) * (s * inv_h);
  }
}

// ---------------------------------------------------------------------------------------
// FiCoCo-L: head mean of the text->vision attention, t[b, k, i] = (1/H) sum_h A[b, h, k, i].
// One CTA per (sequence, text row).
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_head_mean(const float* __restrict__ attn, int H, int M,
                                                   int N, float* __restrict__ t) {
  const int b = blockIdx.x / M, k = blockIdx.x % M;
  const float inv_h = 1.0f / (float)H;
  const float* src = attn + ((size_t)b * H * M + k) * N;
  float* dst = t + ((size_t)b * M + k) * N;
  for (int i = threadIdx.x; i < N; i += 256) {
    float s = 0.f;
    for (int h0 = 0; h0 < H; h0 += 8) {      // eight heads in flight, added in head order
      float a[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) a[q] = h0 + q < H ? __ldg(src + (size_t)(h0 + q) * M * N + i) : 0.f;
#pragma unroll
      for (int q = 0; q < 8; ++q) s += a[q];
    }
    dst[i] = s * inv_h;
  }
}

// ---------------------------------------------------------------------------------------
// Local penalty + top-N^S selection of one image by `nthr` threads (tid 0..nthr-1) that
// synchronise on hardware barrier `bar`.
//   1. every alive token bids (score key, lower index wins ties) for its window with a
//      64-bit shared-memory max; the winner's score is multiplied by `coef`;
//   2. an 8-bit-per-pass radix select over order-preserving keys finds the N^S-th largest
//      score; ties at the threshold go to the lower index;
//   3. a block scan turns the membership flags into ascending index lists S and T, the kept
//      row indices and the surviving grid positions.
// The code runs once per image, so it is kept compact (rolled loops, not inlined): a long
// unrolled body would be paid for in instruction-cache misses.
// `work` is a shared-memory area of select_work_bytes(np, windows) bytes: the scores and grid
// positions are read from global memory once and kept there with the keys and window bids.
// ---------------------------------------------------------------------------------------
__host__ __device__ inline size_t select_work_bytes(int np, int nwin) {
  return (size_t)np * 12 + 8 + (size_t)nwin * 8 + 16 + 4 * 256 * sizeof(int);
}

struct SelectShared {
  int warp_tot[33];
  uint32_t prefix;
  int remaining;
};

__device__ __noinline__ void select_image(
    const ImgDesc& d, const float* s_raw, const int* __restrict__ pos, int window, float coef,
    int penalty, float* __restrict__ s_pen, float* __restrict__ scores_out, int* __restrict__ S_idx,
    int* __restrict__ T_idx, int* __restrict__ kept_idx, int* __restrict__ pos_out,
    unsigned* __restrict__ status, unsigned char* work, SelectShared& sh, int tid, int nthr, int bar) {
  const int np = d.np;
  uint32_t* keys = reinterpret_cast<uint32_t*>(work);
  float* sc = reinterpret_cast<float*>(work + (size_t)np * 4);
  int* pp = reinterpret_cast<int*>(work + (size_t)np * 8);
  unsigned long long* win = reinterpret_cast<unsigned long long*>(work + (((size_t)np * 12 + 7) & ~(size_t)7));
  const int nwc = (d.gw + window - 1) / window;
  const int nwr = (d.gh + window - 1) / window;
  const int nwin = penalty ? nwc * nwr : 0;
  // [4][256], one histogram per digit, 16-byte aligned
  int* hist = reinterpret_cast<int*>((reinterpret_cast<uintptr_t>(win + nwin) + 15) & ~(uintptr_t)15);

  #pragma unroll 1
  for (int i = tid; i < 4 * 256; i += nthr) hist[i] = 0;
  #pragma unroll 1
  for (int i = tid; i < nwin; i += nthr) win[i] = 0ull;
  #pragma unroll 1
  for (int i0 = tid; i0 < np; i0 += 4 * nthr) {    // four tokens' loads in flight per thread
    float a[4];
    int q[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = i0 + j * nthr;
      a[j] = i < np ? __ldcg(s_raw + d.patch0 + i) : 0.f;
      q[j] = (i < np && pos) ? pos[d.patch0 + i] : i;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = i0 + j * nthr;
      if (i < np) { sc[i] = a[j]; pp[i] = q[j]; }
    }
  }
  cta_sync(bar, nthr);

  // ---- local penalty ------------------------------------------------------------------
  if (penalty) {
    #pragma unroll 1
    for (int i = tid; i < np; i += nthr) {
      const int p = pp[i];
      if (p < 0 || p >= d.gh * d.gw) { atomicOr(status, STATUS_POS_RANGE); continue; }
      const int wid = (p / d.gw / window) * nwc + (p % d.gw) / window;
      const unsigned long long bid =
          ((unsigned long long)order_key(sc[i]) << 32) | (unsigned)(0xFFFFFFFFu - (unsigned)i);
      atomicMax(&win[wid], bid);
    }
    cta_sync(bar, nthr);
  }
  #pragma unroll 1
  for (int i = tid; i < np; i += nthr) {
    float s = sc[i];
    if (penalty) {
      const int p = pp[i];
      if (p >= 0 && p < d.gh * d.gw) {
        const int wid = (p / d.gw / window) * nwc + (p % d.gw) / window;
        if ((unsigned)(win[wid] & 0xFFFFFFFFull) == 0xFFFFFFFFu - (unsigned)i) s *= coef;
      }
    }
    s_pen[d.patch0 + i] = s;
    if (scores_out) scores_out[d.patch0 + i] = s;
    keys[i] = order_key(s);
  }
  cta_sync(bar, nthr);

  // ---- radix select: key of the n_src-th largest ------------------------------------------
  // Two barriers per digit: count, then the first warp finds the digit's bin; every digit has a
  // histogram of its own, zeroed up front.
  const int k = d.n_src;
  uint32_t thr = 0;       // threshold key
  int need_eq = 0;        // how many keys equal to thr are selected (lowest indices)
  if (k > 0 && k < np) {
    const int lane = tid & 31;
    uint32_t prefix = 0, mask = 0;
    int remaining = k;
    #pragma unroll 1
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      int* h = hist + 256 * pass;
      #pragma unroll 1
      for (int i = tid; i < np; i += nthr) {
        const uint32_t key = keys[i];
        if ((key & mask) == prefix) atomicAdd(&h[(key >> shift) & 255], 1);
      }
      cta_sync(bar, nthr);
      if (tid < 32) {
        // lane l owns bins 255-8l .. 248-8l (descending); find where the running count from
        // the top reaches `remaining`
        int c[8], tot = 0;
        {
          const int4 lo = *reinterpret_cast<const int4*>(h + 248 - 8 * lane);
          const int4 hi = *reinterpret_cast<const int4*>(h + 252 - 8 * lane);
          c[0] = hi.w; c[1] = hi.z; c[2] = hi.y; c[3] = hi.x;
          c[4] = lo.w; c[5] = lo.z; c[6] = lo.y; c[7] = lo.x;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) tot += c[j];
        int inc = tot;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          int n = __shfl_up_sync(0xFFFFFFFFu, inc, o);
          if (lane >= o) inc += n;
        }
        const int before = inc - tot;
        if (before < remaining && inc >= remaining) {
          int cum = before;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            if (cum < remaining && cum + c[j] >= remaining) {
              sh.prefix = prefix | ((uint32_t)(255 - 8 * lane - j) << shift);
              sh.remaining = remaining - cum;
            }
            cum += c[j];
          }
        }
      }
      cta_sync(bar, nthr);
      prefix = sh.prefix;
      remaining = sh.remaining;
      mask |= 0xFFu << shift;
    }
    thr = prefix;
    need_eq = remaining;
  }

  // ---- ordered compaction into S and T ------------------------------------------------------
  // Each thread takes a run of consecutive tokens; one block scan over packed counts
  // (greater-than in the high half, equal in the low half) places every run.
  {
    const int ipt = (np + nthr - 1) / nthr;
    const int i_lo = min(np, tid * ipt), i_hi = min(np, i_lo + ipt);
    int n_gt = 0, n_eq = 0;
    #pragma unroll 1
    for (int i = i_lo; i < i_hi; ++i) {
      const uint32_t key = keys[i];
      if (k >= np) ++n_gt;
      else if (k > 0) { n_gt += key > thr ? 1 : 0; n_eq += key == thr ? 1 : 0; }
    }
    int tot;
    const int packed = block_exclusive_scan((n_gt << 16) | n_eq, sh.warp_tot, &tot, bar, nthr);
    int gt_before = packed >> 16, eq_before = packed & 0xFFFF;
    #pragma unroll 1
    for (int i = i_lo; i < i_hi; ++i) {
      const uint32_t key = keys[i];
      bool gt, eq;
      if (k <= 0) { gt = false; eq = false; }
      else if (k >= np) { gt = true; eq = false; }
      else { gt = key > thr; eq = key == thr; }
      const bool sel = gt || (eq && eq_before < need_eq);
      const int sel_rank = gt_before + min(eq_before, need_eq);   // selected tokens before i
      if (sel) {
        S_idx[d.src0 + sel_rank] = i;
      } else {
        const int tp = i - sel_rank;
        T_idx[d.tgt0 + tp] = i;
        kept_idx[d.out_row0 + d.n_cls + tp] = d.n_cls + i;
        if (pos_out) pos_out[d.tgt0 + tp] = pp[i];
      }
      gt_before += gt ? 1 : 0;
      eq_before += eq ? 1 : 0;
    }
  }
  #pragma unroll 1
  for (int i = tid; i < d.n_cls; i += nthr) kept_idx[d.out_row0 + i] = i;
  #pragma unroll 1
  for (int i = tid; i < d.n_tail; i += nthr)
    kept_idx[d.out_row0 + d.n_cls + d.n_tgt + i] = d.n_cls + np + i;
}

// One CTA (512 or 1024 threads) per image.
__global__ void __launch_bounds__(1024) k_select(const ImgDesc* __restrict__ desc,
                                                 const float* __restrict__ s_raw,
                                                 const int* __restrict__ pos, int window, float coef,
                                                 int penalty, float* __restrict__ s_pen,
                                                 float* __restrict__ scores_out,
                                                 int* __restrict__ S_idx, int* __restrict__ T_idx,
                                                 int* __restrict__ kept_idx, int* __restrict__ pos_out,
                                                 unsigned* __restrict__ status) {
  extern __shared__ unsigned char sm_raw[];
  __shared__ SelectShared sh;
  const ImgDesc d = desc[blockIdx.x];
  select_image(d, s_raw, pos, window, coef, penalty, s_pen, scores_out, S_idx, T_idx, kept_idx, pos_out,
               status, sm_raw, sh, threadIdx.x, (int)blockDim.x, 0);
}

}  // namespace ficoco
