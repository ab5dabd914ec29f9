// C ABI of libficoco: context, plans, argument validation and kernel launches.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <mutex>
#include <vector>

#include "../../include/ficoco.h"
#include "common.cuh"
#include "kernels_correlate.cuh"
#include "kernels_correlate_umma.cuh"
#include "kernels_correlate_umma_f32.cuh"
#include "kernels_filter.cuh"
#include "kernels_filter_fused.cuh"
#include "kernels_merge.cuh"
#include "kernels_relation.cuh"

using namespace ficoco;

namespace {

constexpr int N_PLANS = 16;
constexpr int PART_PER_TOKEN = 64;   // partial top-list entries budgeted per token row
constexpr int OUT_ROWS_PER_CTA = MROWS_CTA;  // the merge kernel's copy batches are sized for it
constexpr int NSPLIT_MAX = 16;

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// host-buffer entry points: image groups pipelined over upload / kernels / download
constexpr int HOST_MAX_GROUPS = 8;
constexpr size_t HOST_GROUP_BYTES = 8u << 20;   // at least this many token bytes per group

struct PlanKey {
  int mode;  // 0 = V, 1 = L
  int dtype, batch, dim, n_text, has_cls, max_targets, avg;
  int rel = 0;  // 0: cosine relation of the tokens; 1 / 2: caller-supplied relation, by row / by column
  int conv = 0; // 1: "convergent correlation" ablation (one additional token per image, no merging)
  double eps;
  std::vector<int> ntok, keep, gh, gw;
  bool operator==(const PlanKey& o) const {
    return mode == o.mode && dtype == o.dtype && batch == o.batch && dim == o.dim &&
           n_text == o.n_text && has_cls == o.has_cls && max_targets == o.max_targets && avg == o.avg && rel == o.rel && conv == o.conv &&
           eps == o.eps && ntok == o.ntok && keep == o.keep && gh == o.gh && gw == o.gw;
  }
};

struct Plan {
  bool valid = false;
  unsigned long long stamp = 0;
  PlanKey key;
  // device tables (inside the slot)
  ImgDesc* d_desc = nullptr;
  WorkItem* d_rows = nullptr;
  WorkItem* d_corr = nullptr;
  WorkItem* d_out = nullptr;
  int n_rows = 0, n_corr = 0, n_out = 0;
  int out_rows_cta = 0;         // output rows per merge CTA
  // totals and maxima used to size launches and inspection copies
  int tot_patch = 0, tot_src = 0, tot_tgt = 0, tot_out_rows = 0;
  int max_np = 0, max_tgt = 0, max_src = 0, max_rc = 0, max_nwin_cells = 0, max_list = 0;
  // fused persistent filter kernel
  bool fused = false;
  int* d_ctafirst = nullptr;
  int* d_out_cu = nullptr;      // device int32[batch + 1]: first output row of every image, then the total
  int f_grid = 0, f_nstage = 0, f_max_piece = 0, f_vpl = 0;
  size_t f_smem = 0;
  // tensor-core correlate (bf16, hidden size a multiple of 64, FiCoCo-V)
  bool need_finalize = false;   // some image merges nothing: its per-token counts are zeroed by a kernel
  bool umma = false;
  bool um_f32 = false;          // fp32 tokens split into three bf16 terms (k_correlate_umma_f32)
  int um_b_bytes = 0;
  int um_stage_bytes = 0, um_a_bytes = 0, um_tmem_cols = 0, um_nstage = 0;
  size_t um_smem = 0;
  std::vector<ImgDesc> h_desc;
};

// ---- what the last step on a stream wrote ------------------------------------------------------
// The filter grid of a step may start under the tail of the merge grid of the step launched
// before it on the same stream.  That is only sound when the new step does not read what the
// older one is still writing, so the output spans of the last step are remembered per
// (device, stream), over all contexts of the process; a step whose inputs touch them, or whose
// stream has no record, is launched fully serialized.
struct Span {
  const char* lo = nullptr;
  const char* hi = nullptr;
};
inline Span span_of(const void* ptr, size_t bytes) {
  Span s;
  if (ptr != nullptr && bytes > 0) { s.lo = (const char*)ptr; s.hi = s.lo + bytes; }
  return s;
}
inline bool spans_overlap(const Span& a, const Span& b) {
  return a.lo != nullptr && b.lo != nullptr && a.lo < b.hi && b.lo < a.hi;
}
constexpr int N_TAILS = 16, N_SPANS = 4;
struct StreamTail {
  bool used = false;
  int device = 0;
  cudaStream_t st = nullptr;
  Span out[N_SPANS];
  unsigned long long stamp = 0;
};
std::mutex g_tail_mu;
StreamTail g_tail[N_TAILS];
unsigned long long g_tail_clock = 0;

bool inputs_clear_of_last_outputs(int device, cudaStream_t st, const Span* in, int n_in) {
  std::lock_guard<std::mutex> lk(g_tail_mu);
  for (int i = 0; i < N_TAILS; ++i) {
    const StreamTail& t = g_tail[i];
    if (!t.used || t.device != device || t.st != st) continue;
    for (int a = 0; a < n_in; ++a)
      for (int b = 0; b < N_SPANS; ++b)
        if (spans_overlap(in[a], t.out[b])) return false;
    return true;
  }
  return false;
}

void record_last_outputs(int device, cudaStream_t st, const Span* out, int n_out) {
  std::lock_guard<std::mutex> lk(g_tail_mu);
  int slot = -1;
  for (int i = 0; i < N_TAILS && slot < 0; ++i)
    if (g_tail[i].used && g_tail[i].device == device && g_tail[i].st == st) slot = i;
  if (slot < 0) {
    slot = 0;
    for (int i = 0; i < N_TAILS; ++i) {
      if (!g_tail[i].used) { slot = i; break; }
      if (g_tail[i].stamp < g_tail[slot].stamp) slot = i;
    }
  }
  StreamTail& t = g_tail[slot];
  t.used = true;
  t.device = device;
  t.st = st;
  t.stamp = ++g_tail_clock;
  for (int b = 0; b < N_SPANS; ++b) t.out[b] = b < n_out ? out[b] : Span();
}

}  // namespace

__global__ void k_launch_probe() {}

struct ficoco_ctx {
  int device = 0;
  long long max_tokens = 0;
  int max_dim = 0, max_batch = 0, max_text = 0;
  int last_cuda = 0;
  int launches = 0;
  unsigned long long clock = 0;

  char* d_base = nullptr;
  size_t d_bytes = 0;
  // scratch arrays
  float* rn = nullptr;
  float* partial = nullptr;
  float* msum = nullptr;     // [B][max_dim] column sums of the unfused filter
  float* s_raw = nullptr;
  float* s_pen = nullptr;
  int* S_idx = nullptr;
  int* T_idx = nullptr;
  float* part_val = nullptr;
  int* part_idx = nullptr;
  int* corr_cnt = nullptr;
  int* e_tgt = nullptr;     // compact per-image entry arrays, L slots per discarded token
  float* e_w = nullptr;
  float* e_c = nullptr;
  float* tau = nullptr;
  float* tmean = nullptr;
  unsigned* status = nullptr;
  int* tile_cnt = nullptr;  // per source tile: column splits of the correlate kernel that are done
  int merge_ctas_per_sm = 1;    // resident CTAs of the merge kernel per SM (register cap for 3)
  int merge_ctas_per_sm_dense = 1;   // the same with the register cap for 4 (plans without the fused filter)
  int* img_cnt = nullptr;   // two sets of 3 * max_batch per-image counters of the fused filter kernel
  unsigned long long epoch = 0;          // fused filter launches so far (its parity picks the counter set)
  int last_parity = 0;                   // counter set of the latest fused filter launch
  unsigned long long wait_ns = WAIT_NS_DEFAULT;   // bound of every device-side wait
  int dbg_extra_arrivals = 0;            // testing hook: arrivals the fused filter waits for that never come
  int num_sms = 0;
  bool coop_ok = false;
  bool coop_pdl_ok = false;  // a cooperative grid may also be a programmatic dependent
  char* plan_slots = nullptr;
  size_t slot_bytes = 0;
  size_t off_rows = 0, off_corr = 0, off_out = 0, off_ctaf = 0, off_ocu = 0;
  int cap_rows = 0, cap_corr = 0, cap_out = 0;
  long long cap_part = 0;

  char* h_stage = nullptr;  // pinned, slot_bytes
  Plan plans[N_PLANS];
  Plan* last_plan = nullptr;

  // optional per-kernel timing (events recorded between launches)
  bool prof_on = false;
  std::vector<cudaEvent_t> prof_ev;
  size_t prof_used = 0;
  std::vector<int> prof_name;            // per recorded event: index into prof_acc, -1 = end of call
  struct ProfAcc { const char* name; double ms; long long launches; };
  std::vector<ProfAcc> prof_acc;

  // grow-only intermediates of ficoco_v_reduce_schedule: tokens / positions ping-pong, kept indices per step
  char* sch_base = nullptr;
  size_t sch_bytes = 0;

  // grow-only staging for the host-buffer entry points
  char* hs_dev = nullptr;
  size_t hs_dev_bytes = 0;
  cudaStream_t hs_stream = nullptr;
  cudaStream_t hs_run = nullptr, hs_out = nullptr;   // kernels / downloads of the host entry points
  cudaEvent_t hs_ev[2 * HOST_MAX_GROUPS] = {};
};

#define CUDA_TRY(ctx, expr)                                  \
  do {                                                       \
    cudaError_t e__ = (expr);                                \
    if (e__ != cudaSuccess) {                                \
      (ctx)->last_cuda = (int)e__;                           \
      return FICOCO_ERR_CUDA;                                \
    }                                                        \
  } while (0)

namespace {

// Record an event in front of the kernel about to be launched (name) or at the end of a
// call (nullptr).  The time between two consecutive events is attributed to the first.
void prof_tick(ficoco_ctx* c, cudaStream_t st, const char* name) {
  if (!c->prof_on) return;
  if (c->prof_used == c->prof_ev.size()) {
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) return;
    c->prof_ev.push_back(e);
  }
  int idx = -1;
  if (name) {
    for (size_t i = 0; i < c->prof_acc.size(); ++i)
      if (c->prof_acc[i].name == name) idx = (int)i;
    if (idx < 0) { c->prof_acc.push_back({name, 0.0, 0}); idx = (int)c->prof_acc.size() - 1; }
  }
  cudaEventRecord(c->prof_ev[c->prof_used], st);
  if (c->prof_name.size() <= c->prof_used) c->prof_name.resize(c->prof_used + 1);
  c->prof_name[c->prof_used] = idx;
  ++c->prof_used;
}

void prof_flush(ficoco_ctx* c) {
  if (c->prof_used == 0) return;
  cudaDeviceSynchronize();
  for (size_t i = 0; i + 1 < c->prof_used; ++i) {
    const int idx = c->prof_name[i];
    if (idx < 0) continue;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->prof_ev[i], c->prof_ev[i + 1]) == cudaSuccess) {
      c->prof_acc[idx].ms += ms;
      c->prof_acc[idx].launches += 1;
    }
  }
  c->prof_used = 0;
}

}  // namespace

extern "C" int ficoco_profile(ficoco_ctx* c, int enable) {
  if (!c) return FICOCO_ERR_INVALID_ARG;
  cudaSetDevice(c->device);
  c->prof_used = 0;
  c->prof_acc.clear();
  c->prof_on = enable != 0;
  return FICOCO_OK;
}

extern "C" int ficoco_profile_read(ficoco_ctx* c, int index, char* name, int name_cap, double* total_ms,
                                   long long* launches) {
  if (!c || index < 0 || !name || name_cap < 2 || !total_ms || !launches) return FICOCO_ERR_INVALID_ARG;
  cudaSetDevice(c->device);
  prof_flush(c);
  if (index >= (int)c->prof_acc.size()) return FICOCO_ERR_INVALID_ARG;
  strncpy(name, c->prof_acc[index].name, name_cap - 1);
  name[name_cap - 1] = 0;
  *total_ms = c->prof_acc[index].ms;
  *launches = c->prof_acc[index].launches;
  return FICOCO_OK;
}

extern "C" const char* ficoco_strerror(int code) {
  switch (code) {
    case FICOCO_OK: return "ok";
    case FICOCO_ERR_INVALID_ARG: return "invalid argument";
    case FICOCO_ERR_UNSUPPORTED: return "unsupported dtype, size or quantile level";
    case FICOCO_ERR_KEEP_RANGE: return "keep count out of range";
    case FICOCO_ERR_WORKSPACE: return "problem exceeds the sizes given to ficoco_create";
    case FICOCO_ERR_CUDA: return "CUDA runtime error";
    case FICOCO_ERR_TIMEOUT: return "device-side wait timed out";
    case FICOCO_ERR_CAPTURE: return "a new plan cannot be uploaded during stream capture";
    case FICOCO_ERR_GRID: return "grid smaller than the number of alive patches";
    case FICOCO_ERR_STATIC_LIMIT:
      return "problem exceeds the fixed scratch of the allocation-free entry point "
             "(at most 64 images, dim 2048, 32768 patch tokens in total)";
    default: return "unknown error";
  }
}

extern "C" void ficoco_default_params(ficoco_params* p) {
  if (!p) return;
  p->lambda_ = 0.35;
  p->beta = 0.6;
  p->gamma = 0.6;
  p->eps = 0.998;
  p->penalty_coef = 2.0;
  p->window = 2;
  p->max_targets = -1;
  p->flags = FICOCO_HAS_CLS | FICOCO_LOCAL_PENALTY;
  p->reserved = 0;
}

#ifdef FICOCO_PHASE_TIMERS
// Phase timestamps of the most recent launch of every instrumented kernel (profiling builds only).
extern "C" int ficoco_phase_read(void* host_dst, size_t bytes) {
  if (cudaDeviceSynchronize() != cudaSuccess) return FICOCO_ERR_CUDA;
  const size_t n = sizeof(unsigned long long) * PH_KERNELS * PH_CTAS * PH_SLOTS;
  if (cudaMemcpyFromSymbol(host_dst, g_phase_ts, bytes < n ? bytes : n) != cudaSuccess) return FICOCO_ERR_CUDA;
  // start the next run from empty records
  static const unsigned long long zeros[PH_SLOTS * 64] = {0};
  for (size_t o = 0; o < n; o += sizeof(zeros))
    if (cudaMemcpyToSymbol(g_phase_ts, zeros, sizeof(zeros), o) != cudaSuccess) return FICOCO_ERR_CUDA;
  const unsigned zn[PH_KERNELS] = {0};
  return cudaMemcpyToSymbol(g_phase_n, zn, sizeof(zn)) == cudaSuccess ? FICOCO_OK : FICOCO_ERR_CUDA;
}
#endif

extern "C" int ficoco_last_cuda_error(const ficoco_ctx* ctx) { return ctx ? ctx->last_cuda : 0; }
extern "C" int ficoco_debug_waits(ficoco_ctx* c, long long wait_ns, int extra_arrivals) {
  if (!c || wait_ns < 0 || extra_arrivals < 0) return FICOCO_ERR_INVALID_ARG;
  c->wait_ns = wait_ns > 0 ? (unsigned long long)wait_ns : WAIT_NS_DEFAULT;
  c->dbg_extra_arrivals = extra_arrivals;
  return FICOCO_OK;
}
extern "C" int ficoco_last_launch_count(const ficoco_ctx* ctx) { return ctx ? ctx->launches : 0; }

extern "C" int ficoco_create(ficoco_ctx** out, int device, long long max_tokens, int max_dim,
                             int max_batch, int max_text) {
  if (!out || max_tokens <= 0 || max_dim <= 0 || max_batch <= 0 || max_text < 0 || device < 0)
    return FICOCO_ERR_INVALID_ARG;
  if (max_tokens > (1ll << 26) || max_dim > 16384) return FICOCO_ERR_UNSUPPORTED;
  ficoco_ctx* c = new (std::nothrow) ficoco_ctx();
  if (!c) return FICOCO_ERR_INVALID_ARG;
  c->device = device;
  c->max_tokens = max_tokens;
  c->max_dim = max_dim;
  c->max_batch = max_batch;
  c->max_text = max_text;
  cudaError_t e = cudaSetDevice(device);
  if (e != cudaSuccess) { delete c; return FICOCO_ERR_CUDA; }

  const size_t T = (size_t)max_tokens, B = (size_t)max_batch;
  {
    int v = 0;
    cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, device);
    c->num_sms = v > 0 ? v : 1;
    v = 0;
    cudaDeviceGetAttribute(&v, cudaDevAttrCooperativeLaunch, device);
    c->coop_ok = v != 0;
    // Does the runtime take a cooperative launch that also carries programmatic stream
    // serialization?  One empty grid answers it; a refusal only turns the overlap off.
    if (c->coop_ok) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(1);
      cfg.blockDim = dim3(32);
      cudaLaunchAttribute at[2];
      at[0].id = cudaLaunchAttributeCooperative;
      at[0].val.cooperative = 1;
      at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      at[1].val.programmaticStreamSerializationAllowed = 1;
      cfg.attrs = at;
      cfg.numAttrs = 2;
      const cudaError_t pe = cudaLaunchKernelEx(&cfg, k_launch_probe);
      const cudaError_t se = cudaDeviceSynchronize();
      c->coop_pdl_ok = pe == cudaSuccess && se == cudaSuccess;
      if (!c->coop_pdl_ok) cudaGetLastError();
    }
  }
  c->cap_rows = (int)(MAX_CHUNKS * B);
  if (c->cap_rows < c->num_sms + (int)B + 8) c->cap_rows = c->num_sms + (int)B + 8;
  c->cap_corr = (int)(2 * (T / CBM + B) + 2048);
  c->cap_out = (int)(T / OUT_ROWS_PER_CTA + B);
  c->cap_part = (long long)T * PART_PER_TOKEN;
  c->off_rows = align_up(B * sizeof(ImgDesc), 256);
  c->off_corr = c->off_rows + align_up((size_t)c->cap_rows * sizeof(WorkItem), 256);
  c->off_out = c->off_corr + align_up((size_t)c->cap_corr * sizeof(WorkItem), 256);
  c->off_ctaf = c->off_out + align_up((size_t)c->cap_out * sizeof(WorkItem), 256);
  c->off_ocu = c->off_ctaf + align_up((size_t)(c->num_sms + 2) * sizeof(int), 256);
  c->slot_bytes = c->off_ocu + align_up((B + 1) * sizeof(int), 256);

  size_t off = 0;
  auto carve = [&](size_t bytes) { size_t o = off; off += align_up(bytes, 256); return o; };
  const size_t o_rn = carve(T * 4), o_partial = carve((size_t)c->cap_rows * max_dim * 4);
  const size_t o_msum = carve((size_t)B * max_dim * 4);
  const size_t o_icnt = carve(6 * B * 4);
  const size_t o_tcnt = carve((size_t)c->cap_corr * 4);

  const size_t o_sraw = carve(T * 4), o_spen = carve(T * 4);
  const size_t o_S = carve(T * 4), o_T = carve(T * 4);
  const size_t o_pv = carve((size_t)c->cap_part * 4), o_pi = carve((size_t)c->cap_part * 4);
  const size_t o_cc = carve(T * 4), o_ct = carve(T * KCAP * 4), o_cw = carve(T * KCAP * 4);
  const size_t o_c = carve(T * KCAP * 4), o_tau = carve(T * 4);
  const size_t o_tm = carve(max_text > 0 ? T * (size_t)max_text * 4 : 256);
  const size_t o_st = carve(256);
  const size_t o_pl = carve(c->slot_bytes * N_PLANS);
  c->d_bytes = off;
  e = cudaMalloc((void**)&c->d_base, c->d_bytes);
  if (e != cudaSuccess) { c->last_cuda = (int)e; delete c; return FICOCO_ERR_CUDA; }
  e = cudaMemset(c->d_base, 0, c->d_bytes);
  if (e == cudaSuccess) e = cudaMallocHost((void**)&c->h_stage, c->slot_bytes);
  if (e != cudaSuccess) { cudaFree(c->d_base); delete c; return FICOCO_ERR_CUDA; }
  char* b = c->d_base;
  c->rn = (float*)(b + o_rn); c->partial = (float*)(b + o_partial); c->msum = (float*)(b + o_msum);
  c->s_raw = (float*)(b + o_sraw); c->s_pen = (float*)(b + o_spen);
  c->S_idx = (int*)(b + o_S); c->T_idx = (int*)(b + o_T);
  c->part_val = (float*)(b + o_pv); c->part_idx = (int*)(b + o_pi);
  c->corr_cnt = (int*)(b + o_cc); c->e_tgt = (int*)(b + o_ct); c->e_w = (float*)(b + o_cw);
  c->e_c = (float*)(b + o_c); c->tau = (float*)(b + o_tau);
  c->tmean = (float*)(b + o_tm); c->status = (unsigned*)(b + o_st);
  c->img_cnt = (int*)(b + o_icnt);
  c->tile_cnt = (int*)(b + o_tcnt);

  c->plan_slots = b + o_pl;

  // kernels that may need more than 48 KB of dynamic shared memory
  cudaFuncSetAttribute(k_select, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  {
    const int um_smem_max = 221 * 1024;
    cudaFuncSetAttribute(k_correlate_umma<2, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, um_smem_max);
    cudaFuncSetAttribute(k_correlate_umma<3, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, um_smem_max);
    cudaFuncSetAttribute(k_correlate_umma<4, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, um_smem_max);
    cudaFuncSetAttribute(k_correlate_umma<2, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, um_smem_max);
    cudaFuncSetAttribute(k_correlate_umma<3, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, um_smem_max);
    cudaFuncSetAttribute(k_correlate_umma<4, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, um_smem_max);
    cudaFuncSetAttribute(k_correlate_umma<2, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, um_smem_max);
    cudaFuncSetAttribute(k_correlate_umma<3, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, um_smem_max);
    cudaFuncSetAttribute(k_correlate_umma<4, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, um_smem_max);
    cudaFuncSetAttribute(k_correlate_umma<6, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, um_smem_max);
    cudaFuncSetAttribute(k_correlate_umma<6, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, um_smem_max);
    cudaFuncSetAttribute(k_correlate_umma<6, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, um_smem_max);
    cudaFuncSetAttribute(k_correlate_umma_f32<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, um_smem_max);
    cudaFuncSetAttribute(k_correlate_umma_f32<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, um_smem_max);
    cudaFuncSetAttribute(k_correlate_umma_f32<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, um_smem_max);
  }
  {
    const int fmax = 221 * 1024;
#define FICOCO_FUSED_ATTR(TT, V) cudaFuncSetAttribute(k_filter_fused<TT, V>, cudaFuncAttributeMaxDynamicSharedMemorySize, fmax)
    FICOCO_FUSED_ATTR(float, 1); FICOCO_FUSED_ATTR(float, 2); FICOCO_FUSED_ATTR(float, 4);
    FICOCO_FUSED_ATTR(float, 5); FICOCO_FUSED_ATTR(float, 8);
    FICOCO_FUSED_ATTR(__nv_bfloat16, 1); FICOCO_FUSED_ATTR(__nv_bfloat16, 2); FICOCO_FUSED_ATTR(__nv_bfloat16, 4);
    FICOCO_FUSED_ATTR(__nv_bfloat16, 5); FICOCO_FUSED_ATTR(__nv_bfloat16, 8);
#undef FICOCO_FUSED_ATTR
  }
  {
    int nb = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, k_merge_scan<__nv_bfloat16, 3>, 256, 0) == cudaSuccess && nb > 0)
      c->merge_ctas_per_sm = nb;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, k_merge_scan<__nv_bfloat16, 4>, 256, 0) == cudaSuccess && nb > 0)
      c->merge_ctas_per_sm_dense = nb;
  }
  cudaFuncSetAttribute(k_score<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
  cudaFuncSetAttribute(k_score<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
  if (cudaGetLastError() != cudaSuccess) { ficoco_destroy(c); return FICOCO_ERR_CUDA; }
  *out = c;
  return FICOCO_OK;
}

extern "C" int ficoco_destroy(ficoco_ctx* c) {
  if (!c) return FICOCO_ERR_INVALID_ARG;
  cudaSetDevice(c->device);
  cudaDeviceSynchronize();
  if (c->d_base) cudaFree(c->d_base);
  if (c->h_stage) cudaFreeHost(c->h_stage);
  if (c->hs_dev) cudaFree(c->hs_dev);
  if (c->sch_base) cudaFree(c->sch_base);
  if (c->hs_stream) cudaStreamDestroy(c->hs_stream);
  if (c->hs_run) cudaStreamDestroy(c->hs_run);
  if (c->hs_out) cudaStreamDestroy(c->hs_out);
  for (int i = 0; i < 2 * HOST_MAX_GROUPS; ++i)
    if (c->hs_ev[i]) cudaEventDestroy(c->hs_ev[i]);
  for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
  delete c;
  return FICOCO_OK;
}

// ---------------------------------------------------------------------------------------
// Plans
// ---------------------------------------------------------------------------------------
namespace {

int build_plan(ficoco_ctx* c, Plan* p, const PlanKey& key, int slot) {
  const int B = key.batch;
  const int cls = key.mode == 0 ? key.has_cls : 0;
  const int tail = key.mode == 1 ? key.n_text : 0;
  p->h_desc.assign(B, ImgDesc());
  std::vector<WorkItem> rows, corr, outw;
  long long row0 = 0, patch0 = 0, out0 = 0, src0 = 0, tgt0 = 0, ent0 = 0, part0 = 0, chunk0 = 0, rel0 = 0;
  p->max_np = p->max_tgt = p->max_src = p->max_rc = p->max_nwin_cells = p->max_list = 0;
  p->need_finalize = false;
  // tensor-core correlate: bf16 tokens, hidden size a multiple of 64.  FiCoCo-L adds its text term
  // in the epilogue from weights staged in shared memory, 2 KB per text token for the largest tile.
  p->umma = key.dtype == FICOCO_BF16 && key.dim % UKB == 0 &&
            (key.mode == 0 || (size_t)key.n_text * 2048 + 1024 + (size_t)UM * KCAP * 8 <= 220 * 1024);
  // fp32 tokens (FiCoCo-V): the same tiling with narrower column tiles, operands split into bf16 terms
  p->um_f32 = key.dtype == FICOCO_FP32 && key.dim % UKB == 0 && key.mode == 0;
  if (p->um_f32) p->umma = true;
  if (key.rel) p->umma = p->um_f32 = false;           // C is read from the supplied matrix, not contracted
  const int un_max = p->um_f32 ? UF_COLS : UN_MAX;    // accumulator columns per CTA
  int tile_rows_max = p->umma ? UM : CBM;             // source rows per correlate CTA (decided below)
  if (key.rel) {
    // a warp of the relation correlate takes one discarded token at a time and is bound by the
    // latency of its gathers: small tiles put more rows in flight (as far as the work table goes)
    auto strips = [&](int t) {
      long long n = 0;
      for (int b = 0; b < B; ++b) n += (key.ntok[b] - cls - tail - key.keep[b] + t - 1) / t;
      return n;
    };
    tile_rows_max = 16;
    while (tile_rows_max < CBM && strips(tile_rows_max) + 2 * c->num_sms > c->cap_corr) tile_rows_max *= 2;
  }
  const int col_granule = p->umma ? 16 : CBN;
  int um_a_rows = 8, um_cols = 16;

  // first pass: sizes
  for (int b = 0; b < B; ++b) {
    ImgDesc& d = p->h_desc[b];
    const int ntok = key.ntok[b];
    const int np = ntok - cls - tail;
    if (np < 1) return FICOCO_ERR_INVALID_ARG;
    if (np > MAX_IMG_TOKENS) return FICOCO_ERR_UNSUPPORTED;
    const int keep = key.keep[b];
    if (keep < 0 || keep > np) return FICOCO_ERR_KEEP_RANGE;
    d.n_cls = cls; d.np = np; d.n_tgt = keep; d.n_src = np - keep; d.n_tail = tail;
    d.n_extra = (key.conv && np - keep > 0) ? 1 : 0;
    d.gh = key.gh[b]; d.gw = key.gw[b];
    if (key.mode == 0) {
      if (d.gh < 1 || d.gw < 1) return FICOCO_ERR_INVALID_ARG;
      if ((long long)d.gh * d.gw < np) return FICOCO_ERR_GRID;
      if ((long long)d.gh * d.gw > 20000) return FICOCO_ERR_UNSUPPORTED;
    }
    int L = 0;
    float frac = 0.f;
    if (key.max_targets != 0 && d.n_src > 0 && d.n_tgt > 0) {
      if (key.max_targets > 0) {
        L = key.max_targets < d.n_tgt ? key.max_targets : d.n_tgt;
      } else {
        const double q = key.eps * (double)(d.n_tgt - 1);
        const double lo = floor(q);
        L = d.n_tgt - (int)lo;
        frac = (float)(q - lo);
      }
      if (L > KCAP) return FICOCO_ERR_UNSUPPORTED;
    }
    d.list_len = L;
    d.frac = frac;
    d.avg = key.avg;
    if (L > p->max_list) p->max_list = L;
  }
  // ---- fused filter kernel: piece size and feasibility -------------------------------------
  const int esz = key.dtype == FICOCO_BF16 ? 2 : 4;
  const int f_nvec = key.dim / (16 / esz);
  p->f_vpl = (f_nvec + 31) / 32;
  p->fused = c->coop_ok && p->f_vpl <= 8 && !key.rel;
  int f_rc = 0;
  if (p->fused) {
    long long total = 0;
    for (int b = 0; b < B; ++b) total += p->h_desc[b].np;
    auto count = [&](int rc) {
      long long n = 0;
      for (int b = 0; b < B; ++b) n += (p->h_desc[b].np + rc - 1) / rc;
      return n;
    };
    int rc0 = (int)((total + c->num_sms - 1) / c->num_sms);
    if (rc0 < 32) rc0 = 32;
    rc0 = (rc0 + 7) / 8 * 8;
    int rc1 = rc0;
    while (count(rc1) > c->num_sms && rc1 < 2 * rc0) rc1 += 8;
    // one piece per CTA if that costs at most 60 % more rows per CTA, else several pieces per CTA
    f_rc = (count(rc1) <= c->num_sms && rc1 * 10 <= rc0 * 16) ? rc1 : rc0;
  }

  // ---- correlate tiling ---------------------------------------------------------------------
  // A CTA gathers (tile rows + split columns) token rows per k-block from L2, which is what
  // bounds the stage.  Tiles of up to 128 rows let two CTAs share an SM; tiles of up to 256 rows
  // (two MMA sub-tiles sharing one column tile) gather fewer rows in total but have the SM to
  // themselves, and one CTA alone gathers more slowly than two.  Both are costed as
  // (waves x rows gathered per CTA x CTAs per SM); the wide tiles are taken when their cost is
  // at most 0.7 of the narrow ones' (measured: a tie at 0.75 on 32 x 577 tokens, 20 % faster at
  // 0.67 on 16 ragged images keeping 1/9 of their tokens).
  struct CorrChoice { int tile_rows, want_split; long long load; };
  auto cost_corr = [&](int rows_max, int ctas_per_sm) {
    CorrChoice ch{rows_max, 1, 0};
    long long strips = 0;
    for (int b = 0; b < B; ++b)
      if (p->h_desc[b].list_len > 0) strips += (p->h_desc[b].n_src + rows_max - 1) / rows_max;
    if (strips == 0) return ch;
    const long long slots = (long long)c->num_sms * ctas_per_sm;
    long long ws = slots / strips;
    if (ws < 1) ws = 1;
    // (fp32 tiles: the CTA that completes a tile merges nsplit * L entries per token, one thread each)
    const int split_max = p->um_f32 ? 8 : NSPLIT_MAX;
    if (ws > split_max) ws = split_max;
    ch.want_split = (int)ws;
    long long n_ctas = 0, max_rows = 0;
    for (int b = 0; b < B; ++b) {
      const ImgDesc& d = p->h_desc[b];
      if (d.list_len == 0) continue;
      int ns = ch.want_split;
      const int max_by_cols = (d.n_tgt + col_granule - 1) / col_granule;
      if (ns > max_by_cols) ns = max_by_cols;
      int cps = ((d.n_tgt + ns - 1) / ns + col_granule - 1) / col_granule * col_granule;
      if (p->umma && cps > un_max) cps = un_max;
      ns = (d.n_tgt + cps - 1) / cps;
      const int ntile = (d.n_src + rows_max - 1) / rows_max;
      const int trows = ((d.n_src + ntile - 1) / ntile + 7) / 8 * 8;
      n_ctas += (long long)ntile * ns;
      if (trows + cps > max_rows) max_rows = trows + cps;
    }
    const long long waves = (n_ctas + slots - 1) / slots;
    const long long per_sm = n_ctas < slots ? (n_ctas + c->num_sms - 1) / c->num_sms : ctas_per_sm;
    ch.load = waves * max_rows * per_sm;
    return ch;
  };
  int want_split = 1;
  {
    CorrChoice best = cost_corr(tile_rows_max, 2);
    if (p->umma && !p->um_f32) {
      const CorrChoice wide = cost_corr(UM * UM_SUB, 1);
      if (wide.load > 0 && wide.load * 10 <= best.load * 7) best = wide;
    }
    tile_rows_max = best.tile_rows;
    want_split = best.want_split;
  }

  // output rows per merge CTA: fewer than the usual 16 when that would leave most SMs with less
  // than two CTAs (few or very wide rows), as far as the work table goes
  int out_rows_cta = OUT_ROWS_PER_CTA;
  {
    auto n_out_ctas = [&](int r) {
      long long n = 0;
      for (int b = 0; b < B; ++b) n += (cls + key.keep[b] + p->h_desc[b].n_extra + tail + r - 1) / r;
      return n;
    };
    // An output row costs its own input row plus the discarded rows folded into it: with many
    // discarded tokens per preserved one (keep 1/9: nine rows read per row written) the CTAs are
    // kept smaller still, up to four per SM slot pair (measured: 16 ragged images keeping 1/9,
    // 133 -> 125 us per step with 4 instead of 8 rows per CTA; a 1/2 schedule loses 3 us that way).
    long long rows_out = 0, rows_src = 0;
    for (int b = 0; b < B; ++b) {
      rows_out += cls + key.keep[b] + p->h_desc[b].n_extra + tail;
      rows_src += key.ntok[b] - cls - tail - key.keep[b];
    }
    const long long reads_per_row = rows_out > 0 ? (rows_out + rows_src) / rows_out : 1;
    const long long want_ctas = (reads_per_row >= 4 ? 4LL : 2LL) * c->num_sms;
    while (out_rows_cta > 2 && n_out_ctas(out_rows_cta) < want_ctas &&
           n_out_ctas(out_rows_cta / 2) <= c->cap_out)
      out_rows_cta /= 2;
    // 24 rows per CTA when the grid then fits the SMs in one go and did not before.  Not ahead of the
    // persistent filter: the next step's filter grid starts only once every SM has drained, and longer
    // merge CTAs delay that by more than the saved wave gains (measured: +2.4 us per step with, -4.5 us
    // per step on a supplied relation map, whose score kernel is an ordinary grid).
    const long long slots = (long long)c->num_sms * (p->fused ? c->merge_ctas_per_sm : c->merge_ctas_per_sm_dense);
    if (out_rows_cta == OUT_ROWS_PER_CTA && n_out_ctas(16) > slots && n_out_ctas(24) <= slots && !p->fused) out_rows_cta = 24;
    p->out_rows_cta = out_rows_cta;
  }
  for (int b = 0; b < B; ++b) {
    ImgDesc& d = p->h_desc[b];
    d.row0 = (int)row0; d.patch0 = (int)patch0; d.out_row0 = (int)out0;
    d.src0 = (int)src0; d.tgt0 = (int)tgt0; d.ent0 = (int)ent0; d.part0 = (int)part0;
    d.attn0 = 0;  // set by the caller-specific code below
    d.rel0 = rel0;
    rel0 += (long long)d.np * d.np;
    // row chunks (fused filter: equal pieces of at most f_rc rows)
    int rc = (d.np + MAX_CHUNKS - 1) / MAX_CHUNKS;
    rc = (rc + 7) / 8 * 8;
    // unfused filter: chunks of about 256 KB of token rows (at most 64 rows; 32 rows of 4096 bf16), so
    // that wide rows still give every SM several CTAs
    int rc_floor = (int)(262144 / ((size_t)key.dim * (key.dtype == FICOCO_BF16 ? 2 : 4))) / 8 * 8;
    rc_floor = rc_floor < 8 ? 8 : (rc_floor > 64 ? 64 : rc_floor);
    if (rc < rc_floor) rc = rc_floor;
    if (p->fused) {
      const int npc = (d.np + f_rc - 1) / f_rc;
      rc = ((d.np + npc - 1) / npc + 7) / 8 * 8;
    }
    d.n_chunks = (d.np + rc - 1) / rc;
    d.chunk0 = (int)chunk0;
    for (int k = 0; k < d.n_chunks; ++k) {
      WorkItem w; w.img = b; w.r0 = k * rc; w.nrows = (d.np - w.r0 < rc) ? d.np - w.r0 : rc; w.aux = k;
      rows.push_back(w);
    }
    if (rc > p->max_rc) p->max_rc = rc;
    // correlate
    d.nsplit = 1; d.cols_per_split = d.n_tgt > 0 ? d.n_tgt : 1; d.corr_items = 0;
    if (d.list_len == 0 && d.n_src > 0) p->need_finalize = true;
    if (d.list_len > 0) {
      int ns = want_split;
      const int max_by_cols = (d.n_tgt + col_granule - 1) / col_granule;
      if (ns > max_by_cols) ns = max_by_cols;
      int cps = (d.n_tgt + ns - 1) / ns;
      cps = (cps + col_granule - 1) / col_granule * col_granule;
      if (p->umma && cps > un_max) cps = un_max;
      ns = (d.n_tgt + cps - 1) / cps;
      d.nsplit = ns; d.cols_per_split = cps;
      const size_t corr_before = corr.size();
      // source tiles of equal size (rounded to 8 rows)
      const int ntile = (d.n_src + tile_rows_max - 1) / tile_rows_max;
      int trows = (d.n_src + ntile - 1) / ntile;
      trows = (trows + 7) / 8 * 8;
      if (trows > um_a_rows) um_a_rows = trows;
      if (cps > um_cols) um_cols = cps;
      for (int s0 = 0; s0 < d.n_src; s0 += trows)
        for (int sp = 0; sp < ns; ++sp) {
          WorkItem w; w.img = b; w.r0 = s0; w.nrows = (d.n_src - s0 < trows) ? d.n_src - s0 : trows; w.aux = sp;
          corr.push_back(w);
        }
      d.corr_items = (int)(corr.size() - corr_before);
      part0 += (long long)d.n_src * ns * d.list_len;
      ent0 += (long long)d.n_src * d.list_len;
    }
    // output rows
    const int orows = d.n_cls + d.n_tgt + d.n_extra + d.n_tail;
    for (int r0 = 0; r0 < orows; r0 += out_rows_cta) {
      WorkItem w; w.img = b; w.r0 = r0; w.nrows = (orows - r0 < out_rows_cta) ? orows - r0 : out_rows_cta;
      w.aux = r0 / out_rows_cta;
      outw.push_back(w);
    }
    row0 += key.ntok[b]; patch0 += d.np; out0 += orows; src0 += d.n_src; tgt0 += d.n_tgt;
    chunk0 += d.n_chunks;
    if (d.np > p->max_np) p->max_np = d.np;
    if (d.n_tgt > p->max_tgt) p->max_tgt = d.n_tgt;
    if (d.n_src > p->max_src) p->max_src = d.n_src;
    if (key.mode == 0 && d.gh * d.gw > p->max_nwin_cells) p->max_nwin_cells = d.gh * d.gw;
  }
  if (row0 > c->max_tokens || B > c->max_batch || key.dim > c->max_dim || tail > c->max_text)
    return FICOCO_ERR_WORKSPACE;
  // ---- fused filter kernel: pieces -> CTAs, shared memory -----------------------------------
  std::vector<int> cta_first;
  if (p->fused) {
    long long total = 0;
    for (const WorkItem& w : rows) total += w.nrows;
    const long long target = (total + c->num_sms - 1) / c->num_sms;
    cta_first.push_back(0);
    long long acc_rows = 0;
    int items = 0;
    for (size_t i = 0; i < rows.size(); ++i) {
      if (items > 0 && (acc_rows + rows[i].nrows > target + 8 || items >= F_MAXWON) &&
          (int)cta_first.size() < c->num_sms) {
        cta_first.push_back((int)i);
        acc_rows = 0;
        items = 0;
      }
      acc_rows += rows[i].nrows;
      ++items;
      if (items > F_MAXWON) p->fused = false;
    }
    cta_first.push_back((int)rows.size());
    p->f_grid = (int)cta_first.size() - 1;
    p->f_max_piece = p->max_rc;
    const size_t stage = (size_t)FROWS * key.dim * esz;
    const size_t fixed = (size_t)FFOLD * key.dim * 4 + (size_t)p->f_max_piece * 4 + 256;
    const size_t budget = 216 * 1024;
    int ns = budget > fixed ? (int)((budget - fixed) / stage) : 0;
    if (ns > F_MAXSTAGE) ns = F_MAXSTAGE;
    size_t sel_need = 0;
    for (int b = 0; b < B; ++b) {
      const ImgDesc& d = p->h_desc[b];
      const size_t need = d.np <= SEL_SMALL_MAX ? select_small_bytes(d.np, key.mode == 0 ? d.gh * d.gw : 0)
                                                : select_work_bytes(d.np, key.mode == 0 ? d.gh * d.gw : 0);
      if (need > sel_need) sel_need = need;
    }
    if (ns < 2 || sel_need > (size_t)ns * stage) p->fused = false;
    p->f_nstage = ns;
    p->f_smem = (size_t)ns * stage + fixed;
  }
  if (!p->fused && rows.size() > (size_t)MAX_CHUNKS * B) return FICOCO_ERR_UNSUPPORTED;
  if ((int)rows.size() > c->cap_rows || (int)corr.size() > c->cap_corr || (int)outw.size() > c->cap_out ||
      part0 > c->cap_part)
    return FICOCO_ERR_WORKSPACE;
  p->tot_patch = (int)patch0; p->tot_src = (int)src0; p->tot_tgt = (int)tgt0; p->tot_out_rows = (int)out0;
  p->n_rows = (int)rows.size(); p->n_corr = (int)corr.size(); p->n_out = (int)outw.size();
  if (p->um_f32) {
    // two stages of three bf16 tiles per operand, 16 KB behind them for the 128-row reads of the last A tile
    p->um_a_bytes = um_a_rows * 128;
    p->um_b_bytes = (um_cols + 15) / 16 * 16 * 128;
    p->um_tmem_cols = 32;
    while (p->um_tmem_cols < 6 * (p->um_b_bytes / 128)) p->um_tmem_cols *= 2;   // six partial products per entry
    p->um_nstage = UF_STAGES;
    p->um_smem = (size_t)UF_STAGES * 3 * (p->um_a_bytes + p->um_b_bytes) + (size_t)UM * 128 + 2048;
    if (um_a_rows > UM || um_cols > UF_COLS || p->um_smem > 220 * 1024) return FICOCO_ERR_UNSUPPORTED;
  } else if (p->umma) {
    // shared-memory ring of the tensor-core correlate: prefer a size that lets two CTAs share an SM
    p->um_a_bytes = um_a_rows * 128;
    p->um_stage_bytes = p->um_a_bytes + um_cols * 128;
    const int n_sub = (um_a_rows + UM - 1) / UM;       // row sub-tiles (MMAs per k-step) of the largest tile
    p->um_tmem_cols = 32;
    while (p->um_tmem_cols < n_sub * um_cols) p->um_tmem_cols *= 2;
    if (p->um_tmem_cols > 512) return FICOCO_ERR_UNSUPPORTED;
    // every MMA reads 128 A rows: behind the last stage there must be room for the rows past the tile
    const size_t a_span = (size_t)n_sub * UM * 128;
    const size_t slack = 1024 + ((size_t)p->um_stage_bytes < a_span ? a_span - p->um_stage_bytes : 0);
    p->um_nstage = 0;
    // (a CTA that takes more than half of TMEM has the SM to itself anyway: use the deepest ring)
    for (int ns = 4; ns >= 2 && !p->um_nstage && p->um_tmem_cols <= 256; --ns)
      if ((size_t)ns * p->um_stage_bytes + slack <= 106 * 1024) p->um_nstage = ns;
    for (int ns = 6; ns >= 2 && !p->um_nstage; --ns)
      if (ns != 5 && (size_t)ns * p->um_stage_bytes + slack <= 220 * 1024) p->um_nstage = ns;
    if (!p->um_nstage) return FICOCO_ERR_UNSUPPORTED;
    p->um_smem = (size_t)p->um_nstage * p->um_stage_bytes + slack;
    // the epilogue halves hand their lists over through the ring; FiCoCo-L also stages the head-mean
    // text->vision weights of a tile's rows and columns there
    size_t epi = 1024 + (size_t)UM * KCAP * 8;
    if (key.mode == 1) epi += (size_t)key.n_text * ((size_t)n_sub * UM + (size_t)((um_cols + 15) / 16 * 16)) * 4;
    if (p->um_smem < epi) p->um_smem = epi;
    if (p->um_smem > 220 * 1024) return FICOCO_ERR_UNSUPPORTED;
  }

  char* slot_dev = c->plan_slots + (size_t)slot * c->slot_bytes;
  p->d_desc = (ImgDesc*)slot_dev;
  p->d_rows = (WorkItem*)(slot_dev + c->off_rows);
  p->d_corr = (WorkItem*)(slot_dev + c->off_corr);
  p->d_out = (WorkItem*)(slot_dev + c->off_out);
  p->d_ctafirst = (int*)(slot_dev + c->off_ctaf);
  p->d_out_cu = (int*)(slot_dev + c->off_ocu);
  {
    int* ocu = (int*)(c->h_stage + c->off_ocu);
    for (int b = 0; b < B; ++b) ocu[b] = p->h_desc[b].out_row0;
    ocu[B] = p->tot_out_rows;
  }
  p->key = key;
  if (p->fused) memcpy(c->h_stage + c->off_ctaf, cta_first.data(), cta_first.size() * sizeof(int));
  memcpy(c->h_stage + c->off_rows, rows.data(), rows.size() * sizeof(WorkItem));
  memcpy(c->h_stage + c->off_corr, corr.data(), corr.size() * sizeof(WorkItem));
  memcpy(c->h_stage + c->off_out, outw.data(), outw.size() * sizeof(WorkItem));
  return FICOCO_OK;
}

// Finds or builds the plan for `key`.  heads_or_text scales the attention block offsets:
// V: image b's block starts at H * patch0 floats; L: at M * b * N floats of the head-mean
// block t.
int get_plan(ficoco_ctx* c, const PlanKey& key, long long attn_rows, cudaStream_t stream, Plan** out) {
  ++c->clock;
  for (int i = 0; i < N_PLANS; ++i)
    if (c->plans[i].valid && c->plans[i].key == key) {
      // attention offsets depend on the head count, which is not part of the key
      bool same = true;
      for (int b = 0; b < key.batch && same; ++b)
        same = c->plans[i].h_desc[b].attn0 == attn_rows * c->plans[i].h_desc[b].patch0;
      if (same) {
        c->plans[i].stamp = c->clock;
        *out = &c->plans[i];
        return FICOCO_OK;
      }
      c->plans[i].valid = false;
    }
  cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
  CUDA_TRY(c, cudaStreamIsCapturing(stream, &cs));
  if (cs != cudaStreamCaptureStatusNone) return FICOCO_ERR_CAPTURE;
  int slot = 0;
  for (int i = 0; i < N_PLANS; ++i) {
    if (!c->plans[i].valid) { slot = i; break; }
    if (c->plans[i].stamp < c->plans[slot].stamp) slot = i;
  }
  // the staging buffer and the slot may still be read by work enqueued earlier
  CUDA_TRY(c, cudaStreamSynchronize(stream));
  Plan* p = &c->plans[slot];
  p->valid = false;
  int rc = build_plan(c, p, key, slot);
  if (rc != FICOCO_OK) return rc;
  for (int b = 0; b < key.batch; ++b) p->h_desc[b].attn0 = attn_rows * p->h_desc[b].patch0;
  memcpy(c->h_stage, p->h_desc.data(), key.batch * sizeof(ImgDesc));
  CUDA_TRY(c, cudaMemcpyAsync(c->plan_slots + (size_t)slot * c->slot_bytes, c->h_stage, c->slot_bytes,
                              cudaMemcpyHostToDevice, stream));
  CUDA_TRY(c, cudaStreamSynchronize(stream));
  p->valid = true;
  p->stamp = c->clock;
  *out = p;
  return FICOCO_OK;
}

// Launch with programmatic stream serialization: the grid may be staged while the kernel before
// it in the stream is still running; the kernel itself waits (grid_dep_wait) before it reads
// anything that kernel wrote.
template <class... KArgs, class... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t st,
                             Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

template <class T, int VPL>
cudaError_t launch_filter_fused(ficoco_ctx* c, const Plan* p, const T* tok, int D, const float* attn,
                                int attn_rows, float cA, const int* pos, int window, float coef, int penalty,
                                int* kept_idx, int* pos_out, float* scores_out, int overlap_prev,
                                cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p->f_grid);
  cfg.blockDim = dim3(F_THREADS);
  cfg.dynamicSmemBytes = p->f_smem;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeCooperative;
  at[0].val.cooperative = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = (c->coop_pdl_ok && overlap_prev) ? 2 : 1;   // 1: inputs independent of the step before; 2: fed by it
  c->last_parity = (int)(c->epoch++ & 1);
  return cudaLaunchKernelEx(&cfg, k_filter_fused<T, VPL>, tok, D, (const ImgDesc*)p->d_desc,
                            (const WorkItem*)p->d_rows, (const int*)p->d_ctafirst, c->rn, c->partial, attn,
                            attn_rows, cA, c->s_raw, c->img_cnt, p->key.batch, pos, window, coef, penalty,
                            c->s_pen, scores_out, c->S_idx, c->T_idx, kept_idx, pos_out, c->status,
                            p->f_nstage, p->f_max_piece, c->last_parity, 3 * c->max_batch, c->wait_ns,
                            c->dbg_extra_arrivals, (c->coop_pdl_ok && overlap_prev == 2) ? 1 : 0);
}

template <class T, int VPL>
void launch_colsum_fused(ficoco_ctx* c, const Plan* p, const T* tok, int D, cudaStream_t st) {
  constexpr int E = VecTraits<T>::E;
  k_colsum<T, VPL, true><<<dim3(p->n_rows, 1), 256, VPL * 32 * E * sizeof(float), st>>>(
      tok, D, p->d_desc, p->d_rows, c->rn, c->partial);
}

// Runs the whole reduce step for tokens of type T.  `attn` is the per-head CLS attention
// (V) or the head-mean text->vision block (L); `attn_rows` its number of rows per image.
template <class T>
int run_step(ficoco_ctx* c, const Plan* p, const T* tok, int D, const float* attn, int attn_rows,
             float cA, const int* pos, int window, float coef, int penalty, const float* tmean, int M,
             float gamma, T* out_tokens, int* kept_idx, int* pos_out, float* scores_out,
             cudaStream_t st, bool back_to_back, const float* rel = nullptr) {
  constexpr int E = VecTraits<T>::E;
  const int nvec = D / E;
  const int vpl = (nvec + 31) / 32;
  const size_t in_rows = (size_t)p->tot_patch + (size_t)p->key.batch * (p->key.has_cls + (p->key.mode == 1 ? p->key.n_text : 0));
  const Span in_spans[3] = {span_of(tok, in_rows * D * sizeof(T)),
                            span_of(attn, (size_t)attn_rows * p->tot_patch * sizeof(float)),
                            span_of(pos, (size_t)p->tot_patch * sizeof(int))};
  const Span out_spans[N_SPANS] = {span_of(out_tokens, (size_t)p->tot_out_rows * D * sizeof(T)),
                                   span_of(kept_idx, (size_t)p->tot_out_rows * sizeof(int)),
                                   span_of(pos_out, (size_t)p->tot_tgt * sizeof(int)),
                                   span_of(scores_out, (size_t)p->tot_patch * sizeof(float))};
  const Span rel_span = span_of(rel, rel ? (size_t)p->h_desc.back().rel0 * 4 + (size_t)p->h_desc.back().np * p->h_desc.back().np * 4 : 0);
  for (int o = 0; o < N_SPANS; ++o) {
    for (int i = 0; i < 3; ++i)
      if (spans_overlap(out_spans[o], in_spans[i])) return FICOCO_ERR_INVALID_ARG;
    if (spans_overlap(out_spans[o], rel_span)) return FICOCO_ERR_INVALID_ARG;
  }
  // the early start is taken only when the caller vouches for what sits in front of this step
  // 0: plain stream order; 1: the filter grid may read its inputs under the tail of the step before;
  // 2: it is fed by that step: launched early all the same, reads only once that step is complete
  const int overlap_prev = !back_to_back ? 0 : inputs_clear_of_last_outputs(c->device, st, in_spans, 3) ? 1 : 2;
  record_last_outputs(c->device, st, out_spans, N_SPANS);
  if (p->fused) {
    prof_tick(c, st, "filter_fused");
    cudaError_t fe;
#define FICOCO_FUSED_GO(V) fe = launch_filter_fused<T, V>(c, p, tok, D, attn, attn_rows, cA, pos, window, coef, \
                                                          penalty, kept_idx, pos_out, scores_out, overlap_prev, st)
    if (vpl <= 1) FICOCO_FUSED_GO(1);
    else if (vpl <= 2) FICOCO_FUSED_GO(2);
    else if (vpl <= 4) FICOCO_FUSED_GO(4);
    else if (vpl <= 5) FICOCO_FUSED_GO(5);
    else FICOCO_FUSED_GO(8);
#undef FICOCO_FUSED_GO
    if (fe != cudaSuccess) { c->last_cuda = (int)fe; return FICOCO_ERR_CUDA; }
    c->launches += 1;
  } else {
  if (rel) {
    prof_tick(c, st, "score_relation");
    k_score_rel<<<p->n_rows, 256, (size_t)p->max_rc * sizeof(float), st>>>(
        rel, p->d_desc, p->d_rows, attn, attn_rows, cA, p->key.rel == 2 ? 1 : 0, c->s_raw);
    c->launches += 1;
  } else {
  const bool wide = vpl > 8 && nvec <= 1024;   // rows of 257 .. 1024 16-byte vectors: CTA-wide rows
  prof_tick(c, st, (vpl <= 8 || wide) ? "colsum" : "rownorm");
  if (vpl <= 8) {
    if (vpl <= 1) launch_colsum_fused<T, 1>(c, p, tok, D, st);
    else if (vpl <= 2) launch_colsum_fused<T, 2>(c, p, tok, D, st);
    else if (vpl <= 4) launch_colsum_fused<T, 4>(c, p, tok, D, st);
    else if (vpl <= 5) launch_colsum_fused<T, 5>(c, p, tok, D, st);
    else launch_colsum_fused<T, 8>(c, p, tok, D, st);
    c->launches += 1;
  } else if (wide) {
    if (nvec <= 512) k_colsum_wide<T, 2, 8><<<p->n_rows, 256, 0, st>>>(tok, D, p->d_desc, p->d_rows, c->rn, c->partial);
    else k_colsum_wide<T, 4, 4><<<p->n_rows, 256, 0, st>>>(tok, D, p->d_desc, p->d_rows, c->rn, c->partial);
    c->launches += 1;
  } else {
    k_rownorm<T><<<p->n_rows, 256, 0, st>>>(tok, D, p->d_desc, p->d_rows, c->rn);
    prof_tick(c, st, "colsum");
    const int slabs = (nvec + 255) / 256;
    k_colsum<T, 8, false><<<dim3(p->n_rows, slabs), 256, 8 * 32 * E * sizeof(float), st>>>(
        tok, D, p->d_desc, p->d_rows, c->rn, c->partial);
    c->launches += 2;
  }
  prof_tick(c, st, "score");
  k_msum<<<dim3(p->key.batch, (D + 255) / 256), 256, 0, st>>>(D, p->d_desc, c->partial, c->msum);
  if (wide && nvec <= 512)
    k_score_wide<T, 2, 8><<<p->n_rows, 256, (size_t)9 * p->max_rc * sizeof(float), st>>>(
        tok, D, p->d_desc, p->d_rows, c->rn, c->msum, attn, attn_rows, cA, c->s_raw);
  else if (wide)
    k_score_wide<T, 4, 4><<<p->n_rows, 256, (size_t)9 * p->max_rc * sizeof(float), st>>>(
        tok, D, p->d_desc, p->d_rows, c->rn, c->msum, attn, attn_rows, cA, c->s_raw);
  else
    k_score<T><<<p->n_rows, 256, (size_t)(D + 9 * p->max_rc) * sizeof(float), st>>>(
        tok, D, p->d_desc, p->d_rows, c->rn, c->msum, attn, attn_rows, cA, c->s_raw);
  c->launches += 2;
  }
  size_t sel_smem = select_work_bytes(p->max_np, penalty ? p->max_nwin_cells : 0) + 16;
  if (p->max_np <= SEL_SMALL_MAX) {
    const size_t small = select_small_bytes(p->max_np, penalty ? p->max_nwin_cells : 0) + 16;
    if (small > sel_smem) sel_smem = small;
  }
  prof_tick(c, st, "select");
  // images of up to 1024 tokens: half the threads (two tokens each), cheaper barriers
  k_select<<<p->key.batch, p->max_np <= 1024 ? 512 : 1024, sel_smem, st>>>(p->d_desc, c->s_raw, pos, window, coef, penalty,
                                                  c->s_pen, scores_out, c->S_idx, c->T_idx, kept_idx,
                                                  pos_out, c->status);
  c->launches += 1;
  }
  if (p->n_corr > 0) {
    if (rel) {
      prof_tick(c, st, "correlate_relation");
      int rel_cols = 1;
      for (const ImgDesc& d : p->h_desc)
        if (d.list_len > 0 && d.cols_per_split > rel_cols) rel_cols = d.cols_per_split;
#define FICOCO_REL_GO(LC)                                                                              \
  k_correlate_rel<LC><<<p->n_corr, 256, (size_t)rel_cols * sizeof(int), st>>>(rel, p->d_desc, p->d_corr, c->S_idx, c->T_idx, c->part_val, \
                                                 c->part_idx, c->tile_cnt, c->corr_cnt, c->tau, c->e_tgt,    \
                                                 c->e_w, c->e_c, c->status)
      if (p->max_list <= 2) FICOCO_REL_GO(2);
      else if (p->max_list <= 4) FICOCO_REL_GO(4);
      else FICOCO_REL_GO(16);
#undef FICOCO_REL_GO
    } else if (p->um_f32 && sizeof(T) == 4) {
      prof_tick(c, st, "correlate_umma_f32");
      const float* tk = reinterpret_cast<const float*>(tok);
#define FICOCO_UF32_LAUNCH(LC)                                                                         \
  launch_dependent(k_correlate_umma_f32<LC>, p->n_corr, UTHREADS, p->um_smem, st, tk, D,               \
      (const ImgDesc*)p->d_desc, (const WorkItem*)p->d_corr, (const float*)c->rn,                       \
      (const int*)c->S_idx, (const int*)c->T_idx, c->part_val, c->part_idx, c->status,                 \
      p->um_a_bytes, p->um_b_bytes, p->um_tmem_cols, c->tile_cnt, c->corr_cnt, c->tau, c->e_tgt,        \
      c->e_w, c->e_c, c->wait_ns)
      if (p->max_list <= 2) FICOCO_UF32_LAUNCH(2);
      else if (p->max_list <= 4) FICOCO_UF32_LAUNCH(4);
      else FICOCO_UF32_LAUNCH(16);
#undef FICOCO_UF32_LAUNCH
    } else if (p->umma && sizeof(T) == 2) {
      prof_tick(c, st, "correlate_umma");
      const __nv_bfloat16* tk = reinterpret_cast<const __nv_bfloat16*>(tok);
#define FICOCO_UMMA_LAUNCH(NS, LC)                                                                     \
  launch_dependent(k_correlate_umma<NS, LC>, p->n_corr, UTHREADS, p->um_smem, st, tk, D,               \
      (const ImgDesc*)p->d_desc, (const WorkItem*)p->d_corr, (const float*)c->rn,                       \
      (const int*)c->S_idx, (const int*)c->T_idx, c->part_val, c->part_idx, c->status,                 \
      p->um_stage_bytes, p->um_a_bytes, p->um_tmem_cols, c->tile_cnt, c->corr_cnt, c->tau, c->e_tgt,    \
      c->e_w, c->e_c, tmean, M, p->max_np, gamma, c->wait_ns)
#define FICOCO_UMMA_STAGES(LC)                                                                         \
  do {                                                                                                 \
    if (p->um_nstage == 6) FICOCO_UMMA_LAUNCH(6, LC);                                                  \
    else if (p->um_nstage == 4) FICOCO_UMMA_LAUNCH(4, LC);                                             \
    else if (p->um_nstage == 3) FICOCO_UMMA_LAUNCH(3, LC);                                             \
    else FICOCO_UMMA_LAUNCH(2, LC);                                                                    \
  } while (0)
      if (p->max_list <= 2) FICOCO_UMMA_STAGES(2);
      else if (p->max_list <= 4) FICOCO_UMMA_STAGES(4);
      else FICOCO_UMMA_STAGES(16);
#undef FICOCO_UMMA_STAGES
#undef FICOCO_UMMA_LAUNCH
    } else {
      prof_tick(c, st, "correlate_simt");
      k_correlate_simt<T><<<p->n_corr, 256, 0, st>>>(tok, D, p->d_desc, p->d_corr, c->rn, c->S_idx,
                                                     c->T_idx, tmean, M, gamma, c->part_val, c->part_idx,
                                                     c->tile_cnt, c->corr_cnt, c->tau,
                                                     c->e_tgt, c->e_w, c->e_c, c->status);
    }
    c->launches += 1;
  }
  if (p->max_src > 0 && p->need_finalize) {
    prof_tick(c, st, "finalize");
    k_finalize_src<<<dim3(p->key.batch, (p->max_src + 255) / 256), 256, 0, st>>>(
        p->d_desc, c->part_val, c->part_idx, c->corr_cnt, c->tau, c->e_tgt, c->e_w, c->e_c);
    c->launches += 1;
  }
  prof_tick(c, st, "merge_compact");
  const int after_correlate = p->n_corr > 0 ? 1 : 0;   // else the grid before may be the filter itself
  if (p->fused)
    launch_dependent(k_merge_scan<T, 3>, p->n_out, 256, 0, st, tok, D, (const ImgDesc*)p->d_desc,
                     (const WorkItem*)p->d_out, (const int*)c->S_idx, (const int*)c->T_idx,
                     (const int*)c->e_tgt, (const float*)c->e_w, out_tokens, after_correlate,
                     c->status, c->img_cnt + (size_t)c->last_parity * 3 * c->max_batch, 3 * c->max_batch);
  else
    launch_dependent(k_merge_scan<T, 4>, p->n_out, 256, 0, st, tok, D, (const ImgDesc*)p->d_desc,
                     (const WorkItem*)p->d_out, (const int*)c->S_idx, (const int*)c->T_idx,
                     (const int*)c->e_tgt, (const float*)c->e_w, out_tokens, after_correlate,
                     c->status, (int*)nullptr, 0);
  c->launches += 1;
  if (p->key.conv) {
    prof_tick(c, st, "convergent_token");
    k_convergent_token<T><<<p->key.batch, 256, 0, st>>>(tok, D, p->d_desc, c->S_idx, out_tokens, c->status);
    c->launches += 1;
  }
  prof_tick(c, st, nullptr);
  if (c->prof_used > 60000) prof_flush(c);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { c->last_cuda = (int)e; return FICOCO_ERR_CUDA; }
  return FICOCO_OK;
}

int check_common(const ficoco_params* prm, int dtype, int batch, int dim, int heads, const void* tokens,
                 const void* out_tokens) {
  if (!prm || !tokens || !out_tokens) return FICOCO_ERR_INVALID_ARG;
  if (batch < 1 || dim < 1 || heads < 1) return FICOCO_ERR_INVALID_ARG;
  if (dtype != FICOCO_FP32 && dtype != FICOCO_BF16) return FICOCO_ERR_UNSUPPORTED;
  const int e = dtype == FICOCO_BF16 ? 8 : 4;
  if (dim % e != 0) return FICOCO_ERR_UNSUPPORTED;
  if (((uintptr_t)tokens & 15) || ((uintptr_t)out_tokens & 15)) return FICOCO_ERR_INVALID_ARG;
  if (!(prm->eps >= 0.0 && prm->eps <= 1.0) || prm->window < 1) return FICOCO_ERR_INVALID_ARG;
  return FICOCO_OK;
}

}  // namespace

namespace {
int v_reduce_impl(ficoco_ctx* c, const ficoco_v_args* a, const ficoco_params* prm, void* cuda_stream,
                  const float* rel, int rel_mode, bool plan_only = false) {
  if (!c || !a) return FICOCO_ERR_INVALID_ARG;
  // planning needs the shapes only: stand-ins for the data pointers pass the checks
  static const long long dummy[2] = {0, 0};
  int rc = check_common(prm, a->dtype, a->batch, a->dim, a->heads, plan_only ? (const void*)dummy : a->tokens,
                        plan_only ? (const void*)dummy : (const void*)a->out_tokens);
  if (rc) return rc;
  if (!a->grid_h || !a->grid_w || !a->keep) return FICOCO_ERR_INVALID_ARG;
  if (!plan_only && (!a->attn || !a->kept_idx)) return FICOCO_ERR_INVALID_ARG;
  if ((a->n_grid != 1 && a->n_grid != a->batch) || (a->n_keep != 1 && a->n_keep != a->batch))
    return FICOCO_ERR_INVALID_ARG;
  if (!a->seqlens && a->n_tokens < 1) return FICOCO_ERR_INVALID_ARG;
  if (a->batch > c->max_batch) return FICOCO_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  CUDA_TRY(c, cudaSetDevice(c->device));

  PlanKey key;
  key.mode = 0; key.dtype = a->dtype; key.batch = a->batch; key.dim = a->dim; key.n_text = 0;
  key.has_cls = (prm->flags & FICOCO_HAS_CLS) ? 1 : 0;
  key.max_targets = prm->max_targets < 0 ? -1 : prm->max_targets;
  key.avg = (prm->flags & FICOCO_AVERAGE_COMPRESSION) ? 1 : 0;
  key.conv = (prm->flags & FICOCO_CONVERGENT) ? 1 : 0;
  if (key.conv) key.max_targets = 0;               // nothing is merged into the preserved tokens
  key.rel = rel_mode;
  key.eps = prm->eps;
  key.ntok.resize(a->batch); key.keep.resize(a->batch); key.gh.resize(a->batch); key.gw.resize(a->batch);
  for (int b = 0; b < a->batch; ++b) {
    key.ntok[b] = a->seqlens ? a->seqlens[b] : a->n_tokens;
    key.keep[b] = a->keep[a->n_keep == 1 ? 0 : b];
    key.gh[b] = a->grid_h[a->n_grid == 1 ? 0 : b];
    key.gw[b] = a->grid_w[a->n_grid == 1 ? 0 : b];
  }
  Plan* p = nullptr;
  rc = get_plan(c, key, a->heads, st, &p);
  if (rc) return rc;
  if (plan_only) return FICOCO_OK;
  c->last_plan = p;
  c->launches = 0;
  if (a->out_cu_seqlens)       // prefix of the output rows per image, from the plan's device copy
    CUDA_TRY(c, cudaMemcpyAsync(a->out_cu_seqlens, p->d_out_cu, (size_t)(a->batch + 1) * sizeof(int),
                                cudaMemcpyDeviceToDevice, st));
  const int penalty = (prm->flags & FICOCO_LOCAL_PENALTY) ? 1 : 0;
  const bool b2b = (prm->flags & FICOCO_BACK_TO_BACK) != 0;
  if (a->dtype == FICOCO_BF16)
    return run_step<__nv_bfloat16>(c, p, (const __nv_bfloat16*)a->tokens, a->dim, a->attn, a->heads,
                                   (float)prm->lambda_, a->pos, prm->window, (float)prm->penalty_coef,
                                   penalty, nullptr, 0, 1.0f, (__nv_bfloat16*)a->out_tokens, a->kept_idx,
                                   a->pos_out, a->scores_out, st, b2b, rel);
  return run_step<float>(c, p, (const float*)a->tokens, a->dim, a->attn, a->heads, (float)prm->lambda_,
                         a->pos, prm->window, (float)prm->penalty_coef, penalty, nullptr, 0, 1.0f,
                         (float*)a->out_tokens, a->kept_idx, a->pos_out, a->scores_out, st, b2b, rel);
}
}  // namespace

extern "C" int ficoco_v_reduce(ficoco_ctx* c, const ficoco_v_args* a, const ficoco_params* prm,
                               void* cuda_stream) {
  return v_reduce_impl(c, a, prm, cuda_stream, nullptr, 0);
}

extern "C" int ficoco_v_plan(ficoco_ctx* c, const ficoco_v_args* a, const ficoco_params* prm, void* cuda_stream) {
  return v_reduce_impl(c, a, prm, cuda_stream, nullptr, 0, true);
}

extern "C" int ficoco_v_reduce_relation(ficoco_ctx* c, const ficoco_v_args* a, const float* relation,
                                        int by_column, const ficoco_params* prm, void* cuda_stream) {
  if (!relation || ((uintptr_t)relation & 3)) return FICOCO_ERR_INVALID_ARG;
  return v_reduce_impl(c, a, prm, cuda_stream, relation, by_column ? 2 : 1);
}

// kept_idx of a schedule: the chain of the steps' kept indices, last step first.
// kidx[s] : [B, rows_s] row indices into step s's input rows (rows_s = c + keep[s]).
struct ComposeArgs {
  const int* kidx[8];
  int rows[8];
  int n_steps;
};
__global__ void k_compose_kept(ComposeArgs a, int batch, int* __restrict__ out) {
  grid_dep_wait();        // launched under the tail of the last step's merge grid
  grid_dep_launch();
  const int rows_last = a.rows[a.n_steps - 1];
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= batch * rows_last) return;
  const int b = i / rows_last;
  int idx = a.kidx[a.n_steps - 1][i];
  for (int s = a.n_steps - 2; s >= 0 && idx >= 0; --s) idx = a.kidx[s][(size_t)b * a.rows[s] + idx];
  out[i] = idx;
}

extern "C" int ficoco_v_reduce_schedule(ficoco_ctx* c, const ficoco_v_args* first, int n_steps, const int* keep,
                                        const float* const* attn, const ficoco_params* prm, void* cuda_stream) {
  if (!c || !first || !keep || !attn || !prm) return FICOCO_ERR_INVALID_ARG;
  if (n_steps < 1 || n_steps > 8) return FICOCO_ERR_INVALID_ARG;
  if (first->seqlens || (prm->flags & FICOCO_CONVERGENT)) return FICOCO_ERR_UNSUPPORTED;
  if (first->batch < 1 || first->n_tokens < 1 || first->dim < 1 || !first->out_tokens || !first->kept_idx)
    return FICOCO_ERR_INVALID_ARG;
  if (first->dtype != FICOCO_FP32 && first->dtype != FICOCO_BF16) return FICOCO_ERR_UNSUPPORTED;
  const int cls = (prm->flags & FICOCO_HAS_CLS) ? 1 : 0;
  const size_t es = first->dtype == FICOCO_BF16 ? 2 : 4;
  const int B = first->batch;
  int np = first->n_tokens - cls;
  for (int s = 0; s < n_steps; ++s) {
    if (!attn[s]) return FICOCO_ERR_INVALID_ARG;
    if (keep[s] < 0 || keep[s] > np) return FICOCO_ERR_KEEP_RANGE;
    np = keep[s];
  }
  if (n_steps == 1) {
    ficoco_v_args a = *first;
    a.attn = attn[0]; a.keep = keep; a.n_keep = 1; a.scores_out = nullptr;
    return ficoco_v_reduce(c, &a, prm, cuda_stream);
  }
  cudaStream_t st = (cudaStream_t)cuda_stream;
  CUDA_TRY(c, cudaSetDevice(c->device));
  // intermediates: tokens and positions ping-pong (A holds the outputs of even steps, B of odd
  // ones), kept indices of every step
  const size_t rows0 = (size_t)B * (cls + keep[0]), rows1 = (size_t)B * (cls + keep[1 < n_steps ? 1 : 0]);
  const size_t tokA = align_up(rows0 * first->dim * es, 256), tokB = align_up(rows1 * first->dim * es, 256);
  const size_t posA = align_up((size_t)B * keep[0] * 4 + 4, 256), posB = align_up((size_t)B * keep[1] * 4 + 4, 256);
  size_t kid_bytes = 0;
  for (int s = 0; s < n_steps; ++s) kid_bytes += align_up((size_t)B * (cls + keep[s]) * 4, 256);
  const size_t need = tokA + tokB + posA + posB + kid_bytes;
  if (need > c->sch_bytes) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    CUDA_TRY(c, cudaStreamIsCapturing(st, &cs));
    if (cs != cudaStreamCaptureStatusNone) return FICOCO_ERR_CAPTURE;
    CUDA_TRY(c, cudaDeviceSynchronize());
    if (c->sch_base) { cudaFree(c->sch_base); c->sch_base = nullptr; c->sch_bytes = 0; }
    CUDA_TRY(c, cudaMalloc((void**)&c->sch_base, need));
    c->sch_bytes = need;
  }
  char* tok_buf[2] = {c->sch_base, c->sch_base + tokA};
  int* pos_buf[2] = {(int*)(c->sch_base + tokA + tokB), (int*)(c->sch_base + tokA + tokB + posA)};
  ComposeArgs ca = {};
  ca.n_steps = n_steps;
  char* kp = c->sch_base + tokA + tokB + posA + posB;
  for (int s = 0; s < n_steps; ++s) {
    ca.kidx[s] = (const int*)kp;
    ca.rows[s] = cls + keep[s];
    kp += align_up((size_t)B * (cls + keep[s]) * 4, 256);
  }
  ficoco_params ps = *prm;
  int total_launches = 0;
  np = first->n_tokens - cls;
  for (int s = 0; s < n_steps; ++s) {
    const bool last = s + 1 == n_steps;
    ficoco_v_args a = *first;
    a.seqlens = nullptr;
    a.n_tokens = cls + np;
    a.attn = attn[s];
    a.keep = &keep[s];
    a.n_keep = 1;
    a.scores_out = nullptr;
    if (s > 0) {
      a.tokens = tok_buf[(s - 1) & 1];
      a.pos = pos_buf[(s - 1) & 1];
      ps.flags |= FICOCO_BACK_TO_BACK;              // the kernel in front of this step is the library's own
    }
    a.out_tokens = last ? first->out_tokens : (void*)tok_buf[s & 1];
    a.pos_out = last ? first->pos_out : pos_buf[s & 1];
    a.kept_idx = (int*)ca.kidx[s];
    const int rc = ficoco_v_reduce(c, &a, &ps, cuda_stream);
    if (rc) return rc;
    total_launches += c->launches;
    np = keep[s];
  }
  const int n_out = B * (cls + keep[n_steps - 1]);
  launch_dependent(k_compose_kept, (n_out + 255) / 256, 256, 0, st, ca, B, first->kept_idx);
  c->launches = total_launches + 1;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { c->last_cuda = (int)e; return FICOCO_ERR_CUDA; }
  return FICOCO_OK;
}

extern "C" int ficoco_l_reduce(ficoco_ctx* c, const ficoco_l_args* a, const ficoco_params* prm,
                               void* cuda_stream) {
  if (!c || !a) return FICOCO_ERR_INVALID_ARG;
  int rc = check_common(prm, a->dtype, a->batch, a->dim, a->heads, a->tokens, a->out_tokens);
  if (rc) return rc;
  if (!a->attn_t2v || !a->keep || !a->kept_idx) return FICOCO_ERR_INVALID_ARG;
  if (a->n_vision < 1 || a->n_text < 1) return FICOCO_ERR_INVALID_ARG;
  if (a->n_keep != 1 && a->n_keep != a->batch) return FICOCO_ERR_INVALID_ARG;
  if (a->batch > c->max_batch || a->n_text > c->max_text) return FICOCO_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  CUDA_TRY(c, cudaSetDevice(c->device));

  PlanKey key;
  key.mode = 1; key.dtype = a->dtype; key.batch = a->batch; key.dim = a->dim; key.n_text = a->n_text;
  key.has_cls = 0;
  key.max_targets = prm->max_targets < 0 ? -1 : prm->max_targets;
  key.avg = (prm->flags & FICOCO_AVERAGE_COMPRESSION) ? 1 : 0;
  key.conv = (prm->flags & FICOCO_CONVERGENT) ? 1 : 0;
  if (key.conv) key.max_targets = 0;
  key.eps = prm->eps;
  key.ntok.assign(a->batch, a->n_vision + a->n_text);
  key.keep.resize(a->batch);
  key.gh.assign(a->batch, 1); key.gw.assign(a->batch, a->n_vision);
  for (int b = 0; b < a->batch; ++b) key.keep[b] = a->keep[a->n_keep == 1 ? 0 : b];
  Plan* p = nullptr;
  rc = get_plan(c, key, a->n_text, st, &p);
  if (rc) return rc;
  c->last_plan = p;
  c->launches = 0;
  prof_tick(c, st, "head_mean");
  k_head_mean<<<a->batch * a->n_text, 256, 0, st>>>(a->attn_t2v, a->heads, a->n_text, a->n_vision, c->tmean);
  c->launches += 1;
  if (a->dtype == FICOCO_BF16)
    return run_step<__nv_bfloat16>(c, p, (const __nv_bfloat16*)a->tokens, a->dim, c->tmean, a->n_text,
                                   (float)prm->beta, nullptr, 1, 1.0f, 0, c->tmean, a->n_text,
                                   (float)prm->gamma, (__nv_bfloat16*)a->out_tokens, a->kept_idx, nullptr,
                                   a->scores_out, st, false);
  return run_step<float>(c, p, (const float*)a->tokens, a->dim, c->tmean, a->n_text, (float)prm->beta,
                         nullptr, 1, 1.0f, 0, c->tmean, a->n_text, (float)prm->gamma,
                         (float*)a->out_tokens, a->kept_idx, nullptr, a->scores_out, st, false);
}

extern "C" int ficoco_status(ficoco_ctx* c, void* cuda_stream, int* device_status) {
  if (!c || !device_status) return FICOCO_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  CUDA_TRY(c, cudaSetDevice(c->device));
  unsigned v = 0;
  CUDA_TRY(c, cudaMemcpyAsync(&v, c->status, 4, cudaMemcpyDeviceToHost, st));
  CUDA_TRY(c, cudaMemsetAsync(c->status, 0, 4, st));
  CUDA_TRY(c, cudaStreamSynchronize(st));
  if (v & STATUS_TIMEOUT) {
    // a kernel gave up half-way: its per-image counters may be left non-zero
    CUDA_TRY(c, cudaMemsetAsync(c->img_cnt, 0, 6 * (size_t)c->max_batch * sizeof(int), st));
    CUDA_TRY(c, cudaMemsetAsync(c->tile_cnt, 0, (size_t)c->cap_corr * sizeof(int), st));
    CUDA_TRY(c, cudaStreamSynchronize(st));
  }
  *device_status = (int)v;
  return FICOCO_OK;
}

extern "C" int ficoco_inspect(ficoco_ctx* c, int what, void* host_dst, size_t bytes, size_t* bytes_avail) {
  if (!c || !c->last_plan) return FICOCO_ERR_INVALID_ARG;
  const Plan* p = c->last_plan;
  const void* src = nullptr;
  size_t n = 0;
  switch (what) {
    case FICOCO_INSPECT_RNORM: src = c->rn; n = (size_t)p->tot_patch * 4; break;
    case FICOCO_INSPECT_SCORE_RAW: src = c->s_raw; n = (size_t)p->tot_patch * 4; break;
    case FICOCO_INSPECT_SCORE: src = c->s_pen; n = (size_t)p->tot_patch * 4; break;
    case FICOCO_INSPECT_SRC_IDX: src = c->S_idx; n = (size_t)p->tot_src * 4; break;
    case FICOCO_INSPECT_TGT_IDX: src = c->T_idx; n = (size_t)p->tot_tgt * 4; break;
    case FICOCO_INSPECT_CORR_CNT: src = c->corr_cnt; n = (size_t)p->tot_src * 4; break;
    case FICOCO_INSPECT_CORR_TGT: src = c->e_tgt; n = (size_t)p->tot_src * KCAP * 4; break;
    case FICOCO_INSPECT_CORR_W: src = c->e_w; n = (size_t)p->tot_src * KCAP * 4; break;
    case FICOCO_INSPECT_CORR_C: src = c->e_c; n = (size_t)p->tot_src * KCAP * 4; break;
    case FICOCO_INSPECT_TAU: src = c->tau; n = (size_t)p->tot_src * 4; break;
    default: return FICOCO_ERR_INVALID_ARG;
  }
  if (bytes_avail) *bytes_avail = n;
  if (!host_dst || bytes == 0) return FICOCO_OK;
  CUDA_TRY(c, cudaSetDevice(c->device));
  CUDA_TRY(c, cudaDeviceSynchronize());
  if (what == FICOCO_INSPECT_CORR_TGT || what == FICOCO_INSPECT_CORR_W || what == FICOCO_INSPECT_CORR_C) {
    // the device keeps L slots per discarded token; widen to KCAP per token for the caller
    long long tot_ent = 0;
    for (const ImgDesc& d : p->h_desc) tot_ent += (long long)d.n_src * d.list_len;
    std::vector<int> compact((size_t)tot_ent + 1);
    if (tot_ent) CUDA_TRY(c, cudaMemcpy(compact.data(), src, (size_t)tot_ent * 4, cudaMemcpyDeviceToHost));
    std::vector<int> wide((size_t)p->tot_src * KCAP, what == FICOCO_INSPECT_CORR_TGT ? -1 : 0);
    for (const ImgDesc& d : p->h_desc)
      for (int s = 0; s < d.n_src; ++s)
        for (int k = 0; k < d.list_len; ++k)
          wide[(size_t)(d.src0 + s) * KCAP + k] = compact[(size_t)d.ent0 + (size_t)s * d.list_len + k];
    memcpy(host_dst, wide.data(), bytes < n ? bytes : n);
    return FICOCO_OK;
  }
  CUDA_TRY(c, cudaMemcpy(host_dst, src, bytes < n ? bytes : n, cudaMemcpyDeviceToHost));
  return FICOCO_OK;
}

// ---------------------------------------------------------------------------------------
// Host-buffer entry points
// ---------------------------------------------------------------------------------------
namespace {

int ensure_staging(ficoco_ctx* c, size_t dev_bytes) {
  if (!c->hs_stream) CUDA_TRY(c, cudaStreamCreateWithFlags(&c->hs_stream, cudaStreamNonBlocking));
  if (!c->hs_run) CUDA_TRY(c, cudaStreamCreateWithFlags(&c->hs_run, cudaStreamNonBlocking));
  if (!c->hs_out) CUDA_TRY(c, cudaStreamCreateWithFlags(&c->hs_out, cudaStreamNonBlocking));
  for (int i = 0; i < 2 * HOST_MAX_GROUPS; ++i)
    if (!c->hs_ev[i]) CUDA_TRY(c, cudaEventCreateWithFlags(&c->hs_ev[i], cudaEventDisableTiming));
  if (dev_bytes > c->hs_dev_bytes) {
    if (c->hs_dev) { CUDA_TRY(c, cudaDeviceSynchronize()); cudaFree(c->hs_dev); c->hs_dev = nullptr; }
    CUDA_TRY(c, cudaMalloc((void**)&c->hs_dev, dev_bytes));
    c->hs_dev_bytes = dev_bytes;
  }
  return FICOCO_OK;
}

struct Carver {
  char* base;
  size_t off = 0;
  explicit Carver(char* b) : base(b) {}
  template <class U> U* take(size_t bytes) { U* p = (U*)(base + off); off += align_up(bytes, 256); return p; }
};

}  // namespace

extern "C" int ficoco_v_reduce_host(ficoco_ctx* c, const ficoco_v_args* h, const ficoco_params* prm) {
  if (!c || !h || !prm) return FICOCO_ERR_INVALID_ARG;
  if (!h->tokens || !h->attn || !h->keep || !h->out_tokens || !h->kept_idx || h->batch < 1 || h->dim < 1 ||
      h->heads < 1 || (h->n_keep != 1 && h->n_keep != h->batch))
    return FICOCO_ERR_INVALID_ARG;
  if (h->dtype != FICOCO_FP32 && h->dtype != FICOCO_BF16) return FICOCO_ERR_UNSUPPORTED;
  const int cls = (prm->flags & FICOCO_HAS_CLS) ? 1 : 0;
  const size_t es = h->dtype == FICOCO_BF16 ? 2 : 4;
  const int B = h->batch;
  // prefix sums over images: input rows, patch tokens, output rows, preserved tokens
  std::vector<long long> p_rows(B + 1, 0), p_patch(B + 1, 0), p_orow(B + 1, 0), p_kept(B + 1, 0);
  for (int b = 0; b < B; ++b) {
    const int n = h->seqlens ? h->seqlens[b] : h->n_tokens;
    const int k = h->keep[h->n_keep == 1 ? 0 : b];
    if (n < cls + 1 || k < 0 || k > n - cls) return FICOCO_ERR_KEEP_RANGE;
    p_rows[b + 1] = p_rows[b] + n;
    p_patch[b + 1] = p_patch[b] + n - cls;
    p_orow[b + 1] = p_orow[b] + cls + k + (((prm->flags & FICOCO_CONVERGENT) && n - cls - k > 0) ? 1 : 0);
    p_kept[b + 1] = p_kept[b] + k;
  }
  const long long rows = p_rows[B], patches = p_patch[B], orows = p_orow[B], kept = p_kept[B];
  if (rows > c->max_tokens) return FICOCO_ERR_WORKSPACE;
  CUDA_TRY(c, cudaSetDevice(c->device));
  const size_t b_tok = (size_t)rows * h->dim * es, b_attn = (size_t)patches * h->heads * 4;
  const size_t b_pos = h->pos ? (size_t)patches * 4 : 0;
  const size_t b_out = (size_t)orows * h->dim * es, b_kidx = (size_t)orows * 4;
  const size_t b_posout = h->pos_out ? (size_t)kept * 4 : 0, b_sc = h->scores_out ? (size_t)patches * 4 : 0;
  const size_t total = align_up(b_tok, 256) + align_up(b_attn, 256) + align_up(b_pos, 256) +
                       align_up(b_out, 256) + align_up(b_kidx, 256) + align_up(b_posout, 256) +
                       align_up(b_sc, 256) + 256;
  int rc = ensure_staging(c, total);
  if (rc) return rc;
  Carver dv(c->hs_dev);
  char* d_tok = dv.take<char>(b_tok);
  char* d_attn = dv.take<char>(b_attn);
  char* d_pos = dv.take<char>(b_pos);
  char* d_out = dv.take<char>(b_out);
  char* d_kidx = dv.take<char>(b_kidx);
  char* d_po = dv.take<char>(b_posout);
  char* d_sc = dv.take<char>(b_sc);

  // Images are independent, so the batch goes through in groups of images: the upload of a
  // group, the kernels of the group before it and the download of the one before that run at
  // the same time on three streams (PCIe carries both directions at once).  Every group has its
  // own slice of the staging area, so nothing is reused while in flight.
  int n_groups = (int)(b_tok / HOST_GROUP_BYTES);
  if (n_groups > HOST_MAX_GROUPS) n_groups = HOST_MAX_GROUPS;
  if (n_groups > B) n_groups = B;
  if (n_groups < 1) n_groups = 1;
  cudaStream_t s_in = c->hs_stream, s_run = c->hs_run, s_out = c->hs_out;
  if (n_groups == 1) s_run = s_out = s_in;
  const size_t row_b = (size_t)h->dim * es;
  int launches = 0;
  rc = FICOCO_OK;
  auto group_begin = [&](int g) { return (int)((long long)B * g / n_groups); };
  // all uploads first: they depend on nothing, and queued ahead of everything else they never
  // sit behind a download that is itself waiting for kernels
  for (int g = 0; g < n_groups && rc == FICOCO_OK; ++g) {
    const int b0 = group_begin(g), b1 = group_begin(g + 1);
    const size_t o_tok = (size_t)p_rows[b0] * row_b, n_tok = (size_t)(p_rows[b1] - p_rows[b0]) * row_b;
    const size_t o_at = (size_t)p_patch[b0] * h->heads * 4, n_at = (size_t)(p_patch[b1] - p_patch[b0]) * h->heads * 4;
    const size_t o_ps = (size_t)p_patch[b0] * 4, n_ps = (size_t)(p_patch[b1] - p_patch[b0]) * 4;
    cudaError_t e = cudaMemcpyAsync(d_tok + o_tok, (const char*)h->tokens + o_tok, n_tok, cudaMemcpyHostToDevice, s_in);
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(d_attn + o_at, (const char*)h->attn + o_at, n_at, cudaMemcpyHostToDevice, s_in);
    if (e == cudaSuccess && h->pos)
      e = cudaMemcpyAsync(d_pos + o_ps, (const char*)h->pos + o_ps, n_ps, cudaMemcpyHostToDevice, s_in);
    if (e == cudaSuccess && n_groups > 1) e = cudaEventRecord(c->hs_ev[2 * g], s_in);
    if (e != cudaSuccess) { c->last_cuda = (int)e; rc = FICOCO_ERR_CUDA; }
  }
  for (int g = 0; g < n_groups && rc == FICOCO_OK; ++g) {
    const int b0 = group_begin(g), b1 = group_begin(g + 1);
    const size_t o_tok = (size_t)p_rows[b0] * row_b;
    const size_t o_at = (size_t)p_patch[b0] * h->heads * 4;
    const size_t o_ps = (size_t)p_patch[b0] * 4, n_ps = (size_t)(p_patch[b1] - p_patch[b0]) * 4;
    const size_t o_out = (size_t)p_orow[b0] * row_b, n_out = (size_t)(p_orow[b1] - p_orow[b0]) * row_b;
    const size_t o_ki = (size_t)p_orow[b0] * 4, n_ki = (size_t)(p_orow[b1] - p_orow[b0]) * 4;
    const size_t o_po = (size_t)p_kept[b0] * 4, n_po = (size_t)(p_kept[b1] - p_kept[b0]) * 4;
    cudaError_t e = cudaSuccess;
    if (n_groups > 1) e = cudaStreamWaitEvent(s_run, c->hs_ev[2 * g], 0);
    if (e != cudaSuccess) { c->last_cuda = (int)e; rc = FICOCO_ERR_CUDA; break; }
    ficoco_v_args a = *h;
    a.batch = b1 - b0;
    a.tokens = d_tok + o_tok;
    a.attn = (const float*)(d_attn + o_at);
    a.pos = h->pos ? (const int*)(d_pos + o_ps) : nullptr;
    if (h->seqlens) a.seqlens = h->seqlens + b0;
    if (h->n_keep != 1) { a.keep = h->keep + b0; a.n_keep = b1 - b0; }
    if (h->n_grid != 1) { a.grid_h = h->grid_h + b0; a.grid_w = h->grid_w + b0; a.n_grid = b1 - b0; }
    a.out_tokens = d_out + o_out;
    a.kept_idx = (int*)(d_kidx + o_ki);
    a.pos_out = h->pos_out ? (int*)(d_po + o_po) : nullptr;
    a.scores_out = h->scores_out ? (float*)(d_sc + o_ps) : nullptr;
    rc = ficoco_v_reduce(c, &a, prm, s_run);
    if (rc) break;
    launches += c->launches;
    if (n_groups > 1) {
      e = cudaEventRecord(c->hs_ev[2 * g + 1], s_run);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(s_out, c->hs_ev[2 * g + 1], 0);
    }
    if (e == cudaSuccess)
      e = cudaMemcpyAsync((char*)h->out_tokens + o_out, d_out + o_out, n_out, cudaMemcpyDeviceToHost, s_out);
    if (e == cudaSuccess)
      e = cudaMemcpyAsync((char*)h->kept_idx + o_ki, d_kidx + o_ki, n_ki, cudaMemcpyDeviceToHost, s_out);
    if (e == cudaSuccess && h->pos_out)
      e = cudaMemcpyAsync((char*)h->pos_out + o_po, d_po + o_po, n_po, cudaMemcpyDeviceToHost, s_out);
    if (e == cudaSuccess && h->scores_out)
      e = cudaMemcpyAsync((char*)h->scores_out + o_ps, d_sc + o_ps, n_ps, cudaMemcpyDeviceToHost, s_out);
    if (e != cudaSuccess) { c->last_cuda = (int)e; rc = FICOCO_ERR_CUDA; }
  }
  // drain all three streams whatever happened, so that no copy outlives the call
  const cudaError_t e1 = cudaStreamSynchronize(s_in), e2 = cudaStreamSynchronize(s_run),
                    e3 = cudaStreamSynchronize(s_out);
  if (rc) return rc;
  if (e1 != cudaSuccess || e2 != cudaSuccess || e3 != cudaSuccess) {
    c->last_cuda = (int)(e1 != cudaSuccess ? e1 : e2 != cudaSuccess ? e2 : e3);
    return FICOCO_ERR_CUDA;
  }
  c->launches = launches;
  return FICOCO_OK;
}

extern "C" int ficoco_l_reduce_host(ficoco_ctx* c, const ficoco_l_args* h, const ficoco_params* prm) {
  if (!c || !h || !prm) return FICOCO_ERR_INVALID_ARG;
  if (!h->tokens || !h->attn_t2v || !h->keep || !h->out_tokens || !h->kept_idx || h->batch < 1 ||
      h->dim < 1 || h->heads < 1 || h->n_vision < 1 || h->n_text < 1 ||
      (h->n_keep != 1 && h->n_keep != h->batch))
    return FICOCO_ERR_INVALID_ARG;
  if (h->dtype != FICOCO_FP32 && h->dtype != FICOCO_BF16) return FICOCO_ERR_UNSUPPORTED;
  const size_t es = h->dtype == FICOCO_BF16 ? 2 : 4;
  const int B = h->batch;
  std::vector<long long> p_orow(B + 1, 0);
  for (int b = 0; b < B; ++b) {
    const int k = h->keep[h->n_keep == 1 ? 0 : b];
    if (k < 0 || k > h->n_vision) return FICOCO_ERR_KEEP_RANGE;
    p_orow[b + 1] = p_orow[b] + k + h->n_text + (((prm->flags & FICOCO_CONVERGENT) && h->n_vision - k > 0) ? 1 : 0);
  }
  const long long orows = p_orow[B];
  const long long rows = (long long)B * (h->n_vision + h->n_text);
  if (rows > c->max_tokens) return FICOCO_ERR_WORKSPACE;
  CUDA_TRY(c, cudaSetDevice(c->device));
  const size_t seq_tok = (size_t)(h->n_vision + h->n_text) * h->dim * es;      // bytes per sequence
  const size_t seq_attn = (size_t)h->heads * h->n_text * h->n_vision * 4;
  const size_t seq_sc = (size_t)h->n_vision * 4;
  const size_t row_b = (size_t)h->dim * es;
  const size_t b_tok = seq_tok * B, b_attn = seq_attn * B;
  const size_t b_out = (size_t)orows * row_b, b_kidx = (size_t)orows * 4;
  const size_t b_sc = h->scores_out ? seq_sc * B : 0;
  const size_t total = align_up(b_tok, 256) + align_up(b_attn, 256) + align_up(b_out, 256) +
                       align_up(b_kidx, 256) + align_up(b_sc, 256) + 256;
  int rc = ensure_staging(c, total);
  if (rc) return rc;
  Carver dv(c->hs_dev);
  char* d_tok = dv.take<char>(b_tok);
  char* d_attn = dv.take<char>(b_attn);
  char* d_out = dv.take<char>(b_out);
  char* d_kidx = dv.take<char>(b_kidx);
  char* d_sc = dv.take<char>(b_sc);

  // Sequences are independent: groups of sequences go through upload, kernels and download on three
  // streams, as in ficoco_v_reduce_host (every group has its own slice of the staging area).
  int n_groups = (int)((b_tok + b_attn) / HOST_GROUP_BYTES);
  if (n_groups > HOST_MAX_GROUPS) n_groups = HOST_MAX_GROUPS;
  if (n_groups > B) n_groups = B;
  if (n_groups < 1) n_groups = 1;
  cudaStream_t s_in = c->hs_stream, s_run = c->hs_run, s_out = c->hs_out;
  if (n_groups == 1) s_run = s_out = s_in;
  int launches = 0;
  rc = FICOCO_OK;
  auto group_begin = [&](int g) { return (int)((long long)B * g / n_groups); };
  for (int g = 0; g < n_groups && rc == FICOCO_OK; ++g) {
    const int b0 = group_begin(g), b1 = group_begin(g + 1);
    cudaError_t e = cudaMemcpyAsync(d_tok + seq_tok * b0, (const char*)h->tokens + seq_tok * b0, seq_tok * (b1 - b0),
                                    cudaMemcpyHostToDevice, s_in);
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(d_attn + seq_attn * b0, (const char*)h->attn_t2v + seq_attn * b0, seq_attn * (b1 - b0),
                          cudaMemcpyHostToDevice, s_in);
    if (e == cudaSuccess && n_groups > 1) e = cudaEventRecord(c->hs_ev[2 * g], s_in);
    if (e != cudaSuccess) { c->last_cuda = (int)e; rc = FICOCO_ERR_CUDA; }
  }
  for (int g = 0; g < n_groups && rc == FICOCO_OK; ++g) {
    const int b0 = group_begin(g), b1 = group_begin(g + 1);
    const size_t o_out = (size_t)p_orow[b0] * row_b, n_out = (size_t)(p_orow[b1] - p_orow[b0]) * row_b;
    const size_t o_ki = (size_t)p_orow[b0] * 4, n_ki = (size_t)(p_orow[b1] - p_orow[b0]) * 4;
    cudaError_t e = cudaSuccess;
    if (n_groups > 1) e = cudaStreamWaitEvent(s_run, c->hs_ev[2 * g], 0);
    if (e != cudaSuccess) { c->last_cuda = (int)e; rc = FICOCO_ERR_CUDA; break; }
    ficoco_l_args a = *h;
    a.batch = b1 - b0;
    a.tokens = d_tok + seq_tok * b0;
    a.attn_t2v = (const float*)(d_attn + seq_attn * b0);
    if (h->n_keep != 1) { a.keep = h->keep + b0; a.n_keep = b1 - b0; }
    a.out_tokens = d_out + o_out;
    a.kept_idx = (int*)(d_kidx + o_ki);
    a.scores_out = h->scores_out ? (float*)(d_sc + seq_sc * b0) : nullptr;
    rc = ficoco_l_reduce(c, &a, prm, s_run);
    if (rc) break;
    launches += c->launches;
    if (n_groups > 1) {
      e = cudaEventRecord(c->hs_ev[2 * g + 1], s_run);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(s_out, c->hs_ev[2 * g + 1], 0);
    }
    if (e == cudaSuccess)
      e = cudaMemcpyAsync((char*)h->out_tokens + o_out, d_out + o_out, n_out, cudaMemcpyDeviceToHost, s_out);
    if (e == cudaSuccess)
      e = cudaMemcpyAsync((char*)h->kept_idx + o_ki, d_kidx + o_ki, n_ki, cudaMemcpyDeviceToHost, s_out);
    if (e == cudaSuccess && h->scores_out)
      e = cudaMemcpyAsync((char*)h->scores_out + seq_sc * b0, d_sc + seq_sc * b0, seq_sc * (b1 - b0),
                          cudaMemcpyDeviceToHost, s_out);
    if (e != cudaSuccess) { c->last_cuda = (int)e; rc = FICOCO_ERR_CUDA; }
  }
  // drain all three streams whatever happened, so that no copy outlives the call
  const cudaError_t e1 = cudaStreamSynchronize(s_in), e2 = cudaStreamSynchronize(s_run),
                    e3 = cudaStreamSynchronize(s_out);
  if (rc) return rc;
  if (e1 != cudaSuccess || e2 != cudaSuccess || e3 != cudaSuccess) {
    c->last_cuda = (int)(e1 != cudaSuccess ? e1 : e2 != cudaSuccess ? e2 : e3);
    return FICOCO_ERR_CUDA;
  }
  c->launches = launches;
  return FICOCO_OK;
}
