// mbarrier, cp.async and bulk-copy (TMA) primitives shared by the kernels.  Every wait is
// bounded by elapsed time on the GPU's global timer: it gives up after `limit_ns` nanoseconds
// (WAIT_NS_DEFAULT unless the kernel is given another limit) and the caller raises STATUS_TIMEOUT.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace ficoco {

constexpr unsigned STATUS_TIMEOUT = 4u;
constexpr unsigned STATUS_INDEX = 8u;     // an index list held a token index outside its image (replaced by 0)
constexpr unsigned long long WAIT_NS_DEFAULT = 20ull * 1000 * 1000;   // 20 ms: far beyond any wait of a healthy step

__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Optional phase timestamps (compile with -DFICOCO_PHASE_TIMERS): thread 0 of a CTA notes the SM
// clock at named points of a kernel, in a record of its own that it draws from a per-kernel counter
// (so that the records of several launches in a row can be told apart by their order); the record
// also keeps the CTA's index and the global timer at its first and last mark, so that the CTAs of
// all grids can be laid on one time line.  Compiled out by default.
#ifdef FICOCO_PHASE_TIMERS
constexpr int PH_KERNELS = 4, PH_CTAS = 4096, PH_SLOTS = 16;
__device__ unsigned long long g_phase_ts[PH_KERNELS][PH_CTAS][PH_SLOTS];
__device__ unsigned g_phase_n[PH_KERNELS];
#define FICOCO_PHASE_BEGIN(k)                                                          \
  unsigned ph_rec = 0;                                                                 \
  if (threadIdx.x == 0) {                                                              \
    const unsigned long long c0 = (unsigned long long)clock64(), g0 = ficoco::global_ns(); \
    ph_rec = atomicAdd(&ficoco::g_phase_n[k], 1u) % ficoco::PH_CTAS;                   \
    ficoco::g_phase_ts[k][ph_rec][0] = c0;                                             \
    ficoco::g_phase_ts[k][ph_rec][ficoco::PH_SLOTS - 1] = g0;                          \
    ficoco::g_phase_ts[k][ph_rec][ficoco::PH_SLOTS - 2] = blockIdx.x;                  \
  }
#define FICOCO_PHASE(k, p)                                                             \
  do {                                                                                 \
    if (threadIdx.x == 0) ficoco::g_phase_ts[k][ph_rec][p] = (unsigned long long)clock64(); \
  } while (0)
#else
#define FICOCO_PHASE_BEGIN(k) do { } while (0)
#define FICOCO_PHASE(k, p) do { } while (0)
#endif

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Bounded wait on a phase parity; false = gave up after limit_ns.  The clock is read only once
// a try has failed, so a wait that succeeds at once costs one instruction.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity,
                                          unsigned long long limit_ns = WAIT_NS_DEFAULT) {
  const uint32_t a = smem_u32(bar);
  unsigned long long t0 = 0;
  for (;;) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(a), "r"(parity) : "memory");
    if (ok) return true;
    const unsigned long long t = global_ns();
    if (t0 == 0) t0 = t;
    else if (t - t0 > limit_ns) return false;
  }
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
// Programmatic dependent launch.  grid_dep_wait() returns once every grid this one depends on has
// completed and its writes are visible (a no-op for a launch without the attribute);
// grid_dep_launch() lets the next grid in the stream start its blocks early, which then park in
// their own grid_dep_wait().
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Counter updates that publish (release) and, for the second one, also observe (acquire) at GPU
// scope in one round trip.  Called by one thread after a CTA barrier: the barrier orders the other
// threads' stores before it, and the release makes them visible with the count.
__device__ __forceinline__ void red_release_add(int* p, int v) {
  asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int atom_acq_rel_add(int* p, int v) {
  int old;
  asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
  return old;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Arrive on `bar` and announce `bytes` of bulk-copy traffic that will complete on it.
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
// Bulk copy global -> shared (both 16-byte aligned, size a multiple of 16) completing on `bar`.
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst_smem)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

}  // namespace ficoco
