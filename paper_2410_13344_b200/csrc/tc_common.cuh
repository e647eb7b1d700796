// Device-side building blocks shared by the tensor-core kernels (GEMM and tree attention):
// mbarriers with bounded waits, TMA tile loads, tcgen05 MMA / tensor-memory access, shared-memory
// matrix descriptors, and thread-block-cluster rendezvous.  Device code only.
#pragma once

#include "cerb_internal.cuh"

namespace cerb {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---- mbarriers ----
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// What a bounded wait needs to know: the cycle budget, the CTA's abort flag and the status word.
struct WaitCtx {
  long long budget;          // SM clock cycles a wait may take (about 2 s by default: far beyond any legitimate wait)
  volatile int* aborted;     // shared-memory flag of the CTA: set by the first wait that ran out
  int32_t* status;           // device status words: [0] receives CERB_E_TIMEOUT, [1] the site of the first wait that ran
                             // out (a number chosen by the kernel, for diagnosis), [2] its block index (x + 1000 y),
                             // [3] `tag`
  int tag = 0;               // a number identifying the launch (for diagnosis)
};
__device__ __forceinline__ void wait_ran_out(const WaitCtx& w, int site) {
  *w.aborted = 1;
  if (atomicExch(w.status, CERB_E_TIMEOUT) == 0) {
    w.status[1] = site;
    w.status[2] = (int)(blockIdx.x + 1000u * blockIdx.y + 1000000u * blockIdx.z);
    w.status[3] = w.tag;
  }
}
// Once one wait in a CTA has run out (or an earlier kernel already reported a time-out), every later wait
// of that CTA gives up after this many cycles, so the CTA still runs to its end in bounded time.
constexpr long long kAbortedWaitCycles = 40000ll;

// mbarrier.try_wait may suspend the thread for a system-dependent time before it answers "not yet"; with a hint
// it comes back after about that many nanoseconds, which bounds how late a time-out can be noticed.
__device__ __forceinline__ bool mbar_try_wait_hint(uint32_t bar, uint32_t parity, uint32_t ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(ns)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after the budget.  A few plain polls first (almost every wait ends there); then the
// budget is measured with the SM-local cycle counter, which is cheap to read, between short runs of polls
// that each return after two microseconds at the latest.  Returns false when it gave up (the hot loops test this
// value, which costs nothing, rather than re-reading the CTA's abort flag after every wait).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const WaitCtx& w, int site = 0) {
  for (int i = 0; i < 8; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  const long long budget = *w.aborted ? kAbortedWaitCycles : w.budget;
  for (;;) {
    for (int i = 0; i < 16; ++i)
      if (mbar_try_wait_hint(bar, parity, 2000u)) return true;
    if (clock64() - t0 > budget) break;
  }
  wait_ran_out(w, site);
  return false;
}
// Wait used on the way out of a CTA that has given up: for copies and MMAs that are already in flight, so that
// none of them outlives the CTA's shared and tensor memory.  It keeps a budget of its own (what it waits for
// was issued and will complete; the limit only guards against the unforeseen) and reports nothing.
constexpr long long kDrainCycles = 4000000000ll;
__device__ __forceinline__ void mbar_wait_drain(uint32_t bar, uint32_t parity, long long cycles = kDrainCycles) {
  const long long t0 = clock64();
  for (;;) {
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return;
    if (clock64() - t0 > cycles) return;
  }
}
// Same bounded wait for a lane whose warp shares an issue port with busy warps: back off between polls.
__device__ __forceinline__ bool mbar_wait_polite(uint32_t bar, uint32_t parity, const WaitCtx& w, int site = 0) {
  for (int i = 0; i < 4; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  const long long budget = *w.aborted ? kAbortedWaitCycles : w.budget;
  for (;;) {
    for (int i = 0; i < 64; ++i) {
      if (mbar_try_wait(bar, parity)) return true;
      __nanosleep(40);
    }
    if (clock64() - t0 > budget) break;
  }
  wait_ran_out(w, site);
  return false;
}

// ---- TMA tile loads (no multicast anywhere) ----
__device__ __forceinline__ uint64_t l2_policy(bool evict_first) {
  uint64_t pol;
  if (evict_first) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  else asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"((uint64_t)map), "r"(x), "r"(y), "r"(bar), "l"(pol)
      : "memory");
}

// ---- shared-memory matrix descriptors (128-byte swizzle, what TMA writes) ----
// K-major operand tile: rows of 128 bytes (64 bf16 along K), 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t desc_k_sw128(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024u >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}
// MN-major operand tile: rows of 128 bytes hold 64 consecutive M (or N) elements of one k; `lbo` bytes between
// 64-element blocks along M/N, `sbo` bytes between groups of 8 k.
__device__ __forceinline__ uint64_t desc_mn_sw128(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}
// Instruction descriptor of kind::f16 with bf16 operands and fp32 accumulation.
__host__ __device__ constexpr uint32_t idesc_bf16(uint32_t M, uint32_t N, bool a_mn_major, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
         ((N >> 3) << 17) | ((M >> 4) << 24);
}

// ---- tcgen05 ----
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// The same for a pair of CTAs working as one (cta_group::2; issued by one thread of the pair's first CTA): the MMA
// is 256 rows tall, 128 from each CTA's shared memory at the same offsets; the B operand's rows are split likewise;
// each CTA's tensor memory receives its 128 rows of D.  The eight mask words (rows not to write) are zero.
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  const uint32_t z = 0u;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc), "r"(z)
      : "memory");
}
// Arrives, once the pair's MMAs issued so far have retired, on the mbarrier at this shared-memory offset in both
// CTAs of the pair (CTA mask 0b11).
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar), "h"(mask)
               : "memory");
}
// TMA tile load of a CTA of such a pair into its own shared memory; the bytes are counted on `bar`, a
// shared::cluster address that may lie in the other CTA of the pair.  No multicast: each CTA fetches its own tiles.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"((uint64_t)map), "r"(x), "r"(y), "r"(bar), "l"(pol)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void proxy_fence() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// 32 lanes x 16 consecutive columns (one 32-bit value per lane and column); no wait included.
__device__ __forceinline__ void tmem_ld16_nowait(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// ---- thread-block clusters ----
// Rendezvous of the CTAs of a cluster with bounded waits.  Every CTA owns mbarriers that expect one arrival per
// member; to meet, one thread of every CTA arrives on that barrier of every member (remote arrive, release at
// cluster scope) and whoever goes on to read the others' shared memory first waits on its own copy (acquire at
// cluster scope) with the same cycle budget as every other wait of these kernels.  The hardware cluster barrier
// is used once only, split in two: every thread arrives right after the barriers are initialised and waits just
// before the first remote arrive, so that no arrival can reach a barrier that is not initialised yet; that wait
// depends on nothing but the members having started.
__device__ __forceinline__ void cluster_start_arrive() { asm volatile("barrier.cluster.arrive.release;" ::: "memory"); }
__device__ __forceinline__ void cluster_start_wait() { asm volatile("barrier.cluster.wait.acquire;" ::: "memory"); }
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// `idx` numbers the calling threads of the CTA from 0: thread s signals member s (the arrivals leave in parallel).
__device__ __forceinline__ void cluster_meet(uint64_t* bar, int members, int idx, const WaitCtx& w, int site = 0) {
  const uint32_t local = (uint32_t)__cvta_generic_to_shared(bar);
  if (idx < members) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"((uint32_t)idx));
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
  }
  for (int i = 0; i < 1024; ++i)
    if (mbar_try_wait_cluster(local, 0)) return;
  const long long t0 = clock64();
  const long long budget = *w.aborted ? kAbortedWaitCycles : w.budget;
  for (;;) {
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait_cluster(local, 0)) return;
    if (clock64() - t0 > budget) break;
  }
  wait_ran_out(w, site);
}
// Last rendezvous before a CTA of a cluster leaves: the others may still be reading this CTA's shared memory or about to
// arrive on its barriers, so this wait keeps a budget of its own, far above that of the other waits (which shrink to
// microseconds once a wait has run out): a CTA that has given up still waits for its partners here.
__device__ __forceinline__ void cluster_meet_before_exit(uint64_t* bar, int members, int idx, const WaitCtx& w, int* flag, int site) {
  const long long budget = w.budget * 4 > 40000000ll ? w.budget * 4 : 40000000ll;
  const WaitCtx wx{budget, flag, w.status, w.tag};
  cluster_meet(bar, members, idx, wx, site);
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Arrive on an mbarrier anywhere in the cluster (shared::cluster address), release at cluster scope.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Bounded wait on an own mbarrier whose arrivals may come from another CTA of the cluster (acquire at cluster scope).
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, const WaitCtx& w, int site = 0) {
  for (int i = 0; i < 8; ++i)
    if (mbar_try_wait_cluster(bar, parity)) return true;
  const long long t0 = clock64();
  const long long budget = *w.aborted ? kAbortedWaitCycles : w.budget;
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait_cluster(bar, parity)) return true;
    if (clock64() - t0 > budget) break;
  }
  wait_ran_out(w, site);
  return false;
}
__device__ __forceinline__ uint32_t mapa_u32(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ float ld_cluster_f32(uint32_t a) {
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(a) : "memory");
  return v;
}
__device__ __forceinline__ float4 ld_cluster_v4(uint32_t a) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a) : "memory");
  return v;
}

}  // namespace cerb
