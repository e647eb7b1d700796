// bf16 GEMM of the verification forward on the 5th-generation tensor cores (tcgen05 + TMEM).
//
//   out[slot][m][n] = partial sum over some k range of X[m][k] * W[n][k]        (fp32)
//
// A decoding step has few activation rows (tree nodes x batch) and large weight matrices, so the
// kernel is organised around streaming W exactly once at HBM speed ("swap-AB"): a 128-row tile of
// W is the MMA's A operand (M = 128), the activation rows are the B operand (N = rows), and
// D[128][rows] accumulates in tensor memory and is written out transposed.
//
// Up to 128 activation rows (gemm_bf16_kernel): a CTA takes 256 weight rows at a time (two MMA tiles
// that share one activation stage), which halves the activation re-reads through L2; weight tiles
// carry an evict-first L2 hint, activation tiles evict-last; the accumulator is double-buffered.
//
// More than 128 rows (batched trees, prefill chunks of a batch; gemm_bf16_pair_kernel further down):
// two CTAs of a cluster work as one, 256 rows per pass.  More than 256 rows are cut into row chunks of
// 256 that are not queued one after the other: the pairs are grouped, one pair per row chunk in a
// group, and the pairs of a group walk the same weight tiles side by side, so that HBM delivers each
// weight byte once and the other chunks find it in L2.
//
// The kernel is launched programmatically dependent on its predecessor: weights do not depend on
// the previous kernel, so the producer fills the whole stage ring with weight tiles before it
// waits for that kernel; only the activation loads and the output stores come after the wait.
//
// Schedule: persistent, one CTA per SM, stream-K.  The work is the list of (weight tile, 64-wide
// k block) units; every CTA takes an equal, contiguous share of it, so all SMs stream for the same
// time whatever the matrix shape (no partial last wave).  A share may cross tile boundaries: each
// run of units inside one tile is a "segment" that accumulates in TMEM and is written to its own
// fp32 partial slot; consumers add a tile's slots in index order (deterministic).  The CTA that
// owns a tile's last segment zero-fills the slots that tile does not use.
//
// Roles inside a CTA (224 threads): warp 0 = TMA producer (one lane) running ahead through the
// whole share, warp 1 = TMEM allocator and MMA issuer (one lane), warp 6 = second MMA issuer,
// warps 2-5 = epilogue (each owns the 32 TMEM lanes of its warp quarter).  The accumulator is double-buffered in TMEM so a segment's
// epilogue overlaps the next segment's MMAs.  Stages and accumulators are handed over with
// mbarriers; every wait is bounded and reports CERB_E_TIMEOUT through a status word.
#include <stdlib.h>
#include <string.h>

#include <mutex>

#include "tc_common.cuh"

namespace cerb {

namespace {

constexpr int BM = 128;          // weight rows per CTA (MMA M)
constexpr int BK = 64;           // k elements per stage: 64 bf16 = one 128-byte swizzle row
constexpr int MAX_STAGES = 8;
constexpr uint32_t A_STAGE_BYTES = BM * BK * 2;

// Loads 16 accumulator columns of this warp's 32 lanes and waits for them.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  tmem_ld16_nowait(taddr, r);
  tmem_ld_wait();
}

struct GemmParams {
  float* out;
  int32_t* status;
  int M, N, K;
  int n_mma;          // activation rows per pass (16..128, power of two; 256 for CTA pairs)
  int num_kb;         // ceil(K / 64)
  int tiles;          // ceil(N / 128)
  int per;            // work units per CTA
  int total;          // work units in the list: tiles * num_kb (pairs with lock == 1: row chunks * tiles * num_kb)
  int lock;           // CTA pairs only.  > 1: this many pairs (one per chunk of 256 rows) walk the same share of the (tile,
                      // k block) list side by side, so a weight tile is fetched from HBM once and found in L2 by the
                      // others; 1: row chunks are part of the list
  int nslots;         // partial slots per output element
  int stages;
  long long wait_cycles;   // budget of every bounded wait, SM clock cycles
  uint32_t idesc;
  uint32_t acc_cols;  // TMEM columns of one accumulator buffer
  int acc_bufs;       // accumulator buffers in TMEM: 2 (a segment's epilogue overlaps the next segment's MMAs); 1 for CTA
                      // pairs, whose two 256-column accumulators fill all 512 columns
  int tile_rows;      // weight rows between the starts of consecutive tiles
  int half_off;       // weight-row offset of a wide unit's second tile from its first
  int epi;            // fused epilogue (GemmEpilogue::kind)
  int F;              // SwiGLU: width of the gate (and of the up) block
  bf16* act;          // SwiGLU: output [M][F]
  unsigned int* tickets;
  RopeEpilogue re;    // RoPE + cache append (epi == 2)
  unsigned long long* clk;   // measurement only: clk[0] <- min over CTAs of the time the dependency wait returned,
                             // clk[kGemmClockSlots] <- max over CTAs of the time the CTA finished (globaltimer, ns); or null
};

// One run of k blocks inside one (row chunk, weight tile) job.
struct Segment {
  int job, kb0, nkb;
};
__device__ __forceinline__ bool next_segment(int& u, int u1, int num_kb, Segment& sg) {
  if (u >= u1) return false;
  sg.job = u / num_kb;
  sg.kb0 = u - sg.job * num_kb;
  int end = (sg.job + 1) * num_kb;
  if (end > u1) end = u1;
  sg.nkb = end - u;
  u = end;
  return true;
}

__global__ void __launch_bounds__(224, 1) gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmW,
                                                           const __grid_constant__ CUtensorMap tmX, const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t empty_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t acc_full[2];
  __shared__ __align__(8) uint64_t acc_empty[2];
  __shared__ __align__(8) uint64_t drain_bar[2];       // one per MMA issuer: "everything I issued has retired" (give-up path only)
  __shared__ uint32_t tmem_base_slot;
  __shared__ int aborted_s;
  __shared__ unsigned int ticket_s;
  volatile int* aborted = &aborted_s;
  const WaitCtx wc{p.wait_cycles, aborted, p.status, p.N + 100000 * (p.M > 999 ? 999 : p.M)};

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t b_bytes = (uint32_t)p.n_mma * BK * 2;
  const uint32_t a_bytes = 2 * A_STAGE_BYTES;        // two weight tiles of 128 rows per unit
  const uint32_t stage_bytes = a_bytes + b_bytes;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int share = (int)blockIdx.x;                   // which contiguous share of the unit list
  const int u0 = share * p.per;
  const int u1 = (u0 + p.per < p.total) ? u0 + p.per : p.total;

  if (threadIdx.x == 0) {
    aborted_s = 0;
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 2);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&acc_full[i]), 2);
      mbar_init(smem_u32(&acc_empty[i]), 4);
      mbar_init(smem_u32(&drain_bar[i]), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(2u * p.acc_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == 0) {
    if (lane == 0) {
      const int n_units = u1 - u0;
      const uint64_t pol_w = l2_policy(true), pol_x = l2_policy(false);
      // (tile, k block) of the unit being issued, advanced incrementally
      int w_job = u0 / p.num_kb, w_kb = u0 - w_job * p.num_kb;
      int x_kb = w_kb;
      auto load_w = [&](int i) {
        const int tile = w_job % p.tiles;
        const int s = i % p.stages;
        const uint32_t fb = smem_u32(&full_bar[s]);
        const uint32_t a_dst = smem_base + (uint32_t)s * stage_bytes;
        mbar_expect_tx(fb, stage_bytes);
        tma_load_2d_hint(a_dst, &tmW, w_kb * BK, tile * p.tile_rows, fb, pol_w);
        tma_load_2d_hint(a_dst + A_STAGE_BYTES, &tmW, w_kb * BK, tile * p.tile_rows + p.half_off, fb, pol_w);
        if (++w_kb == p.num_kb) { w_kb = 0; ++w_job; }
      };
      auto load_x = [&](int i) {
        const int s = i % p.stages;
        const uint32_t fb = smem_u32(&full_bar[s]);
        const uint32_t x_dst = smem_base + (uint32_t)s * stage_bytes + a_bytes;
        tma_load_2d_hint(x_dst, &tmX, x_kb * BK, 0, fb, pol_x);
        if (++x_kb == p.num_kb) x_kb = 0;
      };
      // Weights do not depend on the kernel before this one: fill the whole ring with weight tiles
      // while that kernel is still finishing, then wait for it and fetch the activations.
      const int pre = n_units < p.stages ? n_units : p.stages;
      for (int i = 0; i < pre; ++i) load_w(i);
      // the activation map's descriptor is fetched now, not by the first load after the wait
      asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tmX) : "memory");
      griddep_wait();
      // Dependents are released only now, after this CTA's own wait: when the kernel after this one starts,
      // the kernel before this one is complete, which is what lets kernels read, ahead of their own wait,
      // anything written at least two launches earlier.
      griddep_launch();
      if (p.clk) atomicMin(p.clk, globaltimer_ns());
      for (int i = 0; i < pre; ++i) load_x(i);
      int issued = pre;
      for (int i = pre; i < n_units; ++i) {
        const int s = i % p.stages;
        const uint32_t ph = (uint32_t)(i / p.stages) & 1u;
        if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, wc, 201)) break;     // this wait gave up (the consumers have stopped): issue nothing more
        load_w(i);
        load_x(i);
        issued = i + 1;
      }
      if (*aborted) {
        // give-up path: the copies already issued still land in this CTA's shared memory; see each of them in
        for (int i = issued > p.stages ? issued - p.stages : 0; i < issued; ++i)
          mbar_wait_drain(smem_u32(&full_bar[i % p.stages]), (uint32_t)(i / p.stages) & 1u);
      }
    }
  } else if (warp == 1 || warp == 6) {
    // MMA issuers.  Issuing one tcgen05.mma occupies its thread for ~100 cycles whatever the MMA's size, and
    // a 64-row step needs eight of them per 32 KB of weights, so each of the two weight tiles of a unit has
    // its own issuing thread (warp 1: first tile, warp 6: second tile).  A stage is free, and an accumulator
    // complete, once both have committed.
    const int hf = warp == 6 ? 1 : 0;
    if (lane == 0) {
      int u = u0;
      Segment sg;
      int i = 0, g = 0;
      while (next_segment(u, u1, p.num_kb, sg)) {
        const int buf = g & 1;
        const uint32_t use = (uint32_t)(g >> 1);      // how often this buffer was used before
        if (!mbar_wait(smem_u32(&acc_empty[buf]), (use & 1u) ^ 1u, wc, 202)) break;
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)buf * p.acc_cols;
        for (int k = 0; k < sg.nkb; ++k, ++i) {
          int s = i % p.stages;
          uint32_t ph = (uint32_t)(i / p.stages) & 1u;
          if (!mbar_wait(smem_u32(&full_bar[s]), ph, wc, 203)) break;
          tc_fence_after();
          uint32_t a_src = smem_base + (uint32_t)s * stage_bytes;
          uint64_t bdesc = desc_k_sw128(a_src + a_bytes);
          const uint64_t adesc = desc_k_sw128(a_src + (uint32_t)hf * A_STAGE_BYTES);
          const uint32_t d = tmem_d + (uint32_t)(hf * p.n_mma);
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk)    // advance 16 k elements = 32 bytes inside the swizzled row: +2 in 16-byte units
            umma_bf16(d, adesc + (uint64_t)(kk * 2), bdesc + (uint64_t)(kk * 2), p.idesc, (k > 0 || kk > 0) ? 1u : 0u);
          umma_commit(smem_u32(&empty_bar[s]));     // the stage is free once the MMAs have read it
        }
        if (*aborted) break;
        umma_commit(smem_u32(&acc_full[buf]));       // this thread's part of the segment's accumulator is complete
        ++g;
      }
      if (*aborted) {
        // give-up path: the MMAs already issued still read shared memory and write tensor memory; see them retire
        umma_commit(smem_u32(&drain_bar[hf]));
        mbar_wait_drain(smem_u32(&drain_bar[hf]), 0);
      }
    }
  } else {
    const int quarter = warp & 3;                    // TMEM lanes 32*quarter .. +31 belong to this warp
    griddep_wait();                                  // the kernel before this one may still be reading the partial buffer
    int u = u0;
    Segment sg;
    int g = 0;
    while (next_segment(u, u1, p.num_kb, sg)) {
      const int buf = g & 1;
      const int tile = sg.job;
      if (!mbar_wait(smem_u32(&acc_full[buf]), (uint32_t)(g >> 1) & 1u, wc, 204)) break;                         // the launch's output is undefined from here on
      tc_fence_after();
      // slot = how many CTAs before this one also work on this job
      const int job_u0 = sg.job * p.num_kb;
      const int first_cta = job_u0 / p.per;
      const int last_cta = (job_u0 + p.num_kb - 1) / p.per;
      const int slot = share - first_cta;
      const int m_base = 0;                            // (all rows in one pass: this kernel takes up to 128)
      const int m_cnt = p.M;
      const size_t ldo = (size_t)p.N;
      const int cnt = last_cta - first_cta + 1;        // CTAs that share this job = slots it uses
      if (p.epi == 1 && cnt == 1) {
        // SwiGLU, whole tile in this CTA: gate in the first accumulator half, up in the second
        const int f = tile * p.tile_rows + quarter * 32 + lane;
        bf16* a = p.act + (size_t)m_base * p.F + f;
        const uint32_t tg = tmem_base + (uint32_t)buf * p.acc_cols + ((uint32_t)(quarter * 32) << 16);
        for (int c0 = 0; c0 < m_cnt; c0 += 16) {
          uint32_t rg[16], ru[16];
          tmem_ld16(tg + (uint32_t)c0, rg);
          tmem_ld16(tg + (uint32_t)p.n_mma + (uint32_t)c0, ru);
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (c0 + j < m_cnt) {
              const float gv = __uint_as_float(rg[j]), uv = __uint_as_float(ru[j]);
              a[(size_t)(c0 + j) * p.F] = __float2bfloat16_rn(gv / (1.0f + expf(-gv)) * uv);
            }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&acc_empty[buf]));
        ++g;
        continue;
      }
      for (int hf = 0; hf < 2; ++hf) {
        const int n_out = tile * p.tile_rows + hf * p.half_off + quarter * 32 + lane;
        const bool n_ok = n_out < p.N;
        // consecutive lanes hold consecutive output columns: every store instruction writes 128 contiguous bytes
        float* o = p.out + ((size_t)slot * p.M + m_base) * ldo + (n_ok ? n_out : 0);
        const uint32_t taddr = tmem_base + (uint32_t)buf * p.acc_cols + (uint32_t)(hf * p.n_mma) + ((uint32_t)(quarter * 32) << 16);
        for (int c0 = 0; c0 < m_cnt; c0 += 16) {
          uint32_t r[16];
          tmem_ld16(taddr + (uint32_t)c0, r);
          if (n_ok) {
            if (c0 + 16 <= m_cnt) {
#pragma unroll
              for (int j = 0; j < 16; ++j) { *o = __uint_as_float(r[j]); o += ldo; }
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j)
                if (c0 + j < m_cnt) { *o = __uint_as_float(r[j]); o += ldo; }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&acc_empty[buf]));
      if (p.epi == 0 && share == last_cta) {
        for (int hf = 0; hf < 2; ++hf) {
          const int n_out = tile * p.tile_rows + hf * p.half_off + quarter * 32 + lane;
          if (n_out >= p.N) continue;
          for (int z = last_cta - first_cta + 1; z < p.nslots; ++z) {
            float* zo = p.out + ((size_t)z * p.M + m_base) * ldo + n_out;
            for (int m = 0; m < m_cnt; ++m) { *zo = 0.f; zo += ldo; }
          }
        }
      }
      if (p.epi == 1) {
        // The CTA that finishes this tile last (by ticket) adds the tile's slots in index order and applies SwiGLU.
        __threadfence();
        asm volatile("bar.sync 2, 128;" ::: "memory");
        if (warp == 2 && lane == 0) ticket_s = atomicAdd(&p.tickets[sg.job], 1u);
        asm volatile("bar.sync 2, 128;" ::: "memory");
        if (ticket_s == (unsigned)cnt - 1u) {
          __threadfence();
          const int f = tile * p.tile_rows + quarter * 32 + lane;
          const float* src = p.out + (size_t)m_base * ldo + f;
          bf16* a = p.act + (size_t)m_base * p.F + f;
          const size_t sstride = (size_t)p.M * ldo;
#pragma unroll 4
          for (int m = 0; m < m_cnt; ++m) {
            float gv = 0.f, uv = 0.f;
            for (int z = 0; z < cnt; ++z) {
              gv += __ldcg(src + z * sstride + (size_t)m * ldo);
              uv += __ldcg(src + z * sstride + (size_t)m * ldo + p.F);
            }
            a[(size_t)m * p.F] = __float2bfloat16_rn(gv / (1.0f + expf(-gv)) * uv);
          }
          if (warp == 2 && lane == 0) p.tickets[sg.job] = 0u;      // ready for the next launch
        }
      }
      if (p.epi == 2) {
        // The CTA that finishes this tile last (by ticket) adds the tile's slots in index order, rotates q and k and
        // stores q, k and v where the attention kernel expects them.  A thread owns one output column (= weight row)
        // of each half of the unit; the other element of its rotation pair is 64 columns away in the same head.
        __threadfence();
        asm volatile("bar.sync 2, 128;" ::: "memory");
        if (warp == 2 && lane == 0) ticket_s = atomicAdd(&p.tickets[sg.job], 1u);
        asm volatile("bar.sync 2, 128;" ::: "memory");
        if (ticket_s == (unsigned)cnt - 1u) {
          __threadfence();
          const RopeEpilogue& e = p.re;
          const int HD = e.H * 128;
          const size_t sstride = (size_t)p.M * ldo;
          // this thread's two output columns (one per half of the unit) and their rotation partners
          int col[2], which[2], hd[2];
          bool col_ok[2];
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            col[hf] = tile * p.tile_rows + hf * p.half_off + quarter * 32 + lane;
            col_ok[hf] = col[hf] < 3 * HD;
            which[hf] = col_ok[hf] ? col[hf] / HD : 2;
            hd[hf] = col[hf] - which[hf] * HD;
          }
          for (int m = 0; m < m_cnt; ++m) {
            int b, v;
            locate_row(m, e.row_off, e.B, e.n, b, v);
            const int na = e.n_active[b], L = e.len[b], dep = e.depth[v];
            // every slot value this thread needs, requested before any of them is used (one round trip to L2)
            constexpr int ZMAX = 6;
            float own[2][ZMAX], oth[2][ZMAX];
            const float* src = p.out + (size_t)m * ldo;
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
              const int i = hd[hf] & 127;
              const int partner = i < 64 ? col[hf] + 64 : col[hf] - 64;
#pragma unroll
              for (int z = 0; z < ZMAX; ++z) {
                const bool take = col_ok[hf] && z < cnt;
                own[hf][z] = take ? __ldcg(src + z * sstride + col[hf]) : 0.f;
                oth[hf][z] = take && which[hf] < 2 ? __ldcg(src + z * sstride + partner) : 0.f;
              }
            }
            const int pos = L + dep, slot = L + v;
            const bool ok = v < na && pos < e.max_pos && slot < e.max_pos;
            const int page = ok ? e.page_table[(size_t)b * e.max_pages + slot / CERB_PAGE] : 0;
            float2 cs[2];
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) cs[hf] = ok && which[hf] < 2 ? e.rope[(size_t)pos * 64 + (hd[hf] & 63)] : make_float2(1.f, 0.f);
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
              if (!col_ok[hf] || !ok) continue;
              const int i = hd[hf] & 127, h = hd[hf] >> 7;
              float a = 0.f, o2 = 0.f;
#pragma unroll
              for (int z = 0; z < ZMAX; ++z) { a += own[hf][z]; o2 += oth[hf][z]; }        // slots in index order
              for (int z = ZMAX; z < cnt; ++z) {                                          // (more slots than usual)
                const int partner = i < 64 ? col[hf] + 64 : col[hf] - 64;
                a += __ldcg(src + z * sstride + col[hf]);
                if (which[hf] < 2) o2 += __ldcg(src + z * sstride + partner);
              }
              float val = a;
              if (which[hf] < 2) val = i < 64 ? a * cs[hf].x - o2 * cs[hf].y : a * cs[hf].x + o2 * cs[hf].y;
              if (which[hf] == 0) {
                reinterpret_cast<bf16*>(e.q)[(size_t)m * HD + hd[hf]] = __float2bfloat16_rn(val);
              } else {
                bf16* pool = reinterpret_cast<bf16*>(which[hf] == 1 ? e.kpool : e.vpool);
                pool[(((size_t)page * e.H + h) * CERB_PAGE + (size_t)(slot % CERB_PAGE)) * 128 + i] = __float2bfloat16_rn(val);
              }
            }
          }
          if (warp == 2 && lane == 0) p.tickets[sg.job] = 0u;      // ready for the next launch
        }
      }
      ++g;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (p.clk && threadIdx.x == 0) atomicMax(p.clk + kGemmClockSlots, globaltimer_ns());
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2u * p.acc_cols) : "memory");
  }
}


// ---------------------------------------------------------------------------------------------------------------
// More than 128 activation rows: two CTAs of a cluster work as one (tcgen05 cta_group::2).
//
// With 256 activation rows per pass a single CTA's stage is half activations (32 KB of weights + 32 KB of
// activations, three stages), so too few weight bytes are in flight per SM to cover HBM's latency, and the two
// 256-column accumulators fill tensor memory.  A pair of CTAs shares the activation tile instead: one MMA is
// 256 weight rows tall, 128 from each CTA's shared memory, and its 256 activation rows come half from each CTA.
// A unit of the work list is then 512 weight rows x 64 k (two such MMA rows, hf = 0 / 1); per CTA a stage holds
// 2 x 16 KB of weights + 16 KB of activations (four stages: 128 KB of weights in flight instead of 96), and each CTA's
// tensor memory holds its 128 rows of both accumulators.  Every CTA fetches its own tiles (no multicast); the
// byte counts of both CTAs' copies go to the first CTA's "landed" barrier, whose two MMA-issuing threads drive the
// pair; their commits arrive on the "free" and "accumulator complete" barriers of both CTAs at once.  The work
// list, the shares, the segments and the partial slots are those of the kernel above, with pairs in the place of
// CTAs.
// ---------------------------------------------------------------------------------------------------------------
constexpr int PAIR_STAGES = 4;
constexpr int PAIR_TILE = 4 * BM;                       // weight rows of a pair's unit
constexpr uint32_t PAIR_STAGE_BYTES = 3 * A_STAGE_BYTES;  // per CTA: weights hf 0, weights hf 1, its half of the activations
constexpr int PAIR_ACT = 2 * BM;                        // activation rows per pass (the MMA's N)

__global__ void __launch_bounds__(224, 1) gemm_bf16_pair_kernel(const __grid_constant__ CUtensorMap tmW,
                                                                const __grid_constant__ CUtensorMap tmX, const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[PAIR_STAGES];     // used in the pair's first CTA only
  __shared__ __align__(8) uint64_t empty_bar[PAIR_STAGES];
  __shared__ __align__(8) uint64_t acc_full, acc_empty;       // acc_empty: first CTA only, 4 epilogue warps of each CTA arrive
  __shared__ __align__(8) uint64_t drain_bar[2];
  __shared__ __align__(8) uint64_t meet_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int aborted_s, meet_flag_s;
  volatile int* aborted = &aborted_s;
  const WaitCtx wc{p.wait_cycles, aborted, p.status, p.N + 100000 * (p.M > 999 ? 999 : p.M)};

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool first = rank == 0;
  const int pair = (int)blockIdx.x >> 1;
  const int share = pair / p.lock;
  const int my_chunk = pair % p.lock;
  const int u0 = share * p.per;
  const int u1 = (u0 + p.per < p.total) ? u0 + p.per : p.total;

  if (threadIdx.x == 0) {
    aborted_s = 0;
    meet_flag_s = 0;
    for (int s = 0; s < PAIR_STAGES; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 2);
    }
    mbar_init(smem_u32(&acc_full), 2);
    mbar_init(smem_u32(&acc_empty), 8);
    mbar_init(smem_u32(&drain_bar[0]), 1);
    mbar_init(smem_u32(&drain_bar[1]), 1);
    mbar_init(smem_u32(&meet_bar), 2);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    // each CTA allocates all 512 columns of its own tensor memory (so both get the same base)
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  cluster_start_arrive();       // the other CTA's barriers exist before anything is signalled across
  cluster_start_wait();
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == 0) {
    if (lane == 0) {
      const int n_units = u1 - u0;
      const uint64_t pol_w = l2_policy(true), pol_x = l2_policy(false);
      int w_job = u0 / p.num_kb, w_kb = u0 - w_job * p.num_kb;
      int x_job = w_job, x_kb = w_kb;
      auto load_w = [&](int i) {
        const int tile = w_job % p.tiles;
        const int s = i % PAIR_STAGES;
        if (first) mbar_expect_tx(smem_u32(&full_bar[s]), 2 * PAIR_STAGE_BYTES);      // both CTAs' copies of this stage
        const uint32_t fb = mapa_u32(smem_u32(&full_bar[s]), 0);
        const uint32_t dst = smem_base + (uint32_t)s * PAIR_STAGE_BYTES;
        const int row = tile * PAIR_TILE + (int)rank * BM;
        tma_load_2d_pair(dst, &tmW, w_kb * BK, row, fb, pol_w);
        tma_load_2d_pair(dst + A_STAGE_BYTES, &tmW, w_kb * BK, row + 2 * BM, fb, pol_w);
        if (++w_kb == p.num_kb) { w_kb = 0; ++w_job; }
      };
      auto load_x = [&](int i) {
        const int mchunk = p.lock > 1 ? my_chunk : x_job / p.tiles;
        const int s = i % PAIR_STAGES;
        const uint32_t fb = mapa_u32(smem_u32(&full_bar[s]), 0);
        tma_load_2d_pair(smem_base + (uint32_t)s * PAIR_STAGE_BYTES + 2 * A_STAGE_BYTES, &tmX, x_kb * BK,
                         mchunk * PAIR_ACT + (int)rank * BM, fb, pol_x);
        if (++x_kb == p.num_kb) { x_kb = 0; ++x_job; }
      };
      const int pre = n_units < PAIR_STAGES ? n_units : PAIR_STAGES;
      for (int i = 0; i < pre; ++i) load_w(i);
      asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tmX) : "memory");
      griddep_wait();
      griddep_launch();
      if (p.clk) atomicMin(p.clk, globaltimer_ns());
      for (int i = 0; i < pre; ++i) load_x(i);
      int issued = pre;
      for (int i = pre; i < n_units; ++i) {
        const int s = i % PAIR_STAGES;
        const uint32_t ph = (uint32_t)(i / PAIR_STAGES) & 1u;
        if (!mbar_wait_cluster(smem_u32(&empty_bar[s]), ph ^ 1u, wc, 211)) break;
        load_w(i);
        load_x(i);
        issued = i + 1;
      }
      if (*aborted) {
        // give-up path: this CTA's copies land in its own shared memory but are counted on the first CTA's
        // barriers, and the two CTAs may have stopped at different units, so neither can see exactly its own
        // copies in.  The first CTA waits for the stages it knows of (short budget); then both let the time of
        // many memory round trips pass before they go on to the rendezvous and leave.
        if (first)
          for (int i = issued > PAIR_STAGES ? issued - PAIR_STAGES : 0; i < issued; ++i)
            mbar_wait_drain(smem_u32(&full_bar[i % PAIR_STAGES]), (uint32_t)(i / PAIR_STAGES) & 1u, 2000000ll);
        const long long t_land = clock64();
        while (clock64() - t_land < 400000ll) __nanosleep(1000);
      }
    }
  } else if (warp == 1 || warp == 6) {
    // MMA issuers of the pair: the first CTA's warps 1 (hf 0) and 6 (hf 1)
    const int hf = warp == 6 ? 1 : 0;
    if (first && lane == 0) {
      const uint32_t idesc = idesc_bf16(2 * BM, PAIR_ACT, false, false);
      int u = u0;
      Segment sg;
      int i = 0, g = 0;
      while (next_segment(u, u1, p.num_kb, sg)) {
        if (!mbar_wait_cluster(smem_u32(&acc_empty), ((uint32_t)g & 1u) ^ 1u, wc, 212)) break;
        tc_fence_after();
        const uint32_t d = tmem_base + (uint32_t)(hf * PAIR_ACT);
        for (int k = 0; k < sg.nkb; ++k, ++i) {
          const int s = i % PAIR_STAGES;
          const uint32_t ph = (uint32_t)(i / PAIR_STAGES) & 1u;
          if (!mbar_wait_cluster(smem_u32(&full_bar[s]), ph, wc, 213)) break;
          tc_fence_after();
          const uint32_t src = smem_base + (uint32_t)s * PAIR_STAGE_BYTES;
          const uint64_t adesc = desc_k_sw128(src + (uint32_t)hf * A_STAGE_BYTES);
          const uint64_t bdesc = desc_k_sw128(src + 2 * A_STAGE_BYTES);
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk)
            umma_bf16_pair(d, adesc + (uint64_t)(kk * 2), bdesc + (uint64_t)(kk * 2), idesc, (k > 0 || kk > 0) ? 1u : 0u);
          umma_commit_pair(smem_u32(&empty_bar[s]));       // the stage is free in both CTAs once these MMAs have read it
        }
        if (*aborted) break;
        umma_commit_pair(smem_u32(&acc_full));
        ++g;
      }
      if (*aborted) {
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&drain_bar[hf])) : "memory");
        mbar_wait_drain(smem_u32(&drain_bar[hf]), 0, 40000000ll);
      }
    }
  } else {
    const int quarter = warp & 3;                    // TMEM lanes 32*quarter .. +31 belong to this warp
    griddep_wait();                                  // the kernel before this one may still be reading the partial buffer
    const uint32_t ae = mapa_u32(smem_u32(&acc_empty), 0);
    int u = u0;
    Segment sg;
    int g = 0;
    while (next_segment(u, u1, p.num_kb, sg)) {
      const int tile = sg.job % p.tiles, mchunk = p.lock > 1 ? my_chunk : sg.job / p.tiles;
      if (!mbar_wait_cluster(smem_u32(&acc_full), (uint32_t)g & 1u, wc, 214)) break;
      tc_fence_after();
      const int job_u0 = sg.job * p.num_kb;
      const int first_share = job_u0 / p.per;
      const int last_share = (job_u0 + p.num_kb - 1) / p.per;
      const int slot = share - first_share;
      const int m_base = mchunk * PAIR_ACT;
      const int m_cnt = min(PAIR_ACT, p.M - m_base);
      const size_t ldo = (size_t)p.N;
      for (int hf = 0; hf < 2; ++hf) {
        const int n_out = tile * PAIR_TILE + hf * 2 * BM + (int)rank * BM + quarter * 32 + lane;
        const bool n_ok = n_out < p.N;
        float* o = p.out + ((size_t)slot * p.M + m_base) * ldo + (n_ok ? n_out : 0);
        const uint32_t taddr = tmem_base + (uint32_t)(hf * PAIR_ACT) + ((uint32_t)(quarter * 32) << 16);
        for (int c0 = 0; c0 < m_cnt; c0 += 16) {
          uint32_t r[16];
          tmem_ld16(taddr + (uint32_t)c0, r);
          if (n_ok) {
            if (c0 + 16 <= m_cnt) {
#pragma unroll
              for (int j = 0; j < 16; ++j) { *o = __uint_as_float(r[j]); o += ldo; }
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j)
                if (c0 + j < m_cnt) { *o = __uint_as_float(r[j]); o += ldo; }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(ae);          // (the first CTA's own warps arrive the same way)
      if (share == last_share) {
        for (int hf = 0; hf < 2; ++hf) {
          const int n_out = tile * PAIR_TILE + hf * 2 * BM + (int)rank * BM + quarter * 32 + lane;
          if (n_out >= p.N) continue;
          for (int z = last_share - first_share + 1; z < p.nslots; ++z) {
            float* zo = p.out + ((size_t)z * p.M + m_base) * ldo + n_out;
            for (int m = 0; m < m_cnt; ++m) { *zo = 0.f; zo += ldo; }
          }
        }
      }
      ++g;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (p.clk && threadIdx.x == 0) atomicMax(p.clk + kGemmClockSlots, globaltimer_ns());
  // Neither CTA leaves (nor frees its tensor memory) before the other is done: copies, commits and arrivals cross
  // between them until then.  The rendezvous keeps a budget of its own, far above that of the other waits, so that a
  // CTA which has given up still finds its partner.
  if (warp == 2) cluster_meet_before_exit(&meet_bar, 2, lane, wc, &meet_flag_s, 215);
  __syncthreads();
  if (warp == 1)
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
}

struct GemmPlan {
  int tiles, mchunks, num_kb, per, ctas, nslots, lock;
  bool pair;         // CTA pairs (gemm_bf16_pair_kernel): `ctas` then counts pairs, a unit is 512 weight rows
  long long total;   // checked to fit 31 bits before launch
};

// Up to 128 rows: single CTAs, one pass over all rows.  More: CTA pairs, 256 rows per pass.
GemmPlan make_plan(int sm_count, int M, int N, int K) {
  GemmPlan g;
  g.pair = M > BM;
  if (g.pair) sm_count /= 2;                   // workers are pairs
  const int rows_per_tile = g.pair ? PAIR_TILE : 2 * BM;     // a unit is two weight tiles of 128 rows (of 256 for a pair)
  g.tiles = (N + rows_per_tile - 1) / rows_per_tile;
  g.mchunks = g.pair ? (M + PAIR_ACT - 1) / PAIR_ACT : 1;
  g.num_kb = (K + BK - 1) / BK;
  // More than one row chunk: the (tile, k block) list of ONE chunk is cut into (pairs / chunks) shares and every
  // share is walked by `chunks` pairs side by side, one per row chunk.  They ask for the same weight tiles at the
  // same time, so HBM delivers every weight byte once instead of once per row chunk (measured at 2048 rows x
  // 22016 x 4096 before this: 1.58 GB of DRAM reads for 180 MB of weights, the kernel at 70 % of DRAM throughput).
  g.lock = (g.mchunks > 1 && g.mchunks * 2 <= sm_count) ? g.mchunks : 1;
  const int jobs = g.lock > 1 ? g.tiles : g.tiles * g.mchunks;
  const int shares = sm_count / g.lock;
  g.total = (long long)jobs * g.num_kb;
  long long per = (g.total + shares - 1) / shares;
  int min_per = g.num_kb < 4 ? g.num_kb : 4;          // do not shred tiny problems into one-block segments
  if (per < min_per) per = min_per;
  g.per = (int)per;
  g.ctas = (int)((g.total + per - 1) / per) * g.lock;
  g.nslots = 1;
  for (long long job = 0; job < (long long)jobs; ++job) {
    int first = (int)(job * g.num_kb / per), last = (int)((job * g.num_kb + g.num_kb - 1) / per);
    if (last - first + 1 > g.nslots) g.nslots = last - first + 1;
  }
  return g;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

// A box row is 128 bytes (64 bf16); with 256-byte L2 promotion the memory side fetches the neighbouring 128
// bytes of every row as well, i.e. the next (or previous) k block of the same rows, which the same CTA asks
// for right afterwards: DRAM bursts twice as long.  Measured on the 7B decoding step: 4.23 -> 4.02 ms per
// 64-node forward, 3.49 -> 3.31 ms per one-node forward (128-byte promotion and none are equal).

// The last descriptors made, by their arguments.  A descriptor depends on nothing else, and the stand-alone entry
// points (which own no context to keep maps in) are typically called again and again on the same buffers: they
// find their maps here instead of encoding two to six of them per call.
struct MapKey {
  const void* base;
  uint64_t inner, outer, row_bytes;
  uint32_t box_inner, box_outer;
  bool operator==(const MapKey& o) const {
    return base == o.base && inner == o.inner && outer == o.outer && row_bytes == o.row_bytes && box_inner == o.box_inner &&
           box_outer == o.box_outer;
  }
};
constexpr int kMapCache = 32;
std::mutex g_map_mutex;
MapKey g_map_key[kMapCache];
CUtensorMap g_map_val[kMapCache];
int g_map_used = 0, g_map_next = 0;

int encode_2d(CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer, uint64_t row_bytes, uint32_t box_inner,
              uint32_t box_outer) {
  if (init_driver_api() != CERB_OK) return CERB_E_CUDA;
  if (((uintptr_t)base & 15) || (row_bytes & 15)) return CERB_E_SHAPE;
  const MapKey key{base, inner, outer, row_bytes, box_inner, box_outer};
  {
    std::lock_guard<std::mutex> lock(g_map_mutex);
    for (int i = 0; i < g_map_used; ++i)
      if (g_map_key[i] == key) {
        *out = g_map_val[i];
        return CERB_OK;
      }
  }
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {row_bytes};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return CERB_E_CUDA;
  std::lock_guard<std::mutex> lock(g_map_mutex);
  g_map_key[g_map_next] = key;
  g_map_val[g_map_next] = *out;
  g_map_next = (g_map_next + 1) % kMapCache;
  if (g_map_used < kMapCache) ++g_map_used;
  return CERB_OK;
}

}  // namespace

int init_driver_api() {
  if (g_encode) return CERB_OK;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn ||
      q != cudaDriverEntryPointSuccess)
    return CERB_E_CUDA;
  g_encode = (EncodeTiledFn)fn;
  return CERB_OK;
}

int make_weight_map(CUtensorMap* out, const void* W, int N, int K) {
  return encode_2d(out, W, (uint64_t)K, (uint64_t)N, (uint64_t)K * 2, BK, BM);
}

int make_act_maps(ActMaps* out, const void* X, int rows_alloc, int K) {
  for (int b = 0; b < kRowBuckets; ++b)
    CERB_TRY(encode_2d(&out->m[b], X, (uint64_t)K, (uint64_t)rows_alloc, (uint64_t)K * 2, BK, (uint32_t)bucket_rows(b)));
  return CERB_OK;
}

// 2-D map over one layer's KV pool viewed as [pages*H*16 rows][Dh]: a box is one page of one head,
// 64 elements (128 bytes) wide.
int make_pool_map(CUtensorMap* out, const void* pool, int n_pool_pages, int H, int Dh) {
  return encode_2d(out, pool, (uint64_t)Dh, (uint64_t)n_pool_pages * H * CERB_PAGE, (uint64_t)Dh * 2, 64, CERB_PAGE);
}

// Number of partial slots the schedule produces for this problem (what consumers must sum).
// The fused SwiGLU epilogue needs the wide schedule (both halves of a unit in one CTA) and whole tiles.
// It pays for few rows only (the auto-regressive step): the CTA that completes a tile re-reads the
// tile's slots with its 128 epilogue threads, which at 64 rows took 55 us per layer against the
// 6.6 us of the separate kernel that spreads the same bytes over every SM (measured).
bool gemm_swiglu_fusable(int M, int F) {
  return M >= 1 && M <= 16 && F % BM == 0;
}
// The same reasoning for the RoPE + cache-append epilogue of the QKV GEMM (head_dim 128: a 128-row weight tile is one
// head, so both elements of every rotation pair lie in the tile that the finishing CTA owns).
bool gemm_rope_fusable(int M, int head_dim) {
  return M >= 1 && M <= 16 && head_dim == 128;
}
int gemm_plan_split(int sm_count, int M, int N, int K) { return make_plan(sm_count, M, N, K).nslots; }

int launch_gemm_bf16(cerb_ctx* c, const CUtensorMap* tmW, const ActMaps* tmX, float* out, int M, int N, int K,
                     int nsplit, int32_t* status, cudaStream_t st, const GemmEpilogue* epi, unsigned long long* clock_slot) {
  if (M <= 0 || N <= 0 || K <= 0 || (K % 8) != 0) return CERB_E_SHAPE;
  static int sm_count = 0;
  if (!sm_count) {
    int dev = 0;
    CERB_CUDA_OK(cudaGetDevice(&dev));
    CERB_CUDA_OK(cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev));
    if (sm_count > 148) sm_count = 148;      // slot counts are planned for at most 148 CTAs
  }
  // Fewer SMs than planned for would need more slots than the caller sized: plan with the number
  // the caller used (148) and simply run that many CTAs; the hardware queues what does not fit.
  GemmPlan g = make_plan(148, M, N, K);
  if (g.nslots != nsplit) return CERB_E_ARG;
  if (g.pair) {
    if (epi && epi->kind != 0) return CERB_E_SHAPE;
    if (g.total >= (1ll << 30)) return CERB_E_SHAPE;
    GemmParams q;
    memset(&q, 0, sizeof(q));
    q.out = out; q.status = status;
    q.M = M; q.N = N; q.K = K;
    q.n_mma = PAIR_ACT; q.num_kb = g.num_kb; q.tiles = g.tiles; q.per = g.per; q.total = (int)g.total; q.lock = g.lock;
    q.nslots = g.nslots; q.stages = PAIR_STAGES; q.wait_cycles = wait_cycles(); q.acc_cols = 2u * PAIR_ACT; q.acc_bufs = 1;
    q.tile_rows = PAIR_TILE; q.half_off = 2 * BM;
    q.clk = clock_slot;
    const size_t smem = (size_t)PAIR_STAGES * PAIR_STAGE_BYTES + 1024;
    static bool pair_configured = false;
    if (!pair_configured) {
      CERB_CUDA_OK(cudaFuncSetAttribute(gemm_bf16_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      pair_configured = true;
    }
    // each CTA loads 128 of the pass's 256 activation rows: the map with 128-row boxes
    if (launch_pdl_cluster(gemm_bf16_pair_kernel, dim3(2 * g.ctas), dim3(224), smem, st, 2u, *tmW, tmX->m[row_bucket(BM)], q) != cudaSuccess)
      return CERB_E_CUDA;
    CERB_LAUNCH_CHECK(c);
    return CERB_OK;
  }
  GemmParams p;
  memset(&p, 0, sizeof(p));
  int bucket = row_bucket(M);                   // (M <= 128 here)
  p.out = out;
  p.status = status;
  p.M = M; p.N = N; p.K = K;
  p.n_mma = bucket_rows(bucket);
  p.num_kb = g.num_kb;
  p.tiles = g.tiles;
  p.per = g.per;
  if (g.total >= (1ll << 30)) return CERB_E_SHAPE;
  p.total = (int)g.total;
  p.lock = 1;
  p.nslots = g.nslots;
  p.tile_rows = 2 * BM;
  p.wait_cycles = wait_cycles();
  p.half_off = BM;
  p.epi = 0; p.F = 0; p.act = nullptr; p.tickets = nullptr;
  p.clk = clock_slot;
  if (epi && epi->kind == 1) {
    if (!gemm_swiglu_fusable(M, N / 2) || (N & 1) || g.tiles * g.mchunks > kGemmTickets || !epi->act || !epi->tickets) return CERB_E_SHAPE;
    p.epi = 1; p.F = N / 2; p.act = (bf16*)epi->act; p.tickets = epi->tickets;
    p.tile_rows = BM;            // a unit = gate tile t (rows t*128..) and up tile t (rows F + t*128..)
    p.half_off = p.F;
  }
  if (epi && epi->kind == 2) {
    if (!epi->rope || !gemm_rope_fusable(M, 128) || N != 3 * epi->rope->H * 128 || g.tiles > kGemmTickets || !epi->tickets) return CERB_E_SHAPE;
    p.epi = 2; p.tickets = epi->tickets; p.re = *epi->rope;
  }
  uint32_t stage_bytes = 2 * A_STAGE_BYTES + (uint32_t)p.n_mma * BK * 2;
  p.stages = (int)((216u * 1024u) / stage_bytes);
  if (p.stages > MAX_STAGES) p.stages = MAX_STAGES;
  if (p.stages < 2) return CERB_E_SHAPE;
  p.acc_cols = 2u * (uint32_t)p.n_mma;            // two weight tiles side by side (at least 32 columns)
  p.acc_bufs = 2;                                 // 2 x (2 x 128) columns at most
  // instruction descriptor: D fp32, A and B bf16, both K-major, N = n_mma, M = 128
  p.idesc = idesc_bf16(BM, (uint32_t)p.n_mma, false, false);
  size_t smem = (size_t)p.stages * stage_bytes + 1024;
  if (smem < 120 * 1024) smem = 120 * 1024;    // one CTA per SM: a CTA may then own all of tensor memory
  static bool configured = false;
  if (!configured) {
    CERB_CUDA_OK(cudaFuncSetAttribute(gemm_bf16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(220 * 1024)));
    configured = true;
  }
  if (launch_pdl(gemm_bf16_kernel, dim3(g.ctas), dim3(224), smem, st, *tmW, tmX->m[bucket], p) != cudaSuccess) return CERB_E_CUDA;
  CERB_LAUNCH_CHECK(c);
  return CERB_OK;
}

}  // namespace cerb
