// Tree-verification attention (Sections 1 and 3.1: all candidates are verified in one pass with
// tree attention).  Query i of a sequence sees every committed prefix key and those tree keys j
// that are its ancestors (bit j of anc[i]), nothing else.
//
// bf16 path: one CTA per (split, head, sequence).  A producer warp streams 64-key tiles (four
// 16-token pages of one head, K and V) into shared memory with TMA, 128-byte swizzled, through an
// mbarrier ring; compute warps run QK^T and PV on tensor cores (warp-level MMA, fp32 accumulate)
// with an online softmax in registers.  Warps are arranged WQ x WK: WQ blocks of 16 query rows,
// WK slices of each key tile, so small trees still use every warp.  Long contexts are split along
// the keys; each split writes an unnormalised partial (m, l, O) and the last CTA to finish for a
// (sequence, head) merges the partials in split order, so the result does not depend on timing.
//
// fp32 path (CERB_F32 models): plain FMA arithmetic, one CTA per (node, head, sequence).
#include <stdlib.h>

#include <atomic>

#include "tc_common.cuh"

namespace cerb {

namespace {

constexpr int TILE = 64;                  // keys per pipeline stage = 4 pages
constexpr int PAGES_PER_TILE = TILE / CERB_PAGE;
constexpr int kTargetCtas = 296;          // two CTAs per SM on a 148-SM part
constexpr int kMaxSplit = 32;
constexpr int kMaxPagesPerCta = 1024;
constexpr size_t kCounterBytes = 4096;    // one ticket counter per (sequence, head)

// K/V tiles are read once per step (the next layer's tiles, and 13 GB of weights, come before they are needed
// again): they enter L2 with evict-first priority so that they do not push out activations and partial sums.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  tma_load_2d_hint(dst, map, x, y, bar, l2_policy(true));
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void compute_bar(int nthreads) { asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory"); }

// Which of the 64 keys key0 .. key0 + 63 one query row may see, as a bit mask (bit j <-> key key0 + j): prefix keys
// (position < L) always, tree keys by the row's ancestor words a0, a1, a2 (tree index = position - L).  Ancestor
// words have no bits at or above the live node count, so keys past the last live tree key come out invisible.
// Called only for tiles that reach past the prefix (key0 + 64 > L).
__device__ __forceinline__ uint64_t tile_visibility(int key0, int L, uint64_t a0, uint64_t a1, uint64_t a2) {
  const int base = key0 - L;                       // tree index of the tile's first key; negative: the tile starts in the prefix
  if (base < 0) {
    const int s = -base;                           // 1 .. 63 prefix keys, then tree keys 0 .. 63 - s
    return (a0 << s) | ((1ull << s) - 1ull);
  }
  const int w = base >> 6, sh = base & 63;
  const uint64_t lo = w == 0 ? a0 : w == 1 ? a1 : w == 2 ? a2 : 0ull;
  const uint64_t hi = w == 0 ? a1 : w == 1 ? a2 : 0ull;
  return sh ? (lo >> sh) | (hi << (64 - sh)) : lo;
}

struct AttnParams {
  const bf16* q;
  const int32_t* page_table;
  const int32_t* len;
  const int32_t* n_active;
  const uint64_t* anc;
  const int32_t* row_off;   // first row of every sequence in q / out, or null: sequence b starts at row b * n
  bf16* out;
  float* lse;
  float* partial;           // [B*H][nsplit][NQ][DH+4]
  unsigned int* counters;   // [B*H]
  int32_t* status;
  int n, H, max_pages, nsplit, oob_row;
  int row0, rows;           // query rows row0 .. row0 + rows - 1 of the tree are this launch's (q, out, lse and anc already point
                            // at row0); a tree of more than 128 nodes takes two launches.  n stays the tree's node count
                            // (the row stride between sequences); only keys below row0 + rows can be ancestors of these rows.
  int rows_pad;             // rows per split in `partial` (16, 32, 64 or 128)
  uint32_t v_lbo, v_sbo;    // byte offsets of the V operand's descriptor (tensor-core path)
  long long wait_cycles;    // budget of every bounded wait, SM clock cycles
  int cluster;              // tensor-core path: the splits of a (sequence, head) form one cluster and merge through shared memory
  float scale_log2;
};

template <int DH, int WQ, int WK, int STAGES>
__global__ void __launch_bounds__((WQ * WK + 1) * 32) tree_attn_bf16_kernel(const __grid_constant__ CUtensorMap tmK,
                                                                          const __grid_constant__ CUtensorMap tmV,
                                                                          const AttnParams p) {
  constexpr int NW = WQ * WK;               // compute warps
  constexpr int NQ = WQ * 16;               // query rows of this CTA
  constexpr int KW = TILE / WK;             // keys per warp per tile
  constexpr int NT = KW / 8;                // 8-key score tiles per warp
  constexpr int HALVES = DH / 64;
  constexpr uint32_t HALF_BYTES = TILE * 128;
  constexpr uint32_t KV_BYTES = HALVES * HALF_BYTES;      // one of K or V for a stage
  constexpr uint32_t STAGE_BYTES = 2 * KV_BYTES;
  constexpr int ROWF = DH + 4;                            // merge row: O[DH], m, l, pad (16-byte rows)
  static_assert(NQ * ROWF * 4 <= STAGES * STAGE_BYTES, "merge buffer must fit in the stage ring");

  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[STAGES];
  __shared__ __align__(8) uint64_t empty_bar[STAGES];
  __shared__ int page_list[kMaxPagesPerCta];
  __shared__ int aborted_s, exit_flag_s;
  __shared__ unsigned int ticket_s;
  __shared__ __align__(8) uint64_t cl_bar[2];
  volatile int* aborted = &aborted_s;
  const WaitCtx wc{p.wait_cycles, aborted, p.status};

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  // Lengths, live node counts, the page table and the prefix keys were written at least two kernels ago:
  // set-up, the page list and the first prefix tiles run before griddep_wait() and overlap the previous
  // kernel's tail; Q and this step's tree keys are only touched after it.
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int L = p.len[b];
  const int nq_all = p.n_active ? min(p.n_active[b], p.n) : p.n;      // live nodes of this sequence
  const size_t qrow = p.row_off ? (size_t)p.row_off[b] : (size_t)b * p.n;   // this sequence's first row of q and out
  const int nq = min(nq_all - p.row0, p.rows);                        // live query rows of this launch
  if (nq <= 0) return;
  const int kv_total = L + min(nq_all, p.row0 + p.rows);
  const int tiles = (kv_total + TILE - 1) / TILE;
  const int per = (tiles + p.nsplit - 1) / p.nsplit;
  const int t0 = min(tiles, split * per), t1 = min(tiles, t0 + per);
  const bool too_long = per * PAGES_PER_TILE > kMaxPagesPerCta;

  if (threadIdx.x == 0) {
    aborted_s = (*p.status != 0);
    exit_flag_s = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), NW);
    }
    mbar_init(smem_u32(&cl_bar[0]), (uint32_t)p.nsplit);
    mbar_init(smem_u32(&cl_bar[1]), (uint32_t)p.nsplit);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (too_long) atomicExch(p.status, CERB_E_SHAPE);
  }
  __syncthreads();
  if (p.cluster) cluster_start_arrive();
  const int t_end = too_long ? t0 : t1;

  float* mrg = reinterpret_cast<float*>(smem_gen);   // [NQ][ROWF], used after the key loop

  if (warp == NW) {
    // ---------------- producer warp ----------------
    const int32_t* pt = p.page_table + (size_t)b * p.max_pages;
    const int n_pages = (t_end - t0) * PAGES_PER_TILE;
    for (int i = lane; i < n_pages; i += 32) {
      int lp = t0 * PAGES_PER_TILE + i;
      page_list[i] = (lp * CERB_PAGE < kv_total && lp < p.max_pages) ? (pt[lp] * p.H + h) * CERB_PAGE : p.oob_row;
    }
    __syncwarp();
    if (lane == 0) {
      int early = 0;
      while (t0 + early < t_end && early < STAGES && (t0 + early + 1) * TILE <= L) ++early;
      // (the abort flag itself is looked at once, for a launch that starts after a time-out: nothing is issued then;
      // later a wait that gives up says so in its return value, which costs the loop nothing)
      const int t_stop = *aborted ? t0 : t_end;
      int i = 0;
      for (int t = t0; t < t_stop; ++t, ++i) {
        if (i == early) { griddep_wait(); griddep_launch(); }
        int s = i % STAGES;
        uint32_t ph = (uint32_t)(i / STAGES) & 1u;
        if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, wc, 301)) break;      // the consumers have stopped: issue nothing more
        uint32_t fb = smem_u32(&full_bar[s]);
        mbar_expect_tx(fb, STAGE_BYTES);
        uint32_t kdst = smem_base + (uint32_t)s * STAGE_BYTES, vdst = kdst + KV_BYTES;
#pragma unroll
        for (int pg = 0; pg < PAGES_PER_TILE; ++pg) {
          int row = page_list[i * PAGES_PER_TILE + pg];      // out-of-range rows are zero-filled by TMA
#pragma unroll
          for (int hf = 0; hf < HALVES; ++hf) {
            uint32_t off = (uint32_t)hf * HALF_BYTES + (uint32_t)pg * (CERB_PAGE * 128);
            tma_load_2d(kdst + off, &tmK, hf * 64, row, fb);
            tma_load_2d(vdst + off, &tmV, hf * 64, row, fb);
          }
        }
      }
      if (*aborted) {
        // give-up path: the copies already issued (units 0 .. i-1) still land in this CTA's shared memory; see each of them in
        for (int j = i > STAGES ? i - STAGES : 0; j < i; ++j)
          mbar_wait_drain(smem_u32(&full_bar[j % STAGES]), (uint32_t)(j / STAGES) & 1u, 20000000ll);
      }
    }
    griddep_wait();      // (a lane that has waited already returns at once)
    griddep_launch();
  } else {
    // ---------------- compute warps ----------------
    griddep_wait();
    griddep_launch();
    const int qi = warp % WQ, ki = warp / WQ;
    const int g = lane >> 2, tq = lane & 3;
    const int r0 = qi * 16 + g, r1 = r0 + 8;                // this thread's two query rows
    // Q fragments straight from global memory (A operand of m16n8k16, one per 16 head-dim elements)
    uint32_t qa[DH / 16][4];
    {
      const bf16* q0 = p.q + ((qrow + r0) * p.H + h) * DH;
      const bf16* q1 = p.q + ((qrow + r1) * p.H + h) * DH;
#pragma unroll
      for (int kk = 0; kk < DH / 16; ++kk) {
        int c = kk * 16 + tq * 2;
        qa[kk][0] = r0 < nq ? *reinterpret_cast<const uint32_t*>(q0 + c) : 0u;
        qa[kk][1] = r1 < nq ? *reinterpret_cast<const uint32_t*>(q1 + c) : 0u;
        qa[kk][2] = r0 < nq ? *reinterpret_cast<const uint32_t*>(q0 + c + 8) : 0u;
        qa[kk][3] = r1 < nq ? *reinterpret_cast<const uint32_t*>(q1 + c + 8) : 0u;
      }
    }
    uint64_t anc0[CERB_ANC_WORDS], anc1[CERB_ANC_WORDS];
#pragma unroll
    for (int w = 0; w < CERB_ANC_WORDS; ++w) {
      anc0[w] = r0 < nq ? p.anc[r0 * CERB_ANC_WORDS + w] : 0ull;
      anc1[w] = r1 < nq ? p.anc[r1 * CERB_ANC_WORDS + w] : 0ull;
    }

    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    float o[DH / 8][4];
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }

    for (int t = t0, it = 0; t < t_end; ++t, ++it) {
      const int s = it % STAGES;
      const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
      mbar_wait(smem_u32(&full_bar[s]), ph, wc, 302);
      const uint32_t kbase = smem_base + (uint32_t)s * STAGE_BYTES, vbase = kbase + KV_BYTES;
      const int key_tile0 = t * TILE;
      if (key_tile0 + TILE > kv_total) {
        // last, partial tile: rows past the end may hold anything (stale pool memory); zero V there so
        // that a zero probability times a non-finite value cannot poison the sum.
        const int first_bad = kv_total - key_tile0;
        uint8_t* vgen = smem_gen + (size_t)s * STAGE_BYTES + KV_BYTES;
        for (int idx = warp * 32 + lane; idx < (TILE - first_bad) * HALVES * 8; idx += NW * 32) {
          int row = first_bad + idx / (HALVES * 8), rem = idx % (HALVES * 8);
          *reinterpret_cast<uint4*>(vgen + (size_t)(rem / 8) * HALF_BYTES + row * 128 + (rem % 8) * 16) = make_uint4(0, 0, 0, 0);
        }
        compute_bar(NW * 32);
      }

      // ---- S = Q K^T for this warp's key slice ----
      float sc[NT][4];
#pragma unroll
      for (int i = 0; i < NT; ++i) { sc[i][0] = sc[i][1] = sc[i][2] = sc[i][3] = 0.f; }
      const int mat = lane >> 3, lr = lane & 7;
#pragma unroll
      for (int kk = 0; kk < DH / 16; ++kk) {
#pragma unroll
        for (int nt = 0; nt < NT; nt += 2) {
          int key = ki * KW + nt * 8 + (mat >> 1) * 8 + lr;
          int chunk = kk * 2 + (mat & 1);
          uint32_t addr = kbase + (uint32_t)(chunk >> 3) * HALF_BYTES + (uint32_t)key * 128 + (uint32_t)(((chunk & 7) ^ (key & 7)) << 4);
          uint32_t b0, b1, b2, b3;
          ldsm_x4(addr, b0, b1, b2, b3);
          mma_bf16(sc[nt], qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], b0, b1);
          mma_bf16(sc[nt + 1], qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], b2, b3);
        }
      }

      // ---- mask, online softmax ----
      const bool need_mask = key_tile0 + TILE > L;
      uint64_t vm0 = ~0ull, vm1 = ~0ull;             // visible keys of this tile for rows r0 and r1
      if (need_mask) {
        vm0 = tile_visibility(key_tile0, L, anc0[0], anc0[1], anc0[2]);
        vm1 = tile_visibility(key_tile0, L, anc1[0], anc1[1], anc1[2]);
      }
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float v = sc[nt][e] * p.scale_log2;
          if (need_mask) {
            const int j = ki * KW + nt * 8 + tq * 2 + (e & 1);          // key's index inside the tile
            if (!((((e < 2) ? vm0 : vm1) >> j) & 1ull)) v = -INFINITY;
          }
          sc[nt][e] = v;
          if (e < 2) mx0 = fmaxf(mx0, v); else mx1 = fmaxf(mx1, v);
        }
      }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
      const float mu0 = mn0 == -INFINITY ? 0.f : mn0, mu1 = mn1 == -INFINITY ? 0.f : mn1;
      const float al0 = exp2f(m0 - mu0), al1 = exp2f(m1 - mu1);
      m0 = mn0; m1 = mn1;
      float rs0 = 0.f, rs1 = 0.f;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        sc[nt][0] = exp2f(sc[nt][0] - mu0); sc[nt][1] = exp2f(sc[nt][1] - mu0);
        sc[nt][2] = exp2f(sc[nt][2] - mu1); sc[nt][3] = exp2f(sc[nt][3] - mu1);
        rs0 += sc[nt][0] + sc[nt][1];
        rs1 += sc[nt][2] + sc[nt][3];
      }
      l0 = l0 * al0 + rs0;
      l1 = l1 * al1 + rs1;
#pragma unroll
      for (int i = 0; i < DH / 8; ++i) { o[i][0] *= al0; o[i][1] *= al0; o[i][2] *= al1; o[i][3] *= al1; }

      // ---- O += P V ----
#pragma unroll
      // Probabilities enter the tensor core as two bf16 terms, p = p_hi + p_lo (about 16 significant
      // bits), so that the product is not limited by bf16's 8-bit significand: with near-uniform
      // attention over many keys a single bf16 term costs as much accuracy as all other roundings together.
      for (int j = 0; j < KW / 16; ++j) {
        uint32_t ah[4], al[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float p0 = sc[2 * j + (e >> 1)][(e & 1) * 2], p1 = sc[2 * j + (e >> 1)][(e & 1) * 2 + 1];
          __nv_bfloat162 hi = __floats2bfloat162_rn(p0, p1);
          float2 hf = __bfloat1622float2(hi);
          ah[e] = *reinterpret_cast<uint32_t*>(&hi);
          al[e] = pack_bf16(p0 - hf.x, p1 - hf.y);
        }
#pragma unroll
        for (int dn = 0; dn < DH / 8; dn += 2) {
          int key = ki * KW + j * 16 + (mat & 1) * 8 + lr;
          int chunk = dn + (mat >> 1);
          uint32_t addr = vbase + (uint32_t)(chunk >> 3) * HALF_BYTES + (uint32_t)key * 128 + (uint32_t)(((chunk & 7) ^ (key & 7)) << 4);
          uint32_t b0, b1, b2, b3;
          ldsm_x4_t(addr, b0, b1, b2, b3);
          mma_bf16(o[dn], ah[0], ah[1], ah[2], ah[3], b0, b1);
          mma_bf16(o[dn + 1], ah[0], ah[1], ah[2], ah[3], b2, b3);
          mma_bf16(o[dn], al[0], al[1], al[2], al[3], b0, b1);
          mma_bf16(o[dn + 1], al[0], al[1], al[2], al[3], b2, b3);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&empty_bar[s]));
    }

    // ---- combine the WK key slices of each query block, through shared memory ----
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    compute_bar(NW * 32);                       // every warp is done with the stage ring
    for (int kslice = 0; kslice < WK; ++kslice) {
      if (ki == kslice) {
        float* row0 = mrg + (size_t)r0 * ROWF;
        float* row1 = mrg + (size_t)r1 * ROWF;
        if (kslice == 0) {
#pragma unroll
          for (int i = 0; i < DH / 8; ++i) {
            int c = i * 8 + tq * 2;
            row0[c] = o[i][0]; row0[c + 1] = o[i][1]; row1[c] = o[i][2]; row1[c + 1] = o[i][3];
          }
          if (tq == 0) { row0[DH] = m0; row0[DH + 1] = l0; row1[DH] = m1; row1[DH + 1] = l1; }
        } else {
          float pm0 = row0[DH], pl0 = row0[DH + 1], pm1 = row1[DH], pl1 = row1[DH + 1];
          float n0 = fmaxf(pm0, m0), n1 = fmaxf(pm1, m1);
          float u0 = n0 == -INFINITY ? 0.f : n0, u1 = n1 == -INFINITY ? 0.f : n1;
          float wa0 = exp2f(pm0 - u0), wb0 = exp2f(m0 - u0), wa1 = exp2f(pm1 - u1), wb1 = exp2f(m1 - u1);
#pragma unroll
          for (int i = 0; i < DH / 8; ++i) {
            int c = i * 8 + tq * 2;
            row0[c] = row0[c] * wa0 + o[i][0] * wb0; row0[c + 1] = row0[c + 1] * wa0 + o[i][1] * wb0;
            row1[c] = row1[c] * wa1 + o[i][2] * wb1; row1[c + 1] = row1[c + 1] * wa1 + o[i][3] * wb1;
          }
          __syncwarp();
          if (tq == 0) {
            row0[DH] = n0; row0[DH + 1] = pl0 * wa0 + l0 * wb0;
            row1[DH] = n1; row1[DH + 1] = pl1 * wa1 + l1 * wb1;
          }
        }
      }
      compute_bar(NW * 32);
    }

    // ---- output: final, or partial + fixed-order merge by the last CTA of this (sequence, head) ----
    const int ct = warp * 32 + lane, nct = NW * 32;
    const float LN2 = 0.6931471805599453f;
    if (p.cluster) {
      // merged after the role branches, where every thread of the cluster meets
    } else if (p.nsplit == 1) {
      for (int idx = ct; idx < nq * DH; idx += nct) {
        int r = idx / DH, c = idx % DH;
        float l = mrg[(size_t)r * ROWF + DH + 1];
        p.out[((qrow + r) * p.H + h) * DH + c] = __float2bfloat16_rn(mrg[(size_t)r * ROWF + c] / l);
      }
      if (p.lse)
        for (int r = ct; r < nq; r += nct)
          p.lse[((size_t)b * p.H + h) * p.n + r] = (mrg[(size_t)r * ROWF + DH] + log2f(mrg[(size_t)r * ROWF + DH + 1])) * LN2;
    } else {
      float* part = p.partial + (((size_t)b * p.H + h) * p.nsplit) * (size_t)(NQ * ROWF);
      float* mine = part + (size_t)split * (NQ * ROWF);
      for (int idx = ct; idx < nq * ROWF; idx += nct) __stcg(mine + idx, mrg[idx]);
      __threadfence();
      compute_bar(NW * 32);
      if (ct == 0) ticket_s = atomicAdd(&p.counters[b * p.H + h], 1u);
      compute_bar(NW * 32);
      if (ticket_s == (unsigned)p.nsplit - 1) {
        __threadfence();
        // per-row merge weights first (one thread per row), then a wide, vectorised weighted sum
        float* wts = mrg;                                   // [nsplit][NQ], the merge buffer is free again
        for (int r = ct; r < nq; r += nct) {
          float M = -INFINITY;
          for (int s2 = 0; s2 < p.nsplit; ++s2) M = fmaxf(M, __ldcg(part + (size_t)s2 * (NQ * ROWF) + r * ROWF + DH));
          float Lsum = 0.f;
          for (int s2 = 0; s2 < p.nsplit; ++s2) {
            const float* pr = part + (size_t)s2 * (NQ * ROWF) + r * ROWF;
            float w = exp2f(__ldcg(pr + DH) - M);
            wts[s2 * NQ + r] = w;
            Lsum += __ldcg(pr + DH + 1) * w;
          }
          float inv = 1.0f / Lsum;
          for (int s2 = 0; s2 < p.nsplit; ++s2) wts[s2 * NQ + r] *= inv;
          if (p.lse) p.lse[((size_t)b * p.H + h) * p.n + r] = (M + log2f(Lsum)) * LN2;
        }
        compute_bar(NW * 32);
        constexpr int C4 = DH / 4;
        for (int idx = ct; idx < nq * C4; idx += nct) {
          const int r = idx / C4, c4 = idx % C4;
          const float4* src = reinterpret_cast<const float4*>(part + (size_t)r * ROWF) + c4;
          float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
          for (int s2 = 0; s2 < p.nsplit; ++s2) {
            float4 v = __ldcg(src + (size_t)s2 * (NQ * ROWF / 4));
            float w = wts[s2 * NQ + r];
            acc.x += v.x * w; acc.y += v.y * w; acc.z += v.z * w; acc.w += v.w * w;
          }
          uint2 packed = make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
          *reinterpret_cast<uint2*>(p.out + ((qrow + r) * p.H + h) * DH + c4 * 4) = packed;
        }
        if (ct == 0) p.counters[b * p.H + h] = 0u;       // ready for the next launch
      }
    }
  }
  if (p.cluster) {
    // The splits of this (sequence, head) are the CTAs of one cluster (rank = split): each holds its rows
    // (O, m, l) in shared memory; after the first barrier CTA r merges rows r, r + nsplit, ... from all members
    // in split order and writes the output.  Nobody leaves before the second meeting.
    cluster_start_wait();
    if (warp < NW) {
      cluster_meet(&cl_bar[0], p.nsplit, (int)threadIdx.x, wc, 303);     // every member's rows are in place
      constexpr int C4 = DH / 4;
      const int ct = warp * 32 + lane, rows_per_pass = (NW * 32) / C4;
      const float LN2 = 0.6931471805599453f;
      const uint32_t mine = smem_u32(smem_gen);
      const int c4 = ct % C4;
      for (int r = split + p.nsplit * (ct / C4); r < nq; r += p.nsplit * rows_per_pass) {
        const uint32_t row_off = (uint32_t)r * (ROWF * 4);
        float M = -INFINITY;
        for (int s2 = 0; s2 < p.nsplit; ++s2) M = fmaxf(M, ld_cluster_f32(mapa_u32(mine, (uint32_t)s2) + row_off + DH * 4));
        const float u = M == -INFINITY ? 0.f : M;
        float Lsum = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s2 = 0; s2 < p.nsplit; ++s2) {
          const uint32_t base = mapa_u32(mine, (uint32_t)s2) + row_off;
          const float w = exp2f(ld_cluster_f32(base + DH * 4) - u);
          Lsum += ld_cluster_f32(base + DH * 4 + 4) * w;
          const float4 v = ld_cluster_v4(base + (uint32_t)c4 * 16u);
          acc.x += v.x * w; acc.y += v.y * w; acc.z += v.z * w; acc.w += v.w * w;
        }
        const float inv = 1.0f / Lsum;
        *reinterpret_cast<uint2*>(p.out + ((qrow + r) * p.H + h) * DH + c4 * 4) =
            make_uint2(pack_bf16(acc.x * inv, acc.y * inv), pack_bf16(acc.z * inv, acc.w * inv));
        if (c4 == 0 && p.lse) p.lse[((size_t)b * p.H + h) * p.n + r] = (M + log2f(Lsum)) * LN2;
      }
      compute_bar(NW * 32);                                                          // this CTA has read all it needs
      if (warp == 0) cluster_meet_before_exit(&cl_bar[1], p.nsplit, lane, wc, &exit_flag_s, 304);
    }
    __syncthreads();                           // nobody exits before warp 0 has seen every member done
  }
}

// ---------------------------------------------------------------------------------------------
// bf16 path on the 5th-generation tensor cores (head_dim 128)
// ---------------------------------------------------------------------------------------------
// Same decomposition as above (one CTA per (split, head, sequence), 64-key tiles streamed by TMA),
// but both products run as tcgen05 MMAs with their results in tensor memory:
//   S[128 x 64]  = Q[128 x 128] . K_tile^T      (Q staged once in shared memory, zero rows past n)
//   O[128 x 128] += P[128 x 64] . V_tile        (P = p_hi + p_lo, two bf16 terms, staged in shared memory)
// Warp 0 = TMA producer, warp 1 = TMEM allocator + MMA issuer, warps 2-5 and 6-9 = two softmax groups
// that take alternate key tiles.  In a group thread t owns query row t (= TMEM lane t): it reads its
// whole S row from tensor memory with back-to-back loads and ONE wait (a dependent TMEM round trip
// costs ~600 cycles here, measured), keeps the running maximum and sum in registers and writes its P
// row (128-byte swizzled, the MMA's K-major A layout).  Each group has its own S buffer, its own O
// accumulator and its own P buffers, i.e. the two groups run two independent online-softmax streams
// over the even and the odd tiles, merged once at the end; one group's TMEM latency and arithmetic
// overlap the other's.  O stays in TMEM across tiles; it is only rescaled when a row's maximum grows
// by more than 2^8 (until then the older maximum keeps being used, which is exact after the final
// normalisation).
namespace {

constexpr uint32_t TC_KV_BYTES = 16384;               // K (or V) of one 64-key tile, two 64-wide halves
// K and V tiles travel through rings of 16 KB stages.  The depth of the rings, not HBM, sets the tile rate
// up to the point where the tensor pipe is busy (a freed stage is back after a TMA round trip of ~2 us;
// measured at 64 nodes: three K+V stages 1.36 us per 64-key tile, four or five 1.0 us).
//  * Trees of up to 64 nodes keep only 64 rows of Q and of every P buffer in shared memory (the MMAs still
//    read 128 rows; what they find past the 64th only reaches score and output rows nobody uses), which
//    leaves room for five K and five V stages; K and V of a tile then share one pair of barriers (UNI).
//  * Wider trees need all 128 rows: two K and five V stages with barriers of their own -- a K tile is
//    free again as soon as its QK^T MMAs have retired, a V tile only after the PV MMAs one softmax later.
// (One QK^T MMA set of N = 128 over two neighbouring key tiles, filling both groups' score buffers at
// once, was tried: 24 instead of 32 MMAs per 128 keys, but the groups then run in lockstep and lose
// their overlap -- 692 against 529 us at batch 16 x 64 nodes x 8K keys.)
__host__ __device__ constexpr size_t tc_smem(int sk, int sv, int qrows) {
  return (size_t)(sk + sv) * TC_KV_BYTES + 2 * (size_t)qrows * 128 + 4 * (size_t)qrows * 128 + 1024;   // rings, Q, P (2 groups x hi, lo)
}
constexpr int TC_DH = 128, TC_ROWF = TC_DH + 4;
constexpr int TC_THREADS = 352;                       // producer, QK^T issuer, two softmax groups of four warps, PV issuer
constexpr float TC_RESCALE = 8.0f;                    // log2 of the growth of a row maximum that forces a rescale

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) { tmem_ld16_nowait(taddr, r); }
__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  umma_bf16(tmem_d, adesc, bdesc, idesc, acc);
}

template <int SK, int SV, int QROWS, bool UNI>
__global__ void __launch_bounds__(TC_THREADS, 1) tree_attn_tc_kernel(const __grid_constant__ CUtensorMap tmK,
                                                                     const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
  constexpr int DH = TC_DH, ROWF = TC_ROWF;
  constexpr uint32_t QHALF = (uint32_t)QROWS * 128u, TC_Q_BYTES = 2 * QHALF;
  constexpr uint32_t TC_P_BYTES = (uint32_t)QROWS * 128u;      // P: one term (hi or lo) of one softmax group
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_k[SK], empty_k[SK], full_v[SV], empty_v[SV], s_full[2], s_free[2], p_ready[2], pv_done[2], q_ready, drain_bar[2];
  __shared__ int page_list[kMaxPagesPerCta];
  __shared__ uint32_t tmem_slot;
  __shared__ int aborted_s, exit_flag_s;
  __shared__ unsigned int ticket_s;
  __shared__ __align__(8) uint64_t cl_bar[2];
  volatile int* aborted = &aborted_s;
  const WaitCtx wc{p.wait_cycles, aborted, p.status};

  // Everything up to the first use of Q or of this step's tree keys runs before griddep_wait(): lengths,
  // live node counts and the page table were written at least two kernels ago, and so were the prefix
  // keys.  Set-up, the page list and the first prefix tiles thus overlap the previous kernel's tail.
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  // Order matters: with 64-row buffers the 128-row MMAs read 8 KB past the end of a P buffer and of Q's
  // second half; P comes first, then Q, then the rings, so that every such read stays inside this CTA's
  // shared memory (the last P buffer runs into Q, Q into the K ring).
  const uint32_t p_base = smem_base;                    // [group][hi, lo] x TC_P_BYTES
  const uint32_t q_base = p_base + 4 * TC_P_BYTES;
  const uint32_t k_ring = q_base + TC_Q_BYTES;
  const uint32_t v_ring = k_ring + SK * TC_KV_BYTES;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int L = p.len[b];
  const int nq_all = p.n_active ? min(p.n_active[b], p.n) : p.n;      // live nodes of this sequence
  const size_t qrow = p.row_off ? (size_t)p.row_off[b] : (size_t)b * p.n;   // this sequence's first row of q and out
  const int nq = min(nq_all - p.row0, p.rows);                        // live query rows of this launch
  if (nq <= 0) return;
  const int kv_total = L + min(nq_all, p.row0 + p.rows);
  const int tiles = (kv_total + TILE - 1) / TILE;
  const int per = (tiles + p.nsplit - 1) / p.nsplit;
  const int t0 = min(tiles, split * per), t1 = min(tiles, t0 + per);
  const bool too_long = per * PAGES_PER_TILE > kMaxPagesPerCta;
  const int T = too_long ? 0 : t1 - t0;

  if (threadIdx.x == 0) {
    aborted_s = (*p.status != 0);
    exit_flag_s = 0;
    for (int s = 0; s < SK; ++s) {
      mbar_init(smem_u32(&full_k[s]), 1);
      mbar_init(smem_u32(&empty_k[s]), 1);
    }
    for (int s = 0; s < SV; ++s) {
      mbar_init(smem_u32(&full_v[s]), 1);
      mbar_init(smem_u32(&empty_v[s]), 1);
    }
    for (int g = 0; g < 2; ++g) {
      mbar_init(smem_u32(&s_full[g]), 1);
      mbar_init(smem_u32(&s_free[g]), 4);
      mbar_init(smem_u32(&p_ready[g]), 4);
      mbar_init(smem_u32(&pv_done[g]), 1);
    }
    mbar_init(smem_u32(&q_ready), 4);
    mbar_init(smem_u32(&drain_bar[0]), 1);
    mbar_init(smem_u32(&drain_bar[1]), 1);
    mbar_init(smem_u32(&cl_bar[0]), (uint32_t)p.nsplit);
    mbar_init(smem_u32(&cl_bar[1]), (uint32_t)p.nsplit);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (too_long) atomicExch(p.status, CERB_E_SHAPE);
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (p.cluster) cluster_start_arrive();
  // tensor memory: columns 0-63 / 64-127 = S of group 0 / 1, 128-255 / 256-383 = O of group 0 / 1
  const uint32_t tmem = tmem_slot;
  float* mrg = reinterpret_cast<float*>(smem_gen);   // [2][128][ROWF] over the whole buffer, once the key loop is over

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    const int32_t* pt = p.page_table + (size_t)b * p.max_pages;
    const int n_pages = T * PAGES_PER_TILE;
    for (int i = lane; i < n_pages; i += 32) {
      int lp = t0 * PAGES_PER_TILE + i;
      page_list[i] = (lp * CERB_PAGE < kv_total && lp < p.max_pages) ? (pt[lp] * p.H + h) * CERB_PAGE : p.oob_row;
    }
    __syncwarp();
    // tiles of the first ring that lie wholly inside the prefix may be fetched before the wait
    int early = 0;
    while (early < T && early < SK && (t0 + early + 1) * TILE <= L) ++early;
    if constexpr (!UNI) {
      // A tile is 16 boxes of 2 KB (K and V, four pages, two 64-wide halves).  With separate K and V rings
      // (128 query rows) 16 lanes issue one box each: 4-7 % faster than one lane issuing them in turn
      // (measured, 16 x 8192 and 4 x 4096 keys); with the shared ring it is 1-5 % slower, hence the other branch.
      static_assert(PAGES_PER_TILE == 4, "the lane -> box map below assumes four pages per tile");
      const int is_v = lane >> 3, pg = (lane >> 1) & 3, hf = lane & 1;
      const int T_stop = *aborted ? 0 : T;         // a launch that starts after a time-out issues nothing
      int i = 0;
      for (; i < T_stop; ++i) {
        if (i == early) { griddep_wait(); griddep_launch(); }
        const int sk = i % SK, sv = i % SV;
        const uint32_t fk = smem_u32(&full_k[sk]), fv = smem_u32(&full_v[sv]);
        int stop = 0;
        if (lane == 0) {
          // (a wait that gives up says so in its return value: the consumers have stopped, nothing more is issued)
          if (mbar_wait_polite(smem_u32(&empty_k[sk]), ((uint32_t)(i / SK) & 1u) ^ 1u, wc, 305) &&
              mbar_wait_polite(smem_u32(&empty_v[sv]), ((uint32_t)(i / SV) & 1u) ^ 1u, wc, 306)) {
            mbar_expect_tx(fk, TC_KV_BYTES);
            mbar_expect_tx(fv, TC_KV_BYTES);
          } else {
            stop = 1;
          }
        }
        if (__any_sync(0xffffffffu, stop)) break;
        if (lane < 16) {
          const int row = page_list[i * PAGES_PER_TILE + pg];       // out-of-range rows are zero-filled by TMA
          const uint32_t dst = (is_v ? v_ring + (uint32_t)sv * TC_KV_BYTES : k_ring + (uint32_t)sk * TC_KV_BYTES) +
                               (uint32_t)hf * 8192u + (uint32_t)pg * (CERB_PAGE * 128);
          tma_load_2d(dst, is_v ? &tmV : &tmK, hf * 64, row, is_v ? fv : fk);
        }
      }
      if (lane == 0 && *aborted) {
        // give-up path: the copies already issued (tiles 0 .. i-1) still land in this CTA's shared memory; see each of them in
        for (int j = i > SK ? i - SK : 0; j < i; ++j)
          mbar_wait_drain(smem_u32(&full_k[j % SK]), (uint32_t)(j / SK) & 1u, 20000000ll);
        for (int j = i > SV ? i - SV : 0; j < i; ++j)
          mbar_wait_drain(smem_u32(&full_v[j % SV]), (uint32_t)(j / SV) & 1u, 20000000ll);
      }
    } else if (lane == 0) {
      // K and V of a tile share the V ring's barriers (SK == SV): one wait and one arrival per tile
      const int T_stop = *aborted ? 0 : T;         // a launch that starts after a time-out issues nothing
      int i = 0;
      for (; i < T_stop; ++i) {
        if (i == early) { griddep_wait(); griddep_launch(); }
        const int sv = i % SV;
        if (!mbar_wait_polite(smem_u32(&empty_v[sv]), ((uint32_t)(i / SV) & 1u) ^ 1u, wc, 307)) break;
        const uint32_t fv = smem_u32(&full_v[sv]);
        mbar_expect_tx(fv, 2 * TC_KV_BYTES);
        const uint32_t kdst = k_ring + (uint32_t)sv * TC_KV_BYTES, vdst = v_ring + (uint32_t)sv * TC_KV_BYTES;
#pragma unroll
        for (int pg = 0; pg < PAGES_PER_TILE; ++pg) {
          const int row = page_list[i * PAGES_PER_TILE + pg];       // out-of-range rows are zero-filled by TMA
#pragma unroll
          for (int hf = 0; hf < 2; ++hf)
            tma_load_2d(kdst + (uint32_t)hf * 8192u + (uint32_t)pg * (CERB_PAGE * 128), &tmK, hf * 64, row, fv);
        }
#pragma unroll
        for (int pg = 0; pg < PAGES_PER_TILE; ++pg) {
          const int row = page_list[i * PAGES_PER_TILE + pg];
#pragma unroll
          for (int hf = 0; hf < 2; ++hf)
            tma_load_2d(vdst + (uint32_t)hf * 8192u + (uint32_t)pg * (CERB_PAGE * 128), &tmV, hf * 64, row, fv);
        }
      }
      if (*aborted)
        for (int j = i > SV ? i - SV : 0; j < i; ++j)
          mbar_wait_drain(smem_u32(&full_v[j % SV]), (uint32_t)(j / SV) & 1u, 20000000ll);
    }
    griddep_wait();      // (a lane that has waited already returns at once)
    griddep_launch();
  } else if (warp == 1) {
    griddep_wait();
    griddep_launch();
    // ---------------- QK^T issuer ----------------
    // (issuing one tcgen05.mma costs this thread ~95 cycles whatever its size, measured, so the two
    // products are issued by two different warps)
    if (lane == 0 && T > 0) {
      const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
      const uint64_t q_desc0 = desc_k_sw128(q_base), q_desc1 = desc_k_sw128(q_base + QHALF);
      mbar_wait(smem_u32(&q_ready), 0, wc, 308);
      const int T_stop = *aborted ? 0 : T;
      for (int i = 0; i < T_stop; ++i) {
        const int g = i & 1, k = i >> 1;
        const bool ok_kv = !UNI ? mbar_wait(smem_u32(&full_k[i % SK]), (uint32_t)(i / SK) & 1u, wc, 309)
                                : mbar_wait(smem_u32(&full_v[i % SV]), (uint32_t)(i / SV) & 1u, wc, 310);
        if (!mbar_wait(smem_u32(&s_free[g]), ((uint32_t)k & 1u) ^ 1u, wc, 311) || !ok_kv) break;
        tc_fence_after();
        const uint32_t kb = k_ring + (uint32_t)(i % SK) * TC_KV_BYTES;
        const uint64_t k_desc0 = desc_k_sw128(kb), k_desc1 = desc_k_sw128(kb + 8192u);
        const uint32_t d = tmem + (uint32_t)g * 64u;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) umma(d, q_desc0 + (uint64_t)(kk * 2), k_desc0 + (uint64_t)(kk * 2), idesc_s, kk ? 1u : 0u);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) umma(d, q_desc1 + (uint64_t)(kk * 2), k_desc1 + (uint64_t)(kk * 2), idesc_s, 1u);
        if (!UNI) umma_commit(smem_u32(&empty_k[i % SK]));     // the K tile is free once these MMAs have retired
        umma_commit(smem_u32(&s_full[g]));
      }
      if (*aborted) {                                // give-up path: see the MMAs already issued retire
        umma_commit(smem_u32(&drain_bar[0]));
        mbar_wait_drain(smem_u32(&drain_bar[0]), 0, 20000000ll);
      }
    }
  } else if (warp == 10) {
    griddep_wait();
    griddep_launch();
    // ---------------- PV issuer ----------------
    if (lane == 0) {
      // B operand (V) is MN-major, N = 128 (two 64-wide swizzle atoms, p.v_lbo bytes apart)
      const uint32_t idesc_pv = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
      const int T_stop = *aborted ? 0 : T;
      for (int j = 0; j < T_stop; ++j) {
        const int g = j & 1, k = j >> 1;
        if (!mbar_wait(smem_u32(&p_ready[g]), (uint32_t)k & 1u, wc, 312)) break;
        if (!mbar_wait(smem_u32(&full_v[j % SV]), (uint32_t)(j / SV) & 1u, wc, 313)) break;
        tc_fence_after();
        const uint32_t vb = v_ring + (uint32_t)(j % SV) * TC_KV_BYTES;
        const uint32_t d = tmem + 128u + (uint32_t)g * 128u;
        const uint64_t ph = desc_k_sw128(p_base + (uint32_t)g * 2u * TC_P_BYTES), pl = desc_k_sw128(p_base + (uint32_t)g * 2u * TC_P_BYTES + TC_P_BYTES);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          const uint64_t vd = desc_mn_sw128(vb + ks * 2048u, p.v_lbo, p.v_sbo);
          umma(d, ph + (uint64_t)(ks * 2), vd, idesc_pv, (k == 0 && ks == 0) ? 0u : 1u);
          umma(d, pl + (uint64_t)(ks * 2), vd, idesc_pv, 1u);
        }
        umma_commit(smem_u32(&empty_v[j % SV]));
        umma_commit(smem_u32(&pv_done[g]));
      }
      if (*aborted) {                                // give-up path: see the MMAs already issued retire
        umma_commit(smem_u32(&drain_bar[1]));
        mbar_wait_drain(smem_u32(&drain_bar[1]), 0, 20000000ll);
      }
    }
  } else {
    // ---------------- softmax groups: thread <-> query row, group g takes tiles g, g+2, ... ----------------
    const int g = (warp - 2) >> 2;
    const int gt = (int)threadIdx.x - 64 - g * 128;           // thread index inside the group
    const int row = (warp & 3) * 32 + lane;                    // = TMEM lane
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const bool valid = row < nq;
    griddep_wait();
    griddep_launch();
    if (g == 0) {
      // stage this row of Q (zeros past the last node) in the swizzled K-major layout
      const uint4* src = reinterpret_cast<const uint4*>(p.q + ((qrow + (valid ? row : 0)) * p.H + h) * DH);
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        uint4 v = valid ? src[c] : make_uint4(0, 0, 0, 0);
        if (row < QROWS)
          *reinterpret_cast<uint4*>(smem_gen + (q_base - smem_base) + (uint32_t)(c >> 3) * QHALF + (uint32_t)row * 128u +
                                    (uint32_t)(((c & 7) ^ (row & 7)) << 4)) = v;
      }
      proxy_fence();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&q_ready));
    }
    uint64_t anc0 = 0, anc1 = 0, anc2 = 0;
    if (valid) { anc0 = p.anc[row * CERB_ANC_WORDS]; anc1 = p.anc[row * CERB_ANC_WORDS + 1]; anc2 = p.anc[row * CERB_ANC_WORDS + 2]; }
    const uint32_t s_addr = tmem + lane_base + (uint32_t)g * 64u;
    const uint32_t o_addr = tmem + lane_base + 128u + (uint32_t)g * 128u;
    uint8_t* ph = smem_gen + (p_base - smem_base) + (uint32_t)g * 2u * TC_P_BYTES + (uint32_t)row * 128u;
    uint8_t* pl = ph + TC_P_BYTES;
    float m_used = -INFINITY, l = 0.f;
    int k = 0;
    for (int i = g; i < T; i += 2, ++k) {
      mbar_wait(smem_u32(&s_full[g]), (uint32_t)k & 1u, wc, 314);
      tc_fence_after();
      float sc[64];
#pragma unroll
      for (int c0 = 0; c0 < 64; c0 += 16) tmem_ld16(s_addr + (uint32_t)c0, reinterpret_cast<uint32_t*>(sc + c0));
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&s_free[g]));       // S is in registers: its buffer may be overwritten
      const int key0 = (t0 + i) * TILE;
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
      if (key0 + TILE > L) {
        const uint64_t vm = tile_visibility(key0, L, anc0, anc1, anc2);
        const uint32_t vm_lo = (uint32_t)vm, vm_hi = (uint32_t)(vm >> 32);
#pragma unroll
        for (int j = 0; j < 64; ++j) {
          const bool vis = ((j < 32 ? vm_lo >> j : vm_hi >> (j - 32)) & 1u) != 0u;      // j is a constant after unrolling
          sc[j] = vis ? sc[j] * p.scale_log2 : -INFINITY;
          mx4[j & 3] = fmaxf(mx4[j & 3], sc[j]);
        }
      } else {
#pragma unroll
        for (int j = 0; j < 64; ++j) {
          sc[j] *= p.scale_log2;
          mx4[j & 3] = fmaxf(mx4[j & 3], sc[j]);
        }
      }
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      float alpha = 1.0f;
      bool rescale = false;
      if (m_used == -INFINITY) m_used = mx;                                   // nothing accumulated for this row yet
      else if (mx > m_used + TC_RESCALE) { alpha = ex2(m_used - mx); m_used = mx; rescale = true; }
      const float mu = m_used == -INFINITY ? 0.f : m_used;
      float rs4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int j = 0; j < 64; ++j) { sc[j] = ex2(sc[j] - mu); rs4[j & 3] += sc[j]; }
      l = l * alpha + ((rs4[0] + rs4[1]) + (rs4[2] + rs4[3]));
      if (k > 0) {
        mbar_wait(smem_u32(&pv_done[g]), (uint32_t)(k - 1) & 1u, wc, 315);   // P buffers free, O at rest
        tc_fence_after();
        if (__any_sync(0xffffffffu, rescale)) {
#pragma unroll 1
          for (int c0 = 0; c0 < DH; c0 += 32) {
            uint32_t r[32];
            tmem_ld16(o_addr + (uint32_t)c0, r);
            tmem_ld16(o_addr + (uint32_t)c0 + 16u, r + 16);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * alpha);
            tmem_st16(o_addr + (uint32_t)c0, r);
            tmem_st16(o_addr + (uint32_t)c0 + 16u, r + 16);
          }
          tmem_st_wait();
        }
      }
      if (key0 + TILE > kv_total) {
        // last, partial tile: rows past the end may hold anything (stale pool memory); zero V there so
        // that a zero probability times a non-finite value cannot poison the sum.  V travels apart
        // from K, so wait until it has landed.
        mbar_wait(smem_u32(&full_v[i % SV]), (uint32_t)(i / SV) & 1u, wc, 316);
        const int first_bad = kv_total - key0;
        uint8_t* vgen = smem_gen + (v_ring - smem_base) + (size_t)(i % SV) * TC_KV_BYTES;
        for (int idx = gt; idx < (TILE - first_bad) * 16; idx += 128) {
          const int r = first_bad + (idx >> 4), c = idx & 15;
          *reinterpret_cast<uint4*>(vgen + (size_t)(c >> 3) * 8192 + r * 128 + (c & 7) * 16) = make_uint4(0, 0, 0, 0);
        }
      }
      // probabilities as two bf16 terms, eight keys (16 bytes) per store
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        uint32_t hi[4], lo[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float p0 = sc[c * 8 + 2 * e], p1 = sc[c * 8 + 2 * e + 1];
          __nv_bfloat162 hb = __floats2bfloat162_rn(p0, p1);
          float2 hf = __bfloat1622float2(hb);
          hi[e] = *reinterpret_cast<uint32_t*>(&hb);
          lo[e] = pack_bf16(p0 - hf.x, p1 - hf.y);
        }
        const uint32_t off = (uint32_t)((c ^ (row & 7)) << 4);
        if (row < QROWS) {
          *reinterpret_cast<uint4*>(ph + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          *reinterpret_cast<uint4*>(pl + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
      }
      proxy_fence();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&p_ready[g]));
    }
    // ---- this group's (m, l, O) rows into shared memory ----
    if (k > 0) {
      mbar_wait(smem_u32(&pv_done[g]), (uint32_t)(k - 1) & 1u, wc, 317);
      tc_fence_after();
    }
    compute_bar(256);                               // every MMA has retired: all of shared memory can be reused
    {
      float* mr = mrg + ((size_t)g * 128 + row) * ROWF;
#pragma unroll 1
      for (int c0 = 0; c0 < DH; c0 += 32) {
        uint32_t r[32];
        if (k > 0) {
          tmem_ld16(o_addr + (uint32_t)c0, r);
          tmem_ld16(o_addr + (uint32_t)c0 + 16u, r + 16);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) r[j] = 0u;
        }
#pragma unroll
        for (int j = 0; j < 32; j += 4)
          *reinterpret_cast<float4*>(mr + c0 + j) = make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]),
                                                                __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
      }
      mr[DH] = m_used;
      mr[DH + 1] = l;
    }
    tc_fence_before();
    compute_bar(256);
    if (g == 0 && !p.cluster) {
      // merge the two groups' streams, row by row, into group 0's rows
      float* ra = mrg + (size_t)row * ROWF;
      const float* rb = mrg + ((size_t)128 + row) * ROWF;
      const float ma = ra[DH], mb = rb[DH];
      const float M = fmaxf(ma, mb), u = M == -INFINITY ? 0.f : M;
      const float wa = ex2(ma - u), wb = ex2(mb - u);
#pragma unroll 4
      for (int c = 0; c < DH; c += 4) {
        float4 a = *reinterpret_cast<float4*>(ra + c);
        const float4 bb = *reinterpret_cast<const float4*>(rb + c);
        a.x = a.x * wa + bb.x * wb; a.y = a.y * wa + bb.y * wb; a.z = a.z * wa + bb.z * wb; a.w = a.w * wa + bb.w * wb;
        *reinterpret_cast<float4*>(ra + c) = a;
      }
      ra[DH] = M;
      ra[DH + 1] = ra[DH + 1] * wa + rb[DH + 1] * wb;
    }
    compute_bar(256);

    // ---- output: final, or partial + fixed-order merge by the last CTA of this (sequence, head) ----
    const int ct = threadIdx.x - 64, nct = 256, RP = p.rows_pad;
    const float LN2 = 0.6931471805599453f;
    if (p.cluster) {
      // merged after the role branches, where every thread of the cluster meets
    } else if (p.nsplit == 1) {
      for (int idx = ct; idx < nq * (DH / 4); idx += nct) {
        const int r = idx / (DH / 4), c4 = idx % (DH / 4);
        const float inv = 1.0f / mrg[(size_t)r * ROWF + DH + 1];
        const float4 v = *reinterpret_cast<const float4*>(mrg + (size_t)r * ROWF + c4 * 4);
        *reinterpret_cast<uint2*>(p.out + ((qrow + r) * p.H + h) * DH + c4 * 4) =
            make_uint2(pack_bf16(v.x * inv, v.y * inv), pack_bf16(v.z * inv, v.w * inv));
      }
      if (p.lse)
        for (int r = ct; r < nq; r += nct)
          p.lse[((size_t)b * p.H + h) * p.n + r] = (mrg[(size_t)r * ROWF + DH] + log2f(mrg[(size_t)r * ROWF + DH + 1])) * LN2;
    } else {
      float* part = p.partial + (((size_t)b * p.H + h) * p.nsplit) * (size_t)(RP * ROWF);
      float* mine = part + (size_t)split * (RP * ROWF);
      for (int idx = ct; idx < nq * ROWF; idx += nct) __stcg(mine + idx, mrg[idx]);
      __threadfence();
      compute_bar(256);
      if (ct == 0) ticket_s = atomicAdd(&p.counters[b * p.H + h], 1u);
      compute_bar(256);
      if (ticket_s == (unsigned)p.nsplit - 1) {
        __threadfence();
        float* wts = mrg;                                   // [nsplit][RP]
        for (int r = ct; r < nq; r += nct) {
          float M = -INFINITY;
          for (int s2 = 0; s2 < p.nsplit; ++s2) M = fmaxf(M, __ldcg(part + (size_t)s2 * (RP * ROWF) + r * ROWF + DH));
          float Lsum = 0.f;
          for (int s2 = 0; s2 < p.nsplit; ++s2) {
            const float* pr = part + (size_t)s2 * (RP * ROWF) + r * ROWF;
            float w = exp2f(__ldcg(pr + DH) - M);
            wts[s2 * RP + r] = w;
            Lsum += __ldcg(pr + DH + 1) * w;
          }
          const float inv = 1.0f / Lsum;
          for (int s2 = 0; s2 < p.nsplit; ++s2) wts[s2 * RP + r] *= inv;
          if (p.lse) p.lse[((size_t)b * p.H + h) * p.n + r] = (M + log2f(Lsum)) * LN2;
        }
        compute_bar(256);
        for (int idx = ct; idx < nq * (DH / 4); idx += nct) {
          const int r = idx / (DH / 4), c4 = idx % (DH / 4);
          const float4* src = reinterpret_cast<const float4*>(part + (size_t)r * ROWF) + c4;
          float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
          for (int s2 = 0; s2 < p.nsplit; ++s2) {
            const float4 v = __ldcg(src + (size_t)s2 * (RP * ROWF / 4));
            const float w = wts[s2 * RP + r];
            acc.x += v.x * w; acc.y += v.y * w; acc.z += v.z * w; acc.w += v.w * w;
          }
          *reinterpret_cast<uint2*>(p.out + ((qrow + r) * p.H + h) * DH + c4 * 4) =
              make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
        }
        if (ct == 0) p.counters[b * p.H + h] = 0u;          // ready for the next launch
      }
    }
  }
  if (p.cluster) {
    // The splits of this (sequence, head) are the CTAs of one cluster (rank = split).  Each holds its merged
    // rows (O, m, l) in shared memory; once all have arrived, CTA r finishes rows r, r + nsplit, ...: it reads
    // those rows from every member in split order, weighs them and writes the final output.  Nobody leaves
    // before the second meeting, so no shared memory is read after its CTA has gone.
    cluster_start_wait();
    if (warp >= 2 && warp < 10) {
      cluster_meet(&cl_bar[0], p.nsplit, (int)threadIdx.x - 64, wc, 318);  // every member's rows are in place
      const int ct = threadIdx.x - 64;
      const float LN2 = 0.6931471805599453f;
      const uint32_t mine = smem_u32(smem_gen);
      const int c4 = ct & 31;
      for (int r = split + p.nsplit * (ct >> 5); r < nq; r += p.nsplit * 8) {
        const uint32_t row_off = (uint32_t)r * (ROWF * 4);
        // 2 * nsplit partial rows: the two softmax groups of every split, in (split, group) order
        constexpr uint32_t GROUP_OFF = 128u * ROWF * 4u;
        float M = -INFINITY;
        for (int s2 = 0; s2 < p.nsplit; ++s2) {
          const uint32_t base = mapa_u32(mine, (uint32_t)s2) + row_off + DH * 4;
          M = fmaxf(M, fmaxf(ld_cluster_f32(base), ld_cluster_f32(base + GROUP_OFF)));
        }
        const float u = M == -INFINITY ? 0.f : M;
        float Lsum = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s2 = 0; s2 < p.nsplit; ++s2) {
#pragma unroll
          for (int gg = 0; gg < 2; ++gg) {
            const uint32_t base = mapa_u32(mine, (uint32_t)s2) + row_off + (uint32_t)gg * GROUP_OFF;
            const float w = ex2(ld_cluster_f32(base + DH * 4) - u);
            Lsum += ld_cluster_f32(base + DH * 4 + 4) * w;
            const float4 v = ld_cluster_v4(base + (uint32_t)c4 * 16u);
            acc.x += v.x * w; acc.y += v.y * w; acc.z += v.z * w; acc.w += v.w * w;
          }
        }
        const float inv = 1.0f / Lsum;
        *reinterpret_cast<uint2*>(p.out + ((qrow + r) * p.H + h) * DH + c4 * 4) =
            make_uint2(pack_bf16(acc.x * inv, acc.y * inv), pack_bf16(acc.z * inv, acc.w * inv));
        if (c4 == 0 && p.lse) p.lse[((size_t)b * p.H + h) * p.n + r] = (M + log2f(Lsum)) * LN2;
      }
      compute_bar(256);                                                              // this CTA has read all it needs
      if (warp == 2) cluster_meet_before_exit(&cl_bar[1], p.nsplit, lane, wc, &exit_flag_s, 319);
    }
  }
  tc_fence_before();
  __syncthreads();                             // nobody exits before warp 2 has seen every member done
  if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
}

}  // namespace

#include "attention_kt.cuh"

// ---------------------------------------------------------------------------------------------
// fp32 path
// ---------------------------------------------------------------------------------------------
template <int DH>
__global__ void __launch_bounds__(128) tree_attn_f32_kernel(const float* __restrict__ q, const float* __restrict__ kpool,
                                                            const float* __restrict__ vpool,
                                                            const int32_t* __restrict__ page_table,
                                                            const int32_t* __restrict__ len,
                                                            const int32_t* __restrict__ n_active,
                                                            const uint64_t* __restrict__ anc, float* __restrict__ out,
                                                            float* __restrict__ lse, int n, int H, int max_pages,
                                                            float scale, const int32_t* __restrict__ row_off) {
  constexpr int E = DH / 32;
  __shared__ float s_o[4][DH];
  __shared__ float s_m[4], s_l[4];
  griddep_wait();
  griddep_launch();
  const int i = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int nq = n_active ? min(n_active[b], n) : n;
  if (i >= nq) return;
  const int L = len[b], warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint64_t a0 = anc[i * CERB_ANC_WORDS], a1 = anc[i * CERB_ANC_WORDS + 1], a2 = anc[i * CERB_ANC_WORDS + 2];
  float qv[E], acc[E];
  const size_t qrow = row_off ? (size_t)row_off[b] : (size_t)b * n;
  const float* qp = q + ((qrow + i) * H + h) * DH;
  for (int e = 0; e < E; ++e) { qv[e] = qp[lane + 32 * e]; acc[e] = 0.f; }
  float m = -INFINITY, l = 0.f;
  for (int kpos = warp; kpos < L + nq; kpos += 4) {
    if (kpos >= L) {
      int j = kpos - L;
      if (!(((j < 64 ? a0 : j < 128 ? a1 : a2) >> (j & 63)) & 1ull)) continue;
    }
    int page = page_table[(size_t)b * max_pages + kpos / CERB_PAGE];
    size_t off = (((size_t)page * H + h) * CERB_PAGE + kpos % CERB_PAGE) * DH;
    float s = 0.f;
    for (int e = 0; e < E; ++e) s += qv[e] * kpool[off + lane + 32 * e];
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    s *= scale;
    float mn = fmaxf(m, s), al = expf(m - mn), pw = expf(s - mn);
    l = l * al + pw;
    for (int e = 0; e < E; ++e) acc[e] = acc[e] * al + pw * vpool[off + lane + 32 * e];
    m = mn;
  }
  for (int e = 0; e < E; ++e) s_o[warp][lane + 32 * e] = acc[e];
  if (lane == 0) { s_m[warp] = m; s_l[warp] = l; }
  __syncthreads();
  float M = fmaxf(fmaxf(s_m[0], s_m[1]), fmaxf(s_m[2], s_m[3]));
  float Ls = 0.f;
  for (int w = 0; w < 4; ++w) Ls += s_m[w] == -INFINITY ? 0.f : s_l[w] * expf(s_m[w] - M);
  for (int c = threadIdx.x; c < DH; c += 128) {
    float a = 0.f;
    for (int w = 0; w < 4; ++w) a += s_m[w] == -INFINITY ? 0.f : s_o[w][c] * expf(s_m[w] - M);
    out[((qrow + i) * H + h) * DH + c] = a / Ls;
  }
  if (threadIdx.x == 0 && lse) lse[((size_t)b * H + h) * n + i] = M + logf(Ls);
}

// A split reads `per` tiles of 64 keys and writes an n-row fp32 partial, so wide trees get fewer,
// longer splits: at least n/8 tiles each keeps the partial traffic near one eighth of the K/V read.
int plan_nsplit(int B, int H, int n, int max_len, int target_ctas, bool one_wave = false, int max_split = kMaxSplit) {
  int tiles = (max_len + TILE - 1) / TILE;
  if (tiles < 1) tiles = 1;
  // the tensor-core kernel holds an SM by itself: its CTAs must fit in one wave, so round down for it
  int want = one_wave ? target_ctas / (B * H) : (target_ctas + B * H - 1) / (B * H);
  int min_tiles = n / 8 > 1 ? n / 8 : 1;
  if (want > tiles / min_tiles) want = tiles / min_tiles;
  if (want > max_split) want = max_split;
  if (want > tiles) want = tiles;
  if (want < 1) want = 1;
  int per = (tiles + want - 1) / want;
  if (per * PAGES_PER_TILE > kMaxPagesPerCta) return -1;       // more than 16K keys per split
  return (tiles + per - 1) / per;
}

inline int nq_pad(int n) { return n <= 16 ? 16 : n <= 32 ? 32 : n <= 64 ? 64 : 128; }

template <int DH, int WQ, int WK, int STAGES>
int launch_cfg(const AttnParams& p, const CUtensorMap* tmK, const CUtensorMap* tmV, int B, cudaStream_t st) {
  constexpr size_t smem = (size_t)STAGES * 2 * (DH / 64) * TILE * 128 + 1024;
  static bool configured = false;
  if (!configured) {
    CERB_CUDA_OK(cudaFuncSetAttribute(tree_attn_bf16_kernel<DH, WQ, WK, STAGES>,
                                      cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    configured = true;
  }
  dim3 grid(p.nsplit, p.H, B);
  if (p.cluster)
    return launch_pdl_cluster(tree_attn_bf16_kernel<DH, WQ, WK, STAGES>, grid, dim3((WQ * WK + 1) * 32), smem, st, (unsigned)p.nsplit,
                              *tmK, *tmV, p) == cudaSuccess ? CERB_OK : CERB_E_CUDA;
  if (launch_pdl(tree_attn_bf16_kernel<DH, WQ, WK, STAGES>, grid, dim3((WQ * WK + 1) * 32), smem, st, *tmK, *tmV, p) != cudaSuccess)
    return CERB_E_CUDA;
  return CERB_OK;
}

}  // namespace

size_t attn_scratch_bytes(int B, int n, int H, int Dh) {
  size_t rows = (size_t)(kTargetCtas + B * H + kMaxSplit);
  return kCounterBytes + rows * (size_t)nq_pad(n) * (size_t)(Dh + 4) * sizeof(float);
}

constexpr int kAttnRowsPerLaunch = 128;

// One launch of the bf16 kernels over query rows row0 .. row0 + rows - 1 (rows <= 128) of every sequence's tree.
static int launch_attn_window(const cerb_attn_args* a, int row0, int rows, const CUtensorMap* tmK, const CUtensorMap* tmV,
                              int32_t* status, cudaStream_t st, const int32_t* row_off) {
  AttnParams p;
  const size_t row_elems = (size_t)a->n_heads * a->head_dim;
  p.q = (const bf16*)a->q + (size_t)row0 * row_elems;
  p.page_table = a->page_table;
  p.len = a->len;
  p.n_active = a->n_active;
  p.anc = a->anc + (size_t)row0 * CERB_ANC_WORDS;
  p.row_off = row_off;
  p.out = (bf16*)a->out + (size_t)row0 * row_elems;
  p.lse = a->lse ? a->lse + row0 : nullptr;
  p.row0 = row0;
  p.rows = rows;
  p.counters = (unsigned int*)a->scratch;
  p.partial = (float*)((char*)a->scratch + kCounterBytes);
  p.status = status;
  p.wait_cycles = wait_cycles();
  p.n = a->n;
  p.H = a->n_heads;
  p.max_pages = a->max_pages;
  // Which kernel: windows of 65 .. 128 rows take the tcgen05 kernel whose MMAs are 128 query rows tall; 17 .. 64 rows
  // the keys-on-M kernel (below); up to 16 rows and one-node steps the warp-MMA kernel, whose 16-row layout wastes
  // no tensor work and streams at 7.0 TB/s at batch 16 x 8K keys.  Short caches and head_dim 64 stay on the
  // warp-MMA kernel too.  CERB_ATTN_TC=0 / 1 forces the warp-MMA / the query-rows-on-M tcgen05 kernel (tests).
  static const int force_tc = getenv("CERB_ATTN_TC") ? atoi(getenv("CERB_ATTN_TC")) : -1;
  const int np_ = nq_pad(rows);
  const bool auto_tc = np_ == 128;
  const bool tensor_path = a->head_dim == 128 && (force_tc < 0 ? auto_tc : force_tc != 0);
  // With clusters the splits of a (sequence, head) merge through distributed shared memory: at most 8 of them
  // (the portable cluster size).  CERB_ATTN_CLUSTER=0 keeps the merge through global partials (up to 32 splits).
  static const int use_cluster = getenv("CERB_ATTN_CLUSTER") ? atoi(getenv("CERB_ATTN_CLUSTER")) : 1;
  // CTAs that fit at once: one per SM for the tensor-core kernel and for the warp-MMA layouts of 32 rows and more
  // (288 threads x 168 registers), two per SM for the 16-row layout (160 threads); the grid is planned to fit one wave
  const int resident = (tensor_path || np_ > 16) ? 148 : kTargetCtas;
  p.nsplit = plan_nsplit(a->B, a->n_heads, nq_pad(rows), a->max_len, resident, true, use_cluster ? 8 : kMaxSplit);
  if (p.nsplit < 1) return CERB_E_SHAPE;
  p.oob_row = a->n_pool_pages * a->n_heads * CERB_PAGE;
  p.scale_log2 = a->scale * 1.4426950408889634f;
  p.rows_pad = nq_pad(rows);
  p.cluster = (use_cluster && p.nsplit >= 2 && p.nsplit <= 8) ? 1 : 0;
  // V tile in shared memory: [half of head_dim][64 keys][128 bytes]; 8-key groups are 1024 bytes apart
  p.v_lbo = 8192u;
  p.v_sbo = 1024u;
  int np = nq_pad(rows), rc = CERB_E_SHAPE;
  // The keys-on-M tensor-core kernel (attention_kt.cuh; 128-key tiles, every MMA row in use whatever the tree's
  // width) takes the trees of 17 to 64 nodes.  Measured inside the 7B decoding step, batch 1, 2K keys, this kernel
  // against the others: 64-node steps 4.33 / 4.47 ms, one-node steps 3.39 / 3.27 ms (the 16-row warp-MMA layout has
  // less to set up); alone at batch 16 x 8K keys: 64 nodes 403 / 537 us, 16 nodes 392 / 308 us, 128 nodes (its
  // 128-query form, not built any more) 654 / 572 us.  CERB_ATTN_KT=0 / 1 keeps it off / uses it for every launch of
  // up to 64 rows (tests).
  static const int force_kt = getenv("CERB_ATTN_KT") ? atoi(getenv("CERB_ATTN_KT")) : -1;
  const bool kt_path = a->head_dim == 128 && force_tc < 0 && rows <= 64 && (force_kt < 0 ? rows > 16 : force_kt != 0);
  if (kt_path) {
    const int tiles = (a->max_len + KT_TILE - 1) / KT_TILE;
    int want = 148 / (a->B * a->n_heads);
    const int max_split = use_cluster ? 8 : kMaxSplit;
    if (want > max_split) want = max_split;
    if (want > tiles) want = tiles;
    if (want < 1) want = 1;
    const int per = (tiles + want - 1) / want;
    if (per * KT_PAGES > kMaxPagesPerCta) return CERB_E_SHAPE;
    p.nsplit = (tiles + per - 1) / per;
    p.cluster = (use_cluster && p.nsplit >= 2 && p.nsplit <= 8) ? 1 : 0;
    constexpr int ncb = 2;             // two blocks of 32 queries: the MMAs are 64 queries wide
    static bool kt_configured = false;
    if (!kt_configured) {
      CERB_CUDA_OK(cudaFuncSetAttribute(tree_attn_kt_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kt_smem(2)));
      kt_configured = true;
    }
    auto kern = tree_attn_kt_kernel<2>;
    const dim3 grid(p.nsplit, p.H, a->B), block(kt_threads(ncb));
    if (p.cluster)
      rc = launch_pdl_cluster(kern, grid, block, kt_smem(ncb), st, (unsigned)p.nsplit, *tmK, *tmV, p) == cudaSuccess ? CERB_OK : CERB_E_CUDA;
    else
      rc = launch_pdl(kern, grid, block, kt_smem(ncb), st, *tmK, *tmV, p) == cudaSuccess ? CERB_OK : CERB_E_CUDA;
  } else if (tensor_path) {
    static bool configured = false;
    if (!configured) {
      CERB_CUDA_OK(cudaFuncSetAttribute(tree_attn_tc_kernel<2, 5, 128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc_smem(2, 5, 128)));
      CERB_CUDA_OK(cudaFuncSetAttribute(tree_attn_tc_kernel<5, 5, 64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc_smem(5, 5, 64)));
      configured = true;
    }
    auto kern = rows <= 64 ? tree_attn_tc_kernel<5, 5, 64, true> : tree_attn_tc_kernel<2, 5, 128, false>;
    const size_t TC_SMEM = rows <= 64 ? tc_smem(5, 5, 64) : tc_smem(2, 5, 128);
    if (p.cluster)
      rc = launch_pdl_cluster(kern, dim3(p.nsplit, p.H, a->B), dim3(TC_THREADS), TC_SMEM, st, (unsigned)p.nsplit,
                              *tmK, *tmV, p) == cudaSuccess ? CERB_OK : CERB_E_CUDA;
    else
      rc = launch_pdl(kern, dim3(p.nsplit, p.H, a->B), dim3(TC_THREADS), TC_SMEM, st, *tmK, *tmV, p) == cudaSuccess
               ? CERB_OK : CERB_E_CUDA;
  } else if (a->head_dim == 128) {
    if (np == 16) rc = launch_cfg<128, 1, 4, 3>(p, tmK, tmV, a->B, st);
    else if (np == 32) rc = launch_cfg<128, 2, 4, 3>(p, tmK, tmV, a->B, st);
    else if (np == 64) rc = launch_cfg<128, 4, 2, 3>(p, tmK, tmV, a->B, st);
    else rc = launch_cfg<128, 8, 1, 3>(p, tmK, tmV, a->B, st);
  } else if (a->head_dim == 64) {
    if (np == 16) rc = launch_cfg<64, 1, 4, 4>(p, tmK, tmV, a->B, st);
    else if (np == 32) rc = launch_cfg<64, 2, 4, 4>(p, tmK, tmV, a->B, st);
    else if (np == 64) rc = launch_cfg<64, 4, 2, 4>(p, tmK, tmV, a->B, st);
    else rc = launch_cfg<64, 8, 1, 4>(p, tmK, tmV, a->B, st);
  }
  return rc;
}

int launch_tree_attention(cerb_ctx* c, const cerb_attn_args* a, const CUtensorMap* tmK, const CUtensorMap* tmV,
                          int sm_count, int32_t* status, cudaStream_t st, const int32_t* row_off) {
  (void)sm_count;
  if (a->dtype == CERB_F32) {
    dim3 grid(a->n, a->n_heads, a->B);
    if (a->head_dim == 64)
      tree_attn_f32_kernel<64><<<grid, 128, 0, st>>>((const float*)a->q, (const float*)a->k_pool, (const float*)a->v_pool,
                                                     a->page_table, a->len, a->n_active, a->anc, (float*)a->out, a->lse,
                                                     a->n, a->n_heads, a->max_pages, a->scale, row_off);
    else if (a->head_dim == 128)
      tree_attn_f32_kernel<128><<<grid, 128, 0, st>>>((const float*)a->q, (const float*)a->k_pool, (const float*)a->v_pool,
                                                      a->page_table, a->len, a->n_active, a->anc, (float*)a->out, a->lse,
                                                      a->n, a->n_heads, a->max_pages, a->scale, row_off);
    else
      return CERB_E_SHAPE;
    CERB_LAUNCH_CHECK(c);
    return CERB_OK;
  }
  if (a->B * a->n_heads > (int)(kCounterBytes / sizeof(unsigned int)) - 4) return CERB_E_SHAPE;   // last 16 bytes: status word
  if (a->scratch_bytes < attn_scratch_bytes(a->B, a->n, a->n_heads, a->head_dim)) return CERB_E_NOMEM;
  // A CTA holds at most 128 query rows (the tensor-core MMA's height, eight 16-row warps in the warp-MMA kernel).
  // A wider tree (Sec. 5.1 goes up to 150 candidates + the root) takes one launch per window of 128 rows; the
  // launches are stream-ordered and share the scratch.  Keys are not windowed: rows of the second window see the
  // whole tree, rows of the first only nodes below 128 (an ancestor has a lower index than its descendant).
  for (int row0 = 0; row0 < a->n; row0 += kAttnRowsPerLaunch) {
    const int rows = a->n - row0 < kAttnRowsPerLaunch ? a->n - row0 : kAttnRowsPerLaunch;
    CERB_TRY(launch_attn_window(a, row0, rows, tmK, tmV, status, st, row_off));
    CERB_LAUNCH_CHECK(c);
  }
  return CERB_OK;
}

}  // namespace cerb

// ---------------------------------------------------------------------------------------------
// Tree attention for callers that cannot allocate device memory
// ---------------------------------------------------------------------------------------------
// The split-KV partials and ticket counters normally live in a scratch buffer the caller allocates.
// Some callers cannot do that: code running inside a memory-pool or allocator callback, a plug-in
// that is handed fixed buffers by its host application, or a process whose device-memory budget was
// fixed at start-up.  For them the scratch lives in this library's image instead, as one static
// device array.  Every GPU that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_attn_scratch[CERB_STATIC_ATTN_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::atomic<void*> g_static_scratch_addr[kMaxDevices];      // device address of the array, per device, once known

// Set-up, once per device, with that device current.  In host code the array's name is only a handle; the
// address a kernel can use has to be asked for.  Two threads racing here both get the same answer from the
// runtime, so the slot is simply an atomic pointer.
int static_scratch(void** out) {
  int dev = -1;
  CERB_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return CERB_E_SHAPE;
  void* ptr = g_static_scratch_addr[dev].load(std::memory_order_acquire);
  if (!ptr) {
    if (cudaGetSymbolAddress(&ptr, g_static_attn_scratch) != cudaSuccess || !ptr) return CERB_E_CUDA;
    g_static_scratch_addr[dev].store(ptr, std::memory_order_release);
  }
  *out = ptr;
  return CERB_OK;
}
}  // namespace

extern "C" int cerb_tree_attention_noalloc(const cerb_attn_args* a, void* stream) {
  using namespace cerb;
  if (!a || !a->q || !a->k_pool || !a->v_pool || !a->page_table || !a->len || !a->anc || !a->out) return CERB_E_ARG;
  if (a->B < 1 || a->n < 1 || a->n > CERB_MAX_NODES || a->n_heads < 1 || a->n_pool_pages < 1) return CERB_E_ARG;
  if (a->dtype != CERB_BF16) return CERB_E_ARG;
  if (a->head_dim != 64 && a->head_dim != 128) return CERB_E_SHAPE;
  const size_t need = attn_scratch_bytes(a->B, a->n, a->n_heads, a->head_dim);
  if (need > (size_t)CERB_STATIC_ATTN_SCRATCH_BYTES) return CERB_E_NOMEM;     // problem too large for the built-in scratch
  void* scratch = nullptr;
  CERB_TRY(static_scratch(&scratch));
  cudaStream_t st = (cudaStream_t)stream;
  // The array keeps whatever the previous call left.  The ticket counters must start at zero; the partials behind
  // them are fully rewritten before being read.  The status words (the last 16 bytes of the first 4 KB) are NOT
  // cleared here: a time-out stays visible until cerb_tree_attention_noalloc_status has read it.
  CERB_CUDA_OK(cudaMemsetAsync(scratch, 0, kCounterBytes - 16, st));
  CUtensorMap tk, tv;
  CERB_TRY(make_pool_map(&tk, a->k_pool, a->n_pool_pages, a->n_heads, a->head_dim));
  CERB_TRY(make_pool_map(&tv, a->v_pool, a->n_pool_pages, a->n_heads, a->head_dim));
  cerb_attn_args b = *a;
  b.scratch = scratch;
  b.scratch_bytes = CERB_STATIC_ATTN_SCRATCH_BYTES;
  int32_t* status = reinterpret_cast<int32_t*>((char*)scratch + kCounterBytes - 16);
  return launch_tree_attention(nullptr, &b, &tk, &tv, 148, status, st);
}

extern "C" int cerb_tree_attention_noalloc_status(void* stream) {
  using namespace cerb;
  void* scratch = nullptr;
  CERB_TRY(static_scratch(&scratch));
  CERB_CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
  int32_t words[4] = {0, 0, 0, 0};
  CERB_CUDA_OK(cudaMemcpy(words, (char*)scratch + kCounterBytes - 16, sizeof(words), cudaMemcpyDeviceToHost));
  if (words[0] != 0) CERB_CUDA_OK(cudaMemset((char*)scratch + kCounterBytes - 16, 0, 16));
  return words[0];
}
