// Tree-verification attention with the KEYS on the tensor core's M side (head_dim 128, bf16).
//
// A verification step has few queries (tree nodes) and many keys, so the products are taken transposed:
//
//   S^T[128 keys x N queries]   = K_tile[128 x 128] . Q^T          (A = K tile as TMA delivers it, B = Q)
//   O^T[128 dh   x N queries]  += V_tile^T[128 dh x 128 keys] . P^T (A = V tile, read M-major; B = P^T in shared memory)
//
// with N = 64 (trees of up to 64 nodes) or 128 query columns.  Every one of the 128 accumulator lanes is a key
// (for S^T) or a head-dim element (for O^T), so no tensor-core row is wasted on a narrow tree, a tile is 128
// keys (half as many MMAs, barriers and tensor-memory round trips per key as with 64-key tiles), and the
// element-wise work of a tile is spread over 128 x N/32 threads: thread (key lane, block of 32 queries).
//
// Softmax.  Thread = key means a row maximum would be a reduction across threads, so none is taken per tile:
// every query keeps a reference exponent m[q] in shared memory and p = 2^(s - m[q]) is used as long as no
// visible score of the tile exceeds m[q] by more than 2^30 (fp32 and the two-term bf16 split of p have the
// exponent range for that); only when one does (the first visible key always does: m[q] starts at -1e30) the
// four warps that share the query block agree (one named barrier per tile) to raise m[q] to the largest score
// seen, rescale those columns of O^T and their running sums, and take the tile's scores again.  The result after the final normalisation is exact for any reference.
// Row sums l[q] accumulate per thread (one partial per key lane) and are added once, at the end.
//
// Probabilities enter the tensor core as two bf16 terms, p = p_hi + p_lo (about 16 significant bits).  The two
// terms sit side by side along N in shared memory, so one MMA of N = 2 x N_queries per 16 keys produces
// O^T_hi | O^T_lo in neighbouring accumulator columns, added when the accumulator is read out: the second term
// costs no extra instruction issue (issuing, not multiplying, is what limits MMAs this small).
//
// Roles: warps 0 .. 4 N/32 - 1 = softmax (warp & 3 = lane quarter, warp / 4 = query block); then the TMA producer
// warps (one ring of 32 KB units, K and V tiles alternating; a K unit is free again as soon as its QK^T MMAs
// have retired, a V unit after its PV MMAs); then the tensor-memory allocator and QK^T issuer; then the PV
// issuer.  A tile of one head arrives as 32 boxes of 2 KB (a 16-token page is 16 rows of two 128-byte swizzle
// rows), and issuing one such copy occupies its thread for ~90 cycles (measured: a unit of 16 boxes issued by
// 16 lanes of one warp takes 1400 cycles, which alone would cap an SM at 64 KB per 2800 cycles), so several
// warps issue the boxes of a unit side by side.
// S^T is double-buffered in tensor memory so that QK^T of the next tile runs during the softmax of this one.
// Split-KV, the cluster merge through distributed shared memory, bounded waits and the pre-wait set-up are the
// same as in the other bf16 kernels of this file.
#pragma once

namespace {

constexpr int KT_TILE = 128;                       // keys per tile = the MMA's M
constexpr int KT_PAGES = KT_TILE / CERB_PAGE;      // 8 pages per tile
constexpr uint32_t KT_UNIT = 32768;                // K (or V) of one tile: [2 halves of head_dim][128 keys][128 bytes]
constexpr uint32_t KT_HALF = 16384;
constexpr int KT_DH = 128, KT_ROWF = KT_DH + 4;
// log2 of the excess over the reference that forces a new reference.  Everything downstream is relative (the
// exponential, the two-term bf16 split, the fp32 sums), so the bound only has to keep 2^30 x (keys per split) x |v|
// far inside the fp32 range.
constexpr float KT_RAISE = 30.0f;
constexpr float KT_UNSET = -1.0e30f;               // reference of a query that has seen no key yet: any real score exceeds it

__host__ __device__ constexpr int kt_nq(int ncb) { return ncb <= 2 ? 64 : 128; }           // query columns of the MMAs
__host__ __device__ constexpr int kt_units(int ncb) { return ncb <= 2 ? 4 : 3; }           // ring depth in 32 KB units
__host__ __device__ constexpr int kt_pbufs(int ncb) { return ncb <= 2 ? 2 : 1; }           // P^T buffers
__host__ __device__ constexpr int kt_producers(int ncb) { return ncb <= 2 ? 4 : 2; }      // TMA-issuing warps
__host__ __device__ constexpr int kt_threads(int ncb) { return 128 * ncb + 32 * (kt_producers(ncb) + 2); }
__host__ __device__ constexpr size_t kt_smem(int ncb) {
  // P^T (hi | lo), Q, ring, alignment slack
  return (size_t)kt_pbufs(ncb) * 2 * kt_nq(ncb) * 256 + (size_t)kt_nq(ncb) * 256 + (size_t)kt_units(ncb) * KT_UNIT + 1024;
}

// Order-preserving map float -> int (for integer atomicMax on floats) and back.
__device__ __forceinline__ int f2ord(float f) {
  const int i = __float_as_int(f);
  return i >= 0 ? i : i ^ 0x7fffffff;
}
__device__ __forceinline__ float ord2f(int i) { return __int_as_float(i >= 0 ? i : i ^ 0x7fffffff); }

template <int NCB>
__global__ void __launch_bounds__(kt_threads(NCB), 1) tree_attn_kt_kernel(const __grid_constant__ CUtensorMap tmK,
                                                                          const __grid_constant__ CUtensorMap tmV,
                                                                          const AttnParams p) {
  constexpr int DH = KT_DH, ROWF = KT_ROWF;
  constexpr int NQ = kt_nq(NCB);                   // query columns of S^T; O^T has 2 * NQ (hi | lo)
  constexpr int NU = kt_units(NCB);
  constexpr int PB = kt_pbufs(NCB);                // P^T buffers: with two, the stores of tile t need not wait for PV of tile t - 1
  constexpr int NSW = 4 * NCB;                     // softmax warps
  constexpr int NPROD = kt_producers(NCB);         // producer warps NSW .. NSW + NPROD - 1; then QK^T issuer, PV issuer
  constexpr int W_QK = NSW + NPROD, W_PV = W_QK + 1;
  constexpr uint32_t QHALF = (uint32_t)NQ * 128u;
  constexpr uint32_t P_TERM = (uint32_t)(NQ / 64) * KT_HALF;        // bytes of one term (hi or lo) of P^T
  constexpr uint32_t TMEM_COLS = NQ == 64 ? 256u : 512u;           // S^T x 2 buffers, then O^T hi | lo
  constexpr uint32_t O_COL = 2u * NQ;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_u[2][NU], empty_u[NU], s_full[2], s_free[2], p_ready[PB], pv_done[PB], q_ready, drain_bar[2];
  __shared__ __align__(8) uint64_t cl_bar[2];
  __shared__ int page_list[kMaxPagesPerCta];
  __shared__ uint32_t desc_t[CERB_MAX_NODES][4];   // per tree key: which queries of this launch see it, 32 per word
  __shared__ __align__(16) float m_ref[128];       // reference exponent per query (KT_UNSET until a key is seen)
  __shared__ int m_pending[128];                   // largest visible score reported since the last raise (ordered int)
  __shared__ int raise_at[2][4];                   // [tile parity][query block]: 1 + the last tile at which a raise was requested
  __shared__ float l_part[4][128];                 // per lane quarter: partial row sums, added at the end
  __shared__ uint32_t tmem_slot;
  __shared__ int aborted_s, exit_flag_s;
  __shared__ unsigned int ticket_s;
  volatile int* aborted = &aborted_s;
  const WaitCtx wc{p.wait_cycles, aborted, p.status};

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t p_base = smem_base;                                 // [buffer][hi, lo][64-query block][128 keys][128 B]
  const uint32_t q_base = p_base + PB * 2 * P_TERM;                       // [half of head_dim][NQ rows][128 B]
  const uint32_t ring = q_base + 2 * QHALF;                          // NU units
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  // Lengths, live node counts, the page table, the tree and the prefix keys are at least two kernels old:
  // everything up to the first use of Q or of this step's tree keys runs before griddep_wait().
  const int L = p.len[b];
  const int nq_all = p.n_active ? min(p.n_active[b], p.n) : p.n;      // live nodes of this sequence
  const size_t qrow = p.row_off ? (size_t)p.row_off[b] : (size_t)b * p.n;   // this sequence's first row of q and out
  const int nq = min(nq_all - p.row0, p.rows);                        // live query rows of this launch
  if (nq <= 0) return;                                                // (uniform over a cluster)
  const int n_tree = min(nq_all, p.row0 + p.rows);                    // tree keys these rows can see
  const int kv_total = L + n_tree;
  const int tiles = (kv_total + KT_TILE - 1) / KT_TILE;
  const int per = (tiles + p.nsplit - 1) / p.nsplit;
  const int t0 = min(tiles, split * per), t1 = min(tiles, t0 + per);
  const bool too_long = per * KT_PAGES > kMaxPagesPerCta;
  const int T = too_long ? 0 : t1 - t0;

  if (threadIdx.x == 0) {
    aborted_s = (*p.status != 0);
    exit_flag_s = 0;
    for (int s = 0; s < NU; ++s) {
      mbar_init(smem_u32(&full_u[0][s]), NPROD);
      mbar_init(smem_u32(&full_u[1][s]), NPROD);
      mbar_init(smem_u32(&empty_u[s]), 1);
    }
    for (int g = 0; g < 2; ++g) {
      mbar_init(smem_u32(&s_full[g]), 1);
      mbar_init(smem_u32(&s_free[g]), NSW);
    }
    for (int g = 0; g < PB; ++g) {
      mbar_init(smem_u32(&p_ready[g]), NSW);
      mbar_init(smem_u32(&pv_done[g]), 1);
    }
    mbar_init(smem_u32(&q_ready), NSW);
    mbar_init(smem_u32(&drain_bar[0]), 1);
    mbar_init(smem_u32(&drain_bar[1]), 1);
    mbar_init(smem_u32(&cl_bar[0]), (uint32_t)p.nsplit);
    mbar_init(smem_u32(&cl_bar[1]), (uint32_t)p.nsplit);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (too_long) atomicExch(p.status, CERB_E_SHAPE);
  }
  // queries that do not exist keep reference 0: their score columns are zero and never ask for a new one
  if (threadIdx.x < 128) { m_ref[threadIdx.x] = (int)threadIdx.x < nq ? KT_UNSET : 0.f; m_pending[threadIdx.x] = f2ord(-INFINITY); }
  if (threadIdx.x < 8) raise_at[threadIdx.x >> 2][threadIdx.x & 3] = 0;
  if (warp == W_QK) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (p.cluster) cluster_start_arrive();
  const uint32_t tmem = tmem_slot;                   // columns [0, 2 NQ): S^T buffers 0 / 1; [2 NQ, 4 NQ): O^T hi | lo
  float* mrg = reinterpret_cast<float*>(smem_gen);   // [NQ][ROWF] over the operand buffers, once the key loop is over

  // Waiting for unit u (K units are even, V units odd) to have landed.  A parity wait only tells "the phase before
  // the current one is complete", so every barrier needs ONE waiter that sees each of its phases in turn.  With
  // an odd ring depth a slot holds K and V units alternately, and a K consumer looking at every other phase of a
  // shared barrier returned at once when its wait began before the V unit in between had landed (a rare
  // dead-lock, measured).  Hence one "landed" barrier per slot and per kind of unit: full_u[kind][slot], whose
  // phases the one consumer of that kind sees in order.
  auto unit_parity = [](int u) { return (uint32_t)((NU & 1) ? (u / NU) >> 1 : u / NU) & 1u; };
  auto wait_unit = [&](int u, int site) { return mbar_wait(smem_u32(&full_u[u & 1][u % NU]), unit_parity(u), wc, site); };
  if (warp >= NSW && warp < NSW + NPROD) {
    // ---------------- TMA producers ----------------
    // producer w issues boxes w, w + NPROD, ... of every unit (box = page * 2 + half of head_dim), one per lane
    const int pw = warp - NSW;
    constexpr int BOXES = 16 / NPROD;                // boxes of a unit per producer warp
    const int32_t* pt = p.page_table + (size_t)b * p.max_pages;
    const int n_pages = T * KT_PAGES;
    if (pw == 0)
      for (int i = lane; i < n_pages; i += 32) {
        const int lp = t0 * KT_PAGES + i;
        page_list[i] = (lp * CERB_PAGE < kv_total && lp < p.max_pages) ? (pt[lp] * p.H + h) * CERB_PAGE : p.oob_row;
      }
    asm volatile("bar.sync 3, %0;" ::"r"(32 * NPROD) : "memory");      // the page list is complete
    // units (K and V) of tiles that lie wholly inside the prefix may be fetched before the wait
    int early = 0;
    while (early < T && 2 * early < NU && (t0 + early + 1) * KT_TILE <= L) ++early;
    const int early_units = min(2 * early, NU);
    static_assert(KT_PAGES == 8, "the lane -> box map below assumes eight pages per tile");
    const int box = pw + NPROD * lane;               // lanes 0 .. BOXES-1
    const int pg = box >> 1, hf = box & 1;
    const uint64_t pol = l2_policy(true);            // K/V are read once per step
    int issued = 0;
    // (the abort flag itself is looked at once, for a launch that starts after a time-out: nothing is issued then;
    // later a wait that gives up says so in its return value, which costs the loop nothing)
    const int u_stop = *aborted ? 0 : 2 * T;
    for (int u = 0; u < u_stop; ++u) {
      if (u == early_units) { griddep_wait(); griddep_launch(); }
      const int slot = u % NU, t = u >> 1;
      const uint32_t fb = smem_u32(&full_u[u & 1][slot]);
      int stop = 0;
      if (lane == 0) {
        stop = !mbar_wait_polite(smem_u32(&empty_u[slot]), ((uint32_t)(u / NU) & 1u) ^ 1u, wc, 101);
        if (!stop) mbar_expect_tx(fb, KT_UNIT / NPROD);
      }
      if (__shfl_sync(0xffffffffu, stop, 0)) break;            // this wait ran out (the consumers have stopped): issue nothing more
      if (lane < BOXES) {
        const int row = page_list[t * KT_PAGES + pg];          // out-of-range rows are zero-filled by TMA
        const uint32_t dst = ring + (uint32_t)slot * KT_UNIT + (uint32_t)hf * KT_HALF + (uint32_t)pg * (CERB_PAGE * 128);
        tma_load_2d_hint(dst, (u & 1) ? &tmV : &tmK, hf * 64, row, fb, pol);
      }
      issued = u + 1;
    }
    if (lane == 0 && *aborted) {
      // give-up path: the copies this warp has issued still land in the CTA's shared memory; see them in (the
      // phase also needs the other producers' shares, hence a limit of its own: 10 ms)
      for (int u = issued > NU ? issued - NU : 0; u < issued; ++u)
        mbar_wait_drain(smem_u32(&full_u[u & 1][u % NU]), unit_parity(u), 20000000ll);
    }
    griddep_wait();      // (a lane that has waited already returns at once)
    griddep_launch();
  } else if (warp == W_QK) {
    griddep_wait();
    griddep_launch();
    // ---------------- QK^T issuer ----------------
    if (lane == 0 && T > 0) {
      constexpr uint32_t idesc_s = idesc_bf16(128, NQ, false, false);
      const uint64_t q_desc0 = desc_k_sw128(q_base), q_desc1 = desc_k_sw128(q_base + QHALF);
      mbar_wait(smem_u32(&q_ready), 0, wc, 102);
      const int t_stop = *aborted ? 0 : T;
      for (int t = 0; t < t_stop; ++t) {
        const int u = 2 * t, slot = u % NU, sb = t & 1;
        if (!wait_unit(u, 103)) break;
        if (!mbar_wait(smem_u32(&s_free[sb]), ((uint32_t)(t >> 1) & 1u) ^ 1u, wc, 104)) break;
        tc_fence_after();
        const uint32_t kb = ring + (uint32_t)slot * KT_UNIT;
        const uint64_t k_desc0 = desc_k_sw128(kb), k_desc1 = desc_k_sw128(kb + KT_HALF);
        const uint32_t d = tmem + (uint32_t)sb * NQ;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) umma_bf16(d, k_desc0 + (uint64_t)(kk * 2), q_desc0 + (uint64_t)(kk * 2), idesc_s, kk ? 1u : 0u);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) umma_bf16(d, k_desc1 + (uint64_t)(kk * 2), q_desc1 + (uint64_t)(kk * 2), idesc_s, 1u);
        umma_commit(smem_u32(&empty_u[slot]));       // the K unit is free once these MMAs have retired
        umma_commit(smem_u32(&s_full[sb]));
      }
      if (*aborted) {                                // give-up path: see the MMAs already issued retire
        umma_commit(smem_u32(&drain_bar[0]));
        mbar_wait_drain(smem_u32(&drain_bar[0]), 0, 20000000ll);
      }
    }
  } else if (warp == W_PV) {
    griddep_wait();
    griddep_launch();
    // ---------------- PV issuer ----------------
    if (lane == 0) {
      // A = V tile read M-major (M = head_dim: two 64-wide blocks KT_HALF apart; 8-key groups 1024 bytes apart),
      // B = P^T read N-major (N = hi and lo terms side by side: 2 NQ / 64 blocks KT_HALF apart)
      constexpr uint32_t idesc_pv = idesc_bf16(128, 2 * NQ, true, true);
      const int t_stop = *aborted ? 0 : T;
      for (int t = 0; t < t_stop; ++t) {
        const int u = 2 * t + 1, slot = u % NU;
        const int pb = t % PB;
        if (!mbar_wait(smem_u32(&p_ready[pb]), (uint32_t)(t / PB) & 1u, wc, 105)) break;
        if (!wait_unit(u, 106)) break;
        tc_fence_after();
        const uint32_t vb = ring + (uint32_t)slot * KT_UNIT;
        const uint32_t d = tmem + O_COL;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
          umma_bf16(d, desc_mn_sw128(vb + ks * 2048u, KT_HALF, 1024u), desc_mn_sw128(p_base + (uint32_t)pb * 2u * P_TERM + ks * 2048u, KT_HALF, 1024u),
                    idesc_pv, (t == 0 && ks == 0) ? 0u : 1u);
        umma_commit(smem_u32(&empty_u[slot]));
        umma_commit(smem_u32(&pv_done[pb]));
      }
      if (*aborted) {                                // give-up path: see the MMAs already issued retire
        umma_commit(smem_u32(&drain_bar[1]));
        mbar_wait_drain(smem_u32(&drain_bar[1]), 0, 20000000ll);
      }
    }
  } else {
    // ---------------- softmax: thread = (key lane of the tile, block of 32 queries) ----------------
    const int lq = warp & 3, cb = warp >> 2;
    const int r = lq * 32 + lane;                               // key row of the tile = tensor-memory lane
    const int st = (int)threadIdx.x, nst = 128 * NCB;           // index among the softmax threads
    const uint32_t lane_base = (uint32_t)(lq * 32) << 16;
    const bool tree_keys = t1 * KT_TILE > L && T > 0;           // this CTA's range reaches past the prefix
    if (tree_keys) {
      // transposed ancestor masks: bit q of desc_t[j] <-> tree key j is visible to query row0 + q
      // A bit-matrix transposition by warp votes: a warp takes one block of 32 queries (lane = query) and one
      // 64-bit ancestor word, and one ballot per tree key of that word gives the key's 32 visibility bits.
      const int n_qb = (nq + 31) >> 5, n_kw = (n_tree + 63) >> 6;
      for (int item = warp; item < n_qb * n_kw; item += NSW) {
        const int qb = item % n_qb, kw = item / n_qb;
        const int q = qb * 32 + lane;
        const uint64_t a = q < nq ? p.anc[(size_t)q * CERB_ANC_WORDS + kw] : 0ull;
        const int j_end = min(64, n_tree - kw * 64);
        for (int jj = 0; jj < j_end; ++jj) {
          const uint32_t bits = __ballot_sync(0xffffffffu, (a >> jj) & 1ull);
          if (lane == (jj & 31)) desc_t[kw * 64 + jj][qb] = bits;
        }
      }
    }
    griddep_wait();
    griddep_launch();
    {
      // stage Q (zeros past the last live node) in the swizzled K-major layout: 16-byte pieces, NQ * 16 of them,
      // spread over all softmax threads so that every thread has its loads in flight at once
      constexpr int PIECES = (NQ * 16 + 128 * NCB - 1) / (128 * NCB);
      uint4 v[PIECES];
#pragma unroll
      for (int i = 0; i < PIECES; ++i) {
        const int piece = st + i * nst, row = piece >> 4, c = piece & 15;
        v[i] = row < nq ? reinterpret_cast<const uint4*>(p.q + ((qrow + row) * p.H + h) * DH)[c] : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int i = 0; i < PIECES; ++i) {
        const int piece = st + i * nst, row = piece >> 4, c = piece & 15;
        if (piece < NQ * 16)
          *reinterpret_cast<uint4*>(smem_gen + (q_base - smem_base) + (uint32_t)(c >> 3) * QHALF + (uint32_t)row * 128u +
                                  (uint32_t)(((c & 7) ^ (row & 7)) << 4)) = v[i];
      }
      proxy_fence();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&q_ready));
    }
    asm volatile("bar.sync 2, %0;" ::"r"(nst) : "memory");      // desc_t is complete
    // queries of this block that exist
    const int qn = nq - cb * 32;
    const uint32_t qmask = qn >= 32 ? 0xffffffffu : qn <= 0 ? 0u : ((1u << qn) - 1u);
    float* mr = m_ref + cb * 32;
    int* pend = m_pending + cb * 32;
    float l_acc[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) l_acc[j] = 0.f;
    uint8_t* prow0 = smem_gen + (p_base - smem_base) + (uint32_t)(cb >> 1) * KT_HALF + (uint32_t)r * 128u;
    for (int t = 0; t < T; ++t) {
      const int sb = t & 1;
      mbar_wait(smem_u32(&s_full[sb]), (uint32_t)(t >> 1) & 1u, wc, 107);
      tc_fence_after();
      float sc[32];
      const uint32_t s_addr = tmem + lane_base + (uint32_t)sb * NQ + (uint32_t)cb * 32u;
      tmem_ld16_nowait(s_addr, reinterpret_cast<uint32_t*>(sc));
      tmem_ld16_nowait(s_addr + 16u, reinterpret_cast<uint32_t*>(sc + 16));
      tmem_ld_wait();
      const int kpos = (t0 + t) * KT_TILE + r;
      const bool masked = (t0 + t + 1) * KT_TILE > L;           // the tile reaches past the prefix (uniform over the CTA)
      const uint32_t vis = !masked ? 0xffffffffu : kpos < L ? qmask : kpos < kv_total ? (desc_t[kpos - L][cb] & qmask) : 0u;
      if (t == 0 && !masked) {
        // First tile, all keys visible: the scores of its first key serve as the reference (any value within the
        // exponent range of the true maximum does; whatever exceeds it by 2^8 later raises it the usual way).
        if (r == 0) {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if ((qmask >> j) & 1u) mr[j] = sc[j] * p.scale_log2;
        }
        asm volatile("bar.sync %0, 128;" ::"r"(4 + cb) : "memory");
      }
      // scores relative to the reference, in bits: t = s * scale - m[q]; the largest decides whether m must rise
      float tmax = -INFINITY;
      if (!masked) {
#pragma unroll
        for (int j4 = 0; j4 < 32; j4 += 4) {
          const float4 m4 = *reinterpret_cast<const float4*>(mr + j4);
          sc[j4] = fmaf(sc[j4], p.scale_log2, -m4.x);
          sc[j4 + 1] = fmaf(sc[j4 + 1], p.scale_log2, -m4.y);
          sc[j4 + 2] = fmaf(sc[j4 + 2], p.scale_log2, -m4.z);
          sc[j4 + 3] = fmaf(sc[j4 + 3], p.scale_log2, -m4.w);
          tmax = fmaxf(fmaxf(tmax, fmaxf(sc[j4], sc[j4 + 1])), fmaxf(sc[j4 + 2], sc[j4 + 3]));
        }
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          sc[j] = ((vis >> j) & 1u) ? fmaf(sc[j], p.scale_log2, -mr[j]) : -INFINITY;
          tmax = fmaxf(tmax, sc[j]);
        }
      }
      if (__any_sync(0xffffffffu, tmax > KT_RAISE)) {
        // Rare: a score of this warp's keys calls for a higher reference.  Report, per query, the largest visible
        // score of these 32 keys (one warp reduction each; lane j then files query j's).
        uint32_t raw[32];
        tmem_ld16_nowait(s_addr, raw);
        tmem_ld16_nowait(s_addr + 16u, raw + 16);
        tmem_ld_wait();
        int mine = f2ord(-INFINITY);
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float v = ((vis >> j) & 1u) ? __uint_as_float(raw[j]) * p.scale_log2 : -INFINITY;
          const int red = __reduce_max_sync(0xffffffffu, f2ord(v));
          if (lane == j) mine = red;
        }
        atomicMax(&pend[lane], mine);
        if (lane == 0) raise_at[t & 1][cb] = t + 1;
      }
      asm volatile("bar.sync %0, 128;" ::"r"(4 + cb) : "memory");     // the four warps of this query block agree
      bool waited_pv = false;
      if (raise_at[t & 1][cb] == t + 1) {
        // New reference m' = max(m, reported) for this block's queries: what was accumulated under m shrinks by
        // 2^(m - m'), this tile's scores are taken again relative to m'.
        auto alpha_of = [&](int j) { return ex2(mr[j] - fmaxf(mr[j], ord2f(pend[j]))); };
        bool any_change = false;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float mo = mr[j], mn = fmaxf(mo, ord2f(pend[j]));
          if (mn != mo) {
            any_change = true;
            l_acc[j] *= ex2(mo - mn);
          }
        }
        if (t > 0 && any_change) {
          mbar_wait(smem_u32(&pv_done[(t - 1) % PB]), (uint32_t)((t - 1) / PB) & 1u, wc, 108);      // O^T at rest (PV retires in order)
          tc_fence_after();
          waited_pv = true;
          // rows of O^T = head-dim lanes of this warp's quarter; columns of this query block, both terms
#pragma unroll 1
          for (int c0 = 0; c0 < 4; ++c0) {
            const uint32_t o_addr = tmem + lane_base + O_COL + (uint32_t)(c0 >> 1) * NQ + (uint32_t)cb * 32u + (uint32_t)(c0 & 1) * 16u;
            uint32_t o[16];
            tmem_ld16_nowait(o_addr, o);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha_of((c0 & 1) * 16 + j));
            tmem_st16(o_addr, o);
          }
          tmem_st_wait();
        }
        {
          uint32_t raw[32];
          tmem_ld16_nowait(s_addr, raw);
          tmem_ld16_nowait(s_addr + 16u, raw + 16);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j)
            sc[j] = ((vis >> j) & 1u) ? fmaf(__uint_as_float(raw[j]), p.scale_log2, -fmaxf(mr[j], ord2f(pend[j]))) : -INFINITY;
        }
        asm volatile("bar.sync %0, 128;" ::"r"(4 + cb) : "memory");   // everyone has read the old reference
        if (lq == 0) mr[lane] = fmaxf(mr[lane], ord2f(pend[lane]));
        asm volatile("bar.sync %0, 128;" ::"r"(4 + cb) : "memory");   // the new reference is in place
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&s_free[sb]));        // S^T is no longer needed: its buffer may be overwritten
      // probabilities, running sums, and the two bf16 terms p = hi + lo: hi is p cut to its upper 16 bits, lo the
      // (exact) remainder cut the same way -- integer operations only, the conversion unit stays free for exp2
      uint32_t hi[16], lo[16];
#pragma unroll
      for (int j = 0; j < 32; j += 2) {
        const float p0 = ex2(sc[j]), p1 = ex2(sc[j + 1]);
        l_acc[j] += p0;
        l_acc[j + 1] += p1;
        const uint32_t b0 = __float_as_uint(p0), b1 = __float_as_uint(p1);
        hi[j >> 1] = __byte_perm(b0, b1, 0x7632);
        const float r0 = p0 - __uint_as_float(b0 & 0xffff0000u), r1 = p1 - __uint_as_float(b1 & 0xffff0000u);
        lo[j >> 1] = __byte_perm(__float_as_uint(r0), __float_as_uint(r1), 0x7632);
      }
      if (t >= PB && !(PB == 1 && waited_pv)) {
        mbar_wait(smem_u32(&pv_done[t % PB]), (uint32_t)(t / PB - 1) & 1u, wc, 109);        // this tile's P^T buffer is free
        tc_fence_after();
      }
      uint8_t* prow = prow0 + (size_t)(t % PB) * (2 * P_TERM);
      if (cb == 0 && kpos >= kv_total) {
        // Keys past the end (only in the last tile): the row of V may hold anything (stale pool memory); zero it
        // so that a zero probability times a non-finite value cannot poison the sum.  V must have landed first.
        const int u = 2 * t + 1;
        wait_unit(u, 110);
        uint8_t* vrow = smem_gen + (ring - smem_base) + (size_t)(u % NU) * KT_UNIT + (size_t)r * 128;
#pragma unroll
        for (int c = 0; c < 16; ++c) *reinterpret_cast<uint4*>(vrow + (size_t)(c >> 3) * KT_HALF + (c & 7) * 16) = make_uint4(0, 0, 0, 0);
      }
      // P^T row of this key: 32 queries = four 16-byte pieces per term
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const uint32_t off = (uint32_t)((((cb & 1) * 4 + c) ^ (r & 7)) << 4);
        *reinterpret_cast<uint4*>(prow + off) = make_uint4(hi[4 * c], hi[4 * c + 1], hi[4 * c + 2], hi[4 * c + 3]);
        *reinterpret_cast<uint4*>(prow + P_TERM + off) = make_uint4(lo[4 * c], lo[4 * c + 1], lo[4 * c + 2], lo[4 * c + 3]);
      }
      proxy_fence();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&p_ready[t % PB]));
    }
    // ---- this CTA's rows (O, m, l) into shared memory ----
    if (T > 0) {
      mbar_wait(smem_u32(&pv_done[(T - 1) % PB]), (uint32_t)((T - 1) / PB) & 1u, wc, 111);
      tc_fence_after();
    }
    // row sums: transpose-reduce the 32 partials of a warp (lane q ends up with the sum for query q)
    {
#pragma unroll
      for (int w = 16; w >= 1; w >>= 1) {
#pragma unroll
        for (int j = 0; j < w; ++j) {
          const bool upper = (lane & w) != 0;
          const float send = upper ? l_acc[j] : l_acc[j + w];
          const float keep = upper ? l_acc[j + w] : l_acc[j];
          l_acc[j] = keep + __shfl_xor_sync(0xffffffffu, send, w);
        }
      }
      // lane's bit pattern now selects the query: bit w of the lane chose the upper half at step w
      l_part[lq][cb * 32 + lane] = l_acc[0];
    }
    asm volatile("bar.sync 2, %0;" ::"r"(nst) : "memory");      // every MMA has retired: shared memory can be reused
    {
      // thread = head-dim element r of this warp's quarter, 32 queries of its block
      uint32_t oh[32], ol[32];
      if (T > 0) {
        const uint32_t o_addr = tmem + lane_base + O_COL + (uint32_t)cb * 32u;
        tmem_ld16_nowait(o_addr, oh);
        tmem_ld16_nowait(o_addr + 16u, oh + 16);
        tmem_ld16_nowait(o_addr + NQ, ol);
        tmem_ld16_nowait(o_addr + NQ + 16u, ol + 16);
        tmem_ld_wait();
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) oh[j] = ol[j] = 0u;
      }
#pragma unroll
      for (int j = 0; j < 32; ++j) mrg[(size_t)(cb * 32 + j) * ROWF + r] = __uint_as_float(oh[j]) + __uint_as_float(ol[j]);
      if (lq == 0) {
        const int q = cb * 32 + lane;
        mrg[(size_t)q * ROWF + DH] = m_ref[q];
        mrg[(size_t)q * ROWF + DH + 1] = (l_part[0][q] + l_part[1][q]) + (l_part[2][q] + l_part[3][q]);
      }
    }
    tc_fence_before();
    asm volatile("bar.sync 2, %0;" ::"r"(nst) : "memory");

    // ---- output: final, or partial + fixed-order merge by the last CTA of this (sequence, head) ----
    const int ct = st, nct = nst, RP = p.rows_pad;
    const float LN2 = 0.6931471805599453f;
    if (p.cluster) {
      // merged after the role branches, where every thread of the cluster meets
    } else if (p.nsplit == 1) {
      for (int idx = ct; idx < nq * (DH / 4); idx += nct) {
        const int rr = idx / (DH / 4), c4 = idx % (DH / 4);
        const float inv = 1.0f / mrg[(size_t)rr * ROWF + DH + 1];
        const float4 v = *reinterpret_cast<const float4*>(mrg + (size_t)rr * ROWF + c4 * 4);
        *reinterpret_cast<uint2*>(p.out + ((qrow + rr) * p.H + h) * DH + c4 * 4) =
            make_uint2(pack_bf16(v.x * inv, v.y * inv), pack_bf16(v.z * inv, v.w * inv));
      }
      if (p.lse)
        for (int rr = ct; rr < nq; rr += nct)
          p.lse[((size_t)b * p.H + h) * p.n + rr] = (mrg[(size_t)rr * ROWF + DH] + log2f(mrg[(size_t)rr * ROWF + DH + 1])) * LN2;
    } else {
      float* part = p.partial + (((size_t)b * p.H + h) * p.nsplit) * (size_t)(RP * ROWF);
      float* mine = part + (size_t)split * (RP * ROWF);
      for (int idx = ct; idx < nq * ROWF; idx += nct) __stcg(mine + idx, mrg[idx]);
      __threadfence();
      asm volatile("bar.sync 2, %0;" ::"r"(nst) : "memory");
      if (ct == 0) ticket_s = atomicAdd(&p.counters[b * p.H + h], 1u);
      asm volatile("bar.sync 2, %0;" ::"r"(nst) : "memory");
      if (ticket_s == (unsigned)p.nsplit - 1) {
        __threadfence();
        float* wts = mrg;                                   // [nsplit][RP]
        for (int rr = ct; rr < nq; rr += nct) {
          float M = -INFINITY;
          for (int s2 = 0; s2 < p.nsplit; ++s2) M = fmaxf(M, __ldcg(part + (size_t)s2 * (RP * ROWF) + rr * ROWF + DH));
          const float u = M == -INFINITY ? 0.f : M;
          float Lsum = 0.f;
          for (int s2 = 0; s2 < p.nsplit; ++s2) {
            const float* pr = part + (size_t)s2 * (RP * ROWF) + rr * ROWF;
            const float ms = __ldcg(pr + DH);
            const float w = exp2f(ms - u);
            wts[s2 * RP + rr] = w;
            Lsum += __ldcg(pr + DH + 1) * w;
          }
          const float inv = 1.0f / Lsum;
          for (int s2 = 0; s2 < p.nsplit; ++s2) wts[s2 * RP + rr] *= inv;
          if (p.lse) p.lse[((size_t)b * p.H + h) * p.n + rr] = (M + log2f(Lsum)) * LN2;
        }
        asm volatile("bar.sync 2, %0;" ::"r"(nst) : "memory");
        for (int idx = ct; idx < nq * (DH / 4); idx += nct) {
          const int rr = idx / (DH / 4), c4 = idx % (DH / 4);
          const float4* src = reinterpret_cast<const float4*>(part + (size_t)rr * ROWF) + c4;
          float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
          for (int s2 = 0; s2 < p.nsplit; ++s2) {
            const float4 v = __ldcg(src + (size_t)s2 * (RP * ROWF / 4));
            const float w = wts[s2 * RP + rr];
            acc.x += v.x * w; acc.y += v.y * w; acc.z += v.z * w; acc.w += v.w * w;
          }
          *reinterpret_cast<uint2*>(p.out + ((qrow + rr) * p.H + h) * DH + c4 * 4) =
              make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
        }
        if (ct == 0) p.counters[b * p.H + h] = 0u;          // ready for the next launch
      }
    }
  }
  if (p.cluster) {
    // The splits of this (sequence, head) are the CTAs of one cluster (rank = split).  Each holds its rows
    // (O, m, l) in shared memory; once all have arrived, CTA r finishes rows r, r + nsplit, ...: it reads those
    // rows from every member in split order, weighs them and writes the final output.  Nobody leaves before
    // the second meeting, so no shared memory is read after its CTA has gone.
    cluster_start_wait();
    if (warp < NSW) {
      const int ct = (int)threadIdx.x, nwarps = NSW;
      cluster_meet(&cl_bar[0], p.nsplit, ct, wc, 112);              // every member's rows are in place
      const float LN2 = 0.6931471805599453f;
      const uint32_t mine = smem_u32(smem_gen);
      const int c4 = ct & 31;
      for (int rr = split + p.nsplit * (ct >> 5); rr < nq; rr += p.nsplit * nwarps) {
        const uint32_t row_off = (uint32_t)rr * (ROWF * 4);
        // every member's (m, l) and this thread's four output columns, all loads in flight at once (a cluster
        // has at most 8 members)
        float ms[8], ls[8];
        float4 vs[8];
#pragma unroll
        for (int s2 = 0; s2 < 8; ++s2) {
          if (s2 < p.nsplit) {
            const uint32_t base = mapa_u32(mine, (uint32_t)s2) + row_off;
            ms[s2] = ld_cluster_f32(base + DH * 4);
            ls[s2] = ld_cluster_f32(base + DH * 4 + 4);
            vs[s2] = ld_cluster_v4(base + (uint32_t)c4 * 16u);
          } else {
            ms[s2] = -INFINITY; ls[s2] = 0.f; vs[s2] = make_float4(0.f, 0.f, 0.f, 0.f);
          }
        }
        float M = -INFINITY;
#pragma unroll
        for (int s2 = 0; s2 < 8; ++s2) M = fmaxf(M, ms[s2]);
        float Lsum = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int s2 = 0; s2 < 8; ++s2) {          // split order: the sum does not depend on timing
          const float w = ex2(ms[s2] - M);
          Lsum += ls[s2] * w;
          acc.x += vs[s2].x * w; acc.y += vs[s2].y * w; acc.z += vs[s2].z * w; acc.w += vs[s2].w * w;
        }
        const float inv = 1.0f / Lsum;
        *reinterpret_cast<uint2*>(p.out + ((qrow + rr) * p.H + h) * DH + c4 * 4) =
            make_uint2(pack_bf16(acc.x * inv, acc.y * inv), pack_bf16(acc.z * inv, acc.w * inv));
        if (c4 == 0 && p.lse) p.lse[((size_t)b * p.H + h) * p.n + rr] = (M + log2f(Lsum)) * LN2;
      }
      asm volatile("bar.sync 2, %0;" ::"r"(128 * NCB) : "memory");            // this CTA has read all it needs
      if (warp == 0) cluster_meet_before_exit(&cl_bar[1], p.nsplit, lane, wc, &exit_flag_s, 113);
    }
  }
  tc_fence_before();
  __syncthreads();                             // nobody exits before warp 0 has seen every member done
  if (warp == W_QK) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
}

}  // namespace
