// bf16 GEMM of the verification forward on the 5th-generation tensor cores (tcgen05 + TMEM).
//
//   out[split][m][n] = sum over this split's k of X[m][k] * W[n][k]        (fp32)
//
// A decoding step has few activation rows (tree nodes x batch) and large weight matrices, so the
// kernel is organised around streaming W exactly once at HBM speed ("swap-AB"): a CTA takes a
// 128-row tile of W as the MMA's A operand (M = 128) and up to 256 activation rows as the B
// operand (N = rows), accumulates D[128][rows] in tensor memory and writes it transposed.
// Where W has too few 128-row tiles to occupy the GPU the K dimension is split across CTAs and
// each split writes its own fp32 partial; consumers add the partials in index order.
//
// Roles inside a CTA (192 threads): warp 0 = TMA producer (one lane), warp 1 = TMEM allocator and
// MMA issuer (one lane), warps 2-5 = epilogue (each owns the 32 TMEM lanes of its warp quarter).
// Stages are handed over with mbarriers; every wait is bounded and reports CERB_E_TIMEOUT through
// a status word instead of hanging.
#include "cerb_internal.cuh"

namespace cerb {

namespace {

constexpr int BM = 128;          // weight rows per CTA (MMA M)
constexpr int BK = 64;           // k elements per stage: 64 bf16 = one 128-byte swizzle row
constexpr int MAX_STAGES = 8;
constexpr uint32_t A_STAGE_BYTES = BM * BK * 2;
constexpr uint64_t kWaitNs = 2000000000ull;   // 2 s: far beyond any legitimate wait

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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
// Bounded wait.  After the first time-out in a CTA every later wait gives up quickly, so the CTA
// still runs to its end (releasing tensor memory) in bounded time.
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: gives up after kWaitNs of wall time.  After the first time-out in a CTA (or when
// an earlier kernel already reported one) every later wait gives up almost at once, so the CTA
// still runs to its end in bounded time.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* aborted, int32_t* status) {
  if (mbar_try_wait(bar, parity)) return;
  const uint64_t t0 = global_ns();
  const uint64_t budget = *aborted ? 20000ull : kWaitNs;
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return;
    if (global_ns() - t0 > budget) break;
  }
  *aborted = 1;
  atomicExch(status, CERB_E_TIMEOUT);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"((uint64_t)map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}

// Shared-memory matrix descriptor for a K-major operand tile stored as rows of 128 bytes with the
// 128-byte swizzle (what TMA writes): 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);        // start address, 16-byte units
  d |= (uint64_t)1 << 16;                           // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024u >> 4) << 32;                // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                           // descriptor version for this architecture
  d |= (uint64_t)2 << 61;                           // layout: 128-byte swizzle
  return d;
}

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
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

struct GemmParams {
  float* out;
  int32_t* status;
  int M, N, K;
  int n_mma;          // activation rows per pass (16..256, power of two)
  int num_kb;         // ceil(K / 64)
  int kb_per_split;
  int stages;
  uint32_t idesc;
  uint32_t tmem_cols;
};

__global__ void __launch_bounds__(192) gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmW,
                                                        const __grid_constant__ CUtensorMap tmX, const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t empty_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t accum_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int aborted_s;
  volatile int* aborted = &aborted_s;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t b_bytes = (uint32_t)p.n_mma * BK * 2;
  const uint32_t stage_bytes = A_STAGE_BYTES + b_bytes;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x, split = blockIdx.y, mchunk = blockIdx.z;
  const int kb0 = split * p.kb_per_split;
  const int kb1 = min(p.num_kb, kb0 + p.kb_per_split);

  if (threadIdx.x == 0) {
    aborted_s = (*p.status != 0);
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    mbar_init(smem_u32(&accum_bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(p.tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == 0) {
    if (lane == 0) {
      for (int kb = kb0, i = 0; kb < kb1; ++kb, ++i) {
        int s = i % p.stages;
        uint32_t ph = (uint32_t)(i / p.stages) & 1u;
        mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, aborted, p.status);
        uint32_t fb = smem_u32(&full_bar[s]);
        mbar_expect_tx(fb, stage_bytes);
        uint32_t a_dst = smem_base + (uint32_t)s * stage_bytes;
        tma_load_2d(a_dst, &tmW, kb * BK, tile * BM, fb);
        tma_load_2d(a_dst + A_STAGE_BYTES, &tmX, kb * BK, mchunk * kGemmRowsPerPass, fb);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      for (int kb = kb0, i = 0; kb < kb1; ++kb, ++i) {
        int s = i % p.stages;
        uint32_t ph = (uint32_t)(i / p.stages) & 1u;
        mbar_wait(smem_u32(&full_bar[s]), ph, aborted, p.status);
        tc_fence_after();
        uint32_t a_src = smem_base + (uint32_t)s * stage_bytes;
        uint64_t adesc = umma_desc_sw128(a_src);
        uint64_t bdesc = umma_desc_sw128(a_src + A_STAGE_BYTES);
#pragma unroll
        for (int kk = 0; kk < BK / 16; ++kk) {
          // advance 16 k elements = 32 bytes inside the swizzled row: +2 in 16-byte units
          umma_bf16(tmem_base, adesc + (uint64_t)(kk * 2), bdesc + (uint64_t)(kk * 2), p.idesc, (i > 0 || kk > 0) ? 1u : 0u);
        }
        umma_commit(smem_u32(&empty_bar[s]));      // frees the stage once these MMAs have read it
      }
      umma_commit(smem_u32(&accum_bar));           // accumulator complete
    }
  } else {
    const int quarter = warp & 3;                  // TMEM lanes 32*quarter .. +31 belong to this warp
    mbar_wait(smem_u32(&accum_bar), 0, aborted, p.status);
    tc_fence_after();
    const int n_out = tile * BM + quarter * 32 + lane;
    const int m_base = mchunk * kGemmRowsPerPass;
    const int m_cnt = min(p.n_mma, p.M - m_base);
    float* o = p.out + ((size_t)split * p.M + m_base) * p.N + n_out;
    const bool n_ok = n_out < p.N;
    for (int c0 = 0; c0 < m_cnt; c0 += 16) {
      uint32_t r[16];
      tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, r);
      if (n_ok) {
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (c0 + j < m_cnt) o[(size_t)(c0 + j) * p.N] = __uint_as_float(r[j]);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

int encode_2d(CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer, uint64_t row_bytes, uint32_t box_inner,
              uint32_t box_outer) {
  if (init_driver_api() != CERB_OK) return CERB_E_CUDA;
  if (((uintptr_t)base & 15) || (row_bytes & 15)) return CERB_E_SHAPE;
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {row_bytes};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? CERB_OK : CERB_E_CUDA;
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

// How many K splits to use so that about two CTAs per SM stream weights concurrently.
int gemm_plan_split(int sm_count, int M, int N, int K) {
  int tiles = (N + BM - 1) / BM;
  int mchunks = (M + kGemmRowsPerPass - 1) / kGemmRowsPerPass;
  int num_kb = (K + BK - 1) / BK;
  int want = (2 * sm_count + tiles * mchunks - 1) / (tiles * mchunks);
  int max_by_k = num_kb / 4 > 0 ? num_kb / 4 : 1;
  int s = want < 1 ? 1 : want;
  if (s > max_by_k) s = max_by_k;
  if (s > kGemmMaxSplit) s = kGemmMaxSplit;
  int per = (num_kb + s - 1) / s;
  return (num_kb + per - 1) / per;
}

int launch_gemm_bf16(cerb_ctx* c, const CUtensorMap* tmW, const ActMaps* tmX, float* out, int M, int N, int K,
                     int nsplit, int32_t* status, cudaStream_t st) {
  if (M <= 0 || N <= 0 || K <= 0 || (K % 8) != 0) return CERB_E_SHAPE;
  GemmParams p;
  int mchunks = (M + kGemmRowsPerPass - 1) / kGemmRowsPerPass;
  int bucket = row_bucket(M < kGemmRowsPerPass ? M : kGemmRowsPerPass);
  p.out = out;
  p.status = status;
  p.M = M; p.N = N; p.K = K;
  p.n_mma = bucket_rows(bucket);
  p.num_kb = (K + BK - 1) / BK;
  p.kb_per_split = (p.num_kb + nsplit - 1) / nsplit;
  int splits = (p.num_kb + p.kb_per_split - 1) / p.kb_per_split;
  if (splits != nsplit) return CERB_E_ARG;
  uint32_t stage_bytes = A_STAGE_BYTES + (uint32_t)p.n_mma * BK * 2;
  uint32_t budget = stage_bytes <= 28 * 1024 ? 110 * 1024 : 200 * 1024;
  p.stages = (int)(budget / stage_bytes);
  if (p.stages > MAX_STAGES) p.stages = MAX_STAGES;
  if (p.stages < 2) return CERB_E_SHAPE;
  p.tmem_cols = p.n_mma < 32 ? 32u : (uint32_t)p.n_mma;
  // instruction descriptor: D fp32, A and B bf16, both K-major, N = n_mma, M = 128
  p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_mma >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
  size_t smem = (size_t)p.stages * stage_bytes + 1024;
  static size_t configured = 0;
  if (smem > configured) {
    CERB_CUDA_OK(cudaFuncSetAttribute(gemm_bf16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(220 * 1024)));
    configured = 220 * 1024;
  }
  dim3 grid((N + BM - 1) / BM, nsplit, mchunks);
  gemm_bf16_kernel<<<grid, 192, smem, st>>>(*tmW, tmX->m[bucket], p);
  CERB_LAUNCH_CHECK(c);
  return CERB_OK;
}

}  // namespace cerb
