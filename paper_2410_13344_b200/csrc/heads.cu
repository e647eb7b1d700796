// Cerberus decoding heads (Section 4.1).  Every head is a stack of Resblocks
//     plain:      out = SiLU((W h + b) + h)
//     two-input:  h = Concat(h_i, h_{i-1});  out = SiLU((W h + b) + h)
// followed by one FC layer to the vocabulary.  The sequential link sits inside the heads, so all
// heads advance level by level together: one launch per level covers every head (grid.y = head),
// the two-input block of head i reads head i-1's state as it entered the same level.  At batch 1
// each level is a matrix-vector product: the kernel streams W once with 16-byte loads, keeps the
// (concatenated) input vector in shared memory as fp32 and fuses bias, residual and SiLU.
// The FC layer reuses the kernel without an epilogue; a per-head top-k (value descending, lower id
// first among equals; per vocabulary chunk, then over the chunks' candidates) and the tree fill follow.
#include "cerb_internal.cuh"

namespace cerb {

namespace {

constexpr int ROWS_PER_WARP = 4;
constexpr int WARPS = 8;
constexpr int ROWS_PER_BLOCK = ROWS_PER_WARP * WARPS;

struct HeadJob {
  const void* W;        // [rows][w_in]
  const void* bias;     // [rows] or null
  int rows;             // output width
  int w0;               // own input width
  int w1;               // appended width (0 for a plain block)
  int src;              // head whose state is appended, or -1
};

struct LevelParams {
  HeadJob job[CERB_MAX_HEADS];
  const float* state_in;    // [B][Hc][wmax]
  float* out;               // state_out [B][Hc][wmax] or logits [B][Hc][out_stride]
  int Hc, wmax, out_stride, B, b0;
  int epilogue;             // 1: SiLU(acc + bias + input[row]); 0: plain product
};

template <typename T> struct Vec16;
template <> struct Vec16<bf16> {
  static constexpr int N = 8;
  static __device__ __forceinline__ void load(const bf16* p, float* f) {
    uint4 v;
    // streamed once: no L1 allocation, and the memory side is asked for 256-byte pieces
    asm volatile("ld.global.nc.L1::no_allocate.L2::256B.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) { float2 t = __bfloat1622float2(h[i]); f[2 * i] = t.x; f[2 * i + 1] = t.y; }
  }
};
template <> struct Vec16<float> {
  static constexpr int N = 4;
  static __device__ __forceinline__ void load(const float* p, float* f) {
    float4 v = __ldg(reinterpret_cast<const float4*>(p));
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
  }
};
template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<bf16>(const bf16* p) { return __bfloat162float(*p); }

template <typename T, int NB>
__global__ void __launch_bounds__(WARPS * 32) head_gemv_kernel(const LevelParams P) {
  extern __shared__ float su[];                       // [NB][w]
  griddep_wait();
  griddep_launch();
  const int head = blockIdx.y;
  const HeadJob J = P.job[head];
  const int w = J.w0 + J.w1;
  const int row_base = blockIdx.x * ROWS_PER_BLOCK;
  if (row_base >= J.rows) return;
  for (int nb = 0; nb < NB; ++nb) {
    int seq = P.b0 + nb;
    const float* own = P.state_in + ((size_t)seq * P.Hc + head) * P.wmax;
    const float* oth = J.src >= 0 ? P.state_in + ((size_t)seq * P.Hc + J.src) * P.wmax : own;
    for (int k = threadIdx.x; k < w; k += blockDim.x)
      su[nb * w + k] = seq < P.B ? (k < J.w0 ? own[k] : oth[k - J.w0]) : 0.f;
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r0 = row_base + warp * ROWS_PER_WARP;
  constexpr int E = Vec16<T>::N;
  float acc[ROWS_PER_WARP][NB];
#pragma unroll
  for (int i = 0; i < ROWS_PER_WARP; ++i)
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) acc[i][nb] = 0.f;
  const T* Wp = reinterpret_cast<const T*>(J.W);
#pragma unroll 2
  for (int k = lane * E; k < w; k += 32 * E) {
    float wv[ROWS_PER_WARP][E];
#pragma unroll
    for (int i = 0; i < ROWS_PER_WARP; ++i) {
      int r = r0 + i;
      if (r < J.rows) Vec16<T>::load(Wp + (size_t)r * w + k, wv[i]);
      else {
#pragma unroll
        for (int e = 0; e < E; ++e) wv[i][e] = 0.f;
      }
    }
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
      float x[E];
#pragma unroll
      for (int e = 0; e < E; ++e) x[e] = su[nb * w + k + e];
#pragma unroll
      for (int i = 0; i < ROWS_PER_WARP; ++i)
#pragma unroll
        for (int e = 0; e < E; ++e) acc[i][nb] = fmaf(wv[i][e], x[e], acc[i][nb]);
    }
  }
#pragma unroll
  for (int i = 0; i < ROWS_PER_WARP; ++i)
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
      for (int o = 16; o > 0; o >>= 1) acc[i][nb] += __shfl_xor_sync(0xffffffffu, acc[i][nb], o);
  if (lane == 0) {
    for (int i = 0; i < ROWS_PER_WARP; ++i) {
      int r = r0 + i;
      if (r >= J.rows) continue;
      for (int nb = 0; nb < NB; ++nb) {
        int seq = P.b0 + nb;
        if (seq >= P.B) continue;
        float y = acc[i][nb];
        if (P.epilogue) {
          y += ldf(reinterpret_cast<const T*>(J.bias) + r) + su[nb * w + r];
          y = y / (1.0f + expf(-y));
        }
        P.out[((size_t)seq * P.Hc + head) * P.out_stride + r] = y;
      }
    }
  }
}

template <typename T>
__global__ void head_init_kernel(const T* __restrict__ h_last, float* __restrict__ state, int Hc, int wmax, int d) {
  griddep_wait();
  griddep_launch();
  int b = blockIdx.x, h = blockIdx.y;
  for (int k = threadIdx.x; k < d; k += blockDim.x)
    state[((size_t)b * Hc + h) * wmax + k] = ldf(h_last + (size_t)b * d + k);
}

__device__ __forceinline__ bool better(float va, int ia, float vb, int ib) { return va > vb || (va == vb && ia < ib); }

// Block-wide arg-best over (value, id) pairs in (value descending, id ascending) order.
__device__ __forceinline__ void block_best(float& best, int& bi, float* sv, int* si) {
  for (int o = 16; o > 0; o >>= 1) {
    float ov = __shfl_xor_sync(0xffffffffu, best, o);
    int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (better(ov, oi, best, bi)) { best = ov; bi = oi; }
  }
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
  if (l == 0) { sv[w] = best; si[w] = bi; }
  __syncthreads();
  if (w == 0) {
    best = l < nw ? sv[l] : -INFINITY;
    bi = l < nw ? si[l] : 0x7fffffff;
    for (int o = 16; o > 0; o >>= 1) {
      float ov = __shfl_xor_sync(0xffffffffu, best, o);
      int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (better(ov, oi, best, bi)) { best = ov; bi = oi; }
    }
    if (l == 0) { sv[0] = best; si[0] = bi; }
  }
  __syncthreads();
  best = sv[0];
  bi = si[0];
  __syncthreads();
}

// Per-head top-k in two steps.  Step 1: the vocabulary is cut into kTopkChunks chunks and one CTA per
// (chunk, head, sequence) finds its chunk's k best in k rounds; round r only considers entries that come
// strictly after the previous winner in (value descending, id ascending) order, so nothing is modified
// in place.  The global k best are among these candidates.  Step 2: one CTA per (head, sequence) runs
// the same k rounds over the kTopkChunks * k candidates.
__global__ void __launch_bounds__(256) topk_part_kernel(const float* __restrict__ logits, int V, int Hc,
                                                        const int32_t* __restrict__ kper, float* __restrict__ cand_v,
                                                        int32_t* __restrict__ cand_i) {
  __shared__ float sv[32];
  __shared__ int si[32];
  griddep_wait();
  griddep_launch();
  const int ch = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const float* r = logits + ((size_t)b * Hc + h) * V;
  const int k = kper[h];
  const int per = (V + kTopkChunks - 1) / kTopkChunks;
  const int j0 = ch * per, j1 = min(V, j0 + per);
  float pv = INFINITY;
  int pi = -1;
  const size_t o = (((size_t)b * Hc + h) * kTopkChunks + ch) * CERB_MAX_TOPK;
  for (int round = 0; round < k; ++round) {
    float best = -INFINITY;
    int bi = 0x7fffffff;
    for (int j = j0 + threadIdx.x; j < j1; j += blockDim.x) {
      const float v = r[j];
      const bool after = v < pv || (v == pv && j > pi);
      if (after && better(v, j, best, bi)) { best = v; bi = j; }
    }
    block_best(best, bi, sv, si);
    pv = best;
    pi = bi;
    if (threadIdx.x == 0) {
      cand_v[o + round] = best;
      cand_i[o + round] = bi == 0x7fffffff ? -1 : bi;
    }
  }
}

__global__ void __launch_bounds__(256) topk_merge_kernel(const float* __restrict__ cand_v, const int32_t* __restrict__ cand_i,
                                                         int Hc, const int32_t* __restrict__ kper, int32_t* __restrict__ topk,
                                                         int32_t* __restrict__ topk_copy) {
  __shared__ float sv[32];
  __shared__ int si[32];
  griddep_wait();
  griddep_launch();
  const int h = blockIdx.x, b = blockIdx.y;
  const int k = kper[h];
  const size_t base = ((size_t)b * Hc + h) * kTopkChunks * CERB_MAX_TOPK;
  // candidate of this thread: (chunk, round) = (t / MAX_TOPK, t % MAX_TOPK)
  float cv = -INFINITY;
  int ci = 0x7fffffff;
  const int t = threadIdx.x;
  if (t < kTopkChunks * CERB_MAX_TOPK && (t % CERB_MAX_TOPK) < k) {
    const int id = cand_i[base + t];
    if (id >= 0) { cv = cand_v[base + t]; ci = id; }
  }
  float pv = INFINITY;
  int pi = -1;
  for (int round = 0; round < CERB_MAX_TOPK; ++round) {
    int32_t res = -1;
    if (round < k) {
      const bool after = ci != 0x7fffffff && (cv < pv || (cv == pv && ci > pi));
      float best = after ? cv : -INFINITY;
      int bi = after ? ci : 0x7fffffff;
      block_best(best, bi, sv, si);
      pv = best;
      pi = bi;
      res = pi == 0x7fffffff ? -1 : pi;
    }
    if (threadIdx.x == 0) {
      const size_t o = ((size_t)b * Hc + h) * CERB_MAX_TOPK + round;
      topk[o] = res;
      if (topk_copy) topk_copy[o] = res;
    }
  }
}

__global__ void tree_fill_kernel(const int32_t* __restrict__ root, const int32_t* __restrict__ topk,
                                 const int32_t* __restrict__ head_of, const int32_t* __restrict__ rank_of,
                                 const int32_t* __restrict__ plant, int Hc, int n, int32_t* __restrict__ tree_tok) {
  griddep_wait();
  griddep_launch();
  int b = blockIdx.x;
  for (int v = threadIdx.x; v < n; v += blockDim.x) {
    int t;
    if (v == 0) t = root[b];
    else {
      t = topk[((size_t)b * Hc + head_of[v]) * CERB_MAX_TOPK + rank_of[v]];
      if (plant && plant[(size_t)b * n + v] >= 0) t = plant[(size_t)b * n + v];
    }
    tree_tok[(size_t)b * n + v] = t;
  }
}

template <typename T>
int launch_level(cerb_ctx* c, const LevelParams& P, int max_rows, int max_w, cudaStream_t st) {
  dim3 grid((max_rows + ROWS_PER_BLOCK - 1) / ROWS_PER_BLOCK, P.Hc);
  size_t smem1 = (size_t)max_w * sizeof(float);
  static bool configured = false;
  if (!configured) {
    CERB_CUDA_OK(cudaFuncSetAttribute(head_gemv_kernel<T, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    CERB_CUDA_OK(cudaFuncSetAttribute(head_gemv_kernel<T, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    configured = true;
  }
  LevelParams Q = P;
  if (P.B == 1) {
    Q.b0 = 0;
    launch_pdl(head_gemv_kernel<T, 1>, grid, dim3(WARPS * 32), smem1, st, Q);
    CERB_LAUNCH_CHECK(c);
  } else {
    if (smem1 * 4 > 200 * 1024) return CERB_E_SHAPE;
    for (int b0 = 0; b0 < P.B; b0 += 4) {
      Q.b0 = b0;
      launch_pdl(head_gemv_kernel<T, 4>, grid, dim3(WARPS * 32), smem1 * 4, st, Q);
      CERB_LAUNCH_CHECK(c);
    }
  }
  return CERB_OK;
}

}  // namespace

int launch_heads(cerb_ctx* c, const cerb_tree* tree, int32_t* tree_tok, const int32_t* plant, int32_t* topk_out,
                 float* logits_out, cudaStream_t st) {
  const cerb_config& g = c->cfg;
  const int Hc = g.n_cheads, L = g.n_levels, d = g.d_model, B = c->B;
  if (Hc <= 0) return CERB_E_STATE;
  if (c->bf16) launch_pdl(head_init_kernel<bf16>, dim3(B, Hc), dim3(256), 0, st, (const bf16*)c->d_hlast, c->d_hstate[0], Hc, c->head_wmax, d);
  else launch_pdl(head_init_kernel<float>, dim3(B, Hc), dim3(256), 0, st, (const float*)c->d_hlast, c->d_hstate[0], Hc, c->head_wmax, d);
  CERB_LAUNCH_CHECK(c);
  for (int j = 0; j <= L; ++j) {
    LevelParams P;
    P.state_in = c->d_hstate[j & 1];
    P.Hc = Hc; P.wmax = c->head_wmax; P.B = B; P.b0 = 0;
    int max_rows = 0, max_w = 0;
    for (int h = 0; h < Hc; ++h) {
      HeadJob& J = P.job[h];
      if (j < L) {
        int src = g.concat_src[h][j];
        J.W = c->head_W[h * L + j];
        J.bias = c->head_b[h * L + j];
        J.w0 = c->head_w[h][j];
        J.w1 = src >= 0 ? c->head_w[src][j] : 0;
        J.src = src;
        J.rows = J.w0 + J.w1;
      } else {
        J.W = c->head_fc[h];
        J.bias = nullptr;
        J.w0 = c->head_w[h][L];
        J.w1 = 0;
        J.src = -1;
        J.rows = g.vocab;
      }
      if (J.rows > max_rows) max_rows = J.rows;
      if (J.w0 + J.w1 > max_w) max_w = J.w0 + J.w1;
    }
    if (j < L) { P.out = c->d_hstate[(j + 1) & 1]; P.out_stride = c->head_wmax; P.epilogue = 1; }
    else { P.out = logits_out ? logits_out : c->d_hlogits; P.out_stride = g.vocab; P.epilogue = 0; }
    if (c->bf16) CERB_TRY(launch_level<bf16>(c, P, max_rows, max_w, st));
    else CERB_TRY(launch_level<float>(c, P, max_rows, max_w, st));
  }
  const float* lg = logits_out ? logits_out : c->d_hlogits;
  static_assert(kTopkChunks * CERB_MAX_TOPK <= 256, "one candidate per thread in the merge");
  launch_pdl(topk_part_kernel, dim3(kTopkChunks, Hc, B), dim3(256), 0, st, lg, g.vocab, Hc, (const int32_t*)c->d_kper, c->d_topk_cv, c->d_topk_ci);
  CERB_LAUNCH_CHECK(c);
  launch_pdl(topk_merge_kernel, dim3(Hc, B), dim3(256), 0, st, (const float*)c->d_topk_cv, (const int32_t*)c->d_topk_ci, Hc, (const int32_t*)c->d_kper, c->d_topk, topk_out);
  CERB_LAUNCH_CHECK(c);
  if (tree_tok) {
    launch_pdl(tree_fill_kernel, dim3(B), dim3(128), 0, st, (const int32_t*)c->d_root, (const int32_t*)c->d_topk,
               (const int32_t*)tree->dev.head_of, (const int32_t*)tree->dev.rank_of, plant, Hc, tree->n, tree_tok);
    CERB_LAUNCH_CHECK(c);
  }
  return CERB_OK;
}

}  // namespace cerb
