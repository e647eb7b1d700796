// Small element-wise kernels of the base-model forward (Algorithm 1: embedding, TL_i, LH):
// embedding gather, RMSNorm, RoPE + KV-page append, residual add, SwiGLU, row argmax.
// GEMM outputs arrive as fp32 split-K partial sums [split][row][col]; every consumer here
// adds the splits in index order, so results do not depend on scheduling.
#include "cerb_internal.cuh"

namespace cerb {

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<bf16>(const bf16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void stf(T* p, float v);
template <> __device__ __forceinline__ void stf<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void stf<bf16>(bf16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float block_sum(float v, float* red) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  float t = 0.f;
  for (int i = 0; i < nw; ++i) t += red[i];
  return t;
}

// cos/sin of pos * base^(-2i/Dh), evaluated once in double precision.
__global__ void rope_table_kernel(float2* tab, int max_pos, int half, double base) {
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= max_pos * half) return;
  int pos = idx / half, i = idx % half;
  double inv = pow(base, -2.0 * (double)i / (double)(2 * half));
  double s, c;
  sincos((double)pos * inv, &s, &c);
  tab[idx] = make_float2((float)c, (float)s);
}

template <typename T>
__global__ void embed_kernel(const T* __restrict__ embed, const int32_t* __restrict__ tok, int tok_stride, int tok_off,
                             const int32_t* __restrict__ n_active, int n, int d, int V, T* __restrict__ x) {
  int row = blockIdx.x, b = row / n, v = row % n;
  int t = 0;
  if (v < n_active[b]) t = tok[(size_t)b * tok_stride + tok_off + v];
  if (t < 0 || t >= V) t = 0;
  const T* src = embed + (size_t)t * d;
  T* dst = x + (size_t)row * d;
  for (int j = threadIdx.x; j < d; j += blockDim.x) dst[j] = src[j];
}

template <typename T>
__global__ void rmsnorm_kernel(const T* __restrict__ x, const T* __restrict__ gain, T* __restrict__ out, int d, float eps) {
  __shared__ float red[32];
  const T* xr = x + (size_t)blockIdx.x * d;
  float ss = 0.f;
  for (int j = threadIdx.x; j < d; j += blockDim.x) { float v = ldf(xr + j); ss += v * v; }
  ss = block_sum(ss, red);
  float r = 1.0f / sqrtf(ss / (float)d + eps);
  T* o = out + (size_t)blockIdx.x * d;
  for (int j = threadIdx.x; j < d; j += blockDim.x) stf(o + j, ldf(xr + j) * r * ldf(gain + j));
}

// q,k rotated at position len + depth; k,v stored at slot len + node of the paged pools; q kept dense.
template <typename T>
__global__ void rope_append_kernel(const float* __restrict__ part, int nsplit, size_t split_stride,
                                   const int32_t* __restrict__ len, const int32_t* __restrict__ n_active,
                                   const int32_t* __restrict__ depth, const int32_t* __restrict__ page_table,
                                   int max_pages, const float2* __restrict__ rope, int max_pos, int n, int H, int Dh,
                                   T* __restrict__ q, T* __restrict__ kpool, T* __restrict__ vpool) {
  int row = blockIdx.x, b = row / n, v = row % n;
  if (v >= n_active[b]) return;
  int HD = H * Dh, half = Dh >> 1;
  int L = len[b];
  int pos = L + depth[v], slot = L + v;
  if (pos >= max_pos || slot >= max_pos) return;
  int page = page_table[(size_t)b * max_pages + slot / CERB_PAGE];
  size_t kv_base = ((size_t)page * H) * CERB_PAGE * Dh + (size_t)(slot % CERB_PAGE) * Dh;
  const float* pr = part + (size_t)row * 3 * HD;
  for (int idx = threadIdx.x; idx < H * half; idx += blockDim.x) {
    int h = idx / half, i = idx % half;
    float2 cs = rope[(size_t)pos * half + i];
    float q1 = 0.f, q2 = 0.f, k1 = 0.f, k2 = 0.f;
    for (int s = 0; s < nsplit; ++s) {
      const float* p = pr + s * split_stride + h * Dh + i;
      q1 += p[0]; q2 += p[half]; k1 += p[HD]; k2 += p[HD + half];
    }
    T* qo = q + (size_t)row * HD + h * Dh + i;
    stf(qo, q1 * cs.x - q2 * cs.y);
    stf(qo + half, q2 * cs.x + q1 * cs.y);
    T* ko = kpool + kv_base + (size_t)h * CERB_PAGE * Dh + i;
    stf(ko, k1 * cs.x - k2 * cs.y);
    stf(ko + half, k2 * cs.x + k1 * cs.y);
  }
  for (int idx = threadIdx.x; idx < HD; idx += blockDim.x) {
    int h = idx / Dh, i = idx % Dh;
    float vv = 0.f;
    for (int s = 0; s < nsplit; ++s) vv += pr[s * split_stride + 2 * HD + idx];
    stf(vpool + kv_base + (size_t)h * CERB_PAGE * Dh + i, vv);
  }
}

template <typename T>
__global__ void residual_kernel(T* __restrict__ x, const float* __restrict__ part, int nsplit, size_t split_stride,
                                size_t total) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  float a = 0.f;
  for (int s = 0; s < nsplit; ++s) a += part[s * split_stride + i];
  stf(x + i, ldf(x + i) + a);
}

template <typename T>
__global__ void swiglu_kernel(const float* __restrict__ part, int nsplit, size_t split_stride, T* __restrict__ act,
                              int rows, int F) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (size_t)rows * F) return;
  size_t row = i / F, j = i % F;
  float g = 0.f, u = 0.f;
  for (int s = 0; s < nsplit; ++s) {
    const float* p = part + s * split_stride + row * 2 * F;
    g += p[j];
    u += p[F + j];
  }
  stf(act + i, g / (1.0f + expf(-g)) * u);
}

// Row argmax over logits given as split-K partial sums; ties go to the lower index.  When
// `summed` is not null the summed logits are also written there ([rows][V]).
__global__ void argmax_rows_kernel(const float* __restrict__ part, int nsplit, size_t split_stride, int V,
                                   int32_t* __restrict__ out, float* __restrict__ summed) {
  __shared__ float sv[32];
  __shared__ int si[32];
  const float* r = part + (size_t)blockIdx.x * V;
  float best = -INFINITY;
  int bi = 0x7fffffff;
  for (int j = threadIdx.x; j < V; j += blockDim.x) {
    float v = 0.f;
    for (int s = 0; s < nsplit; ++s) v += r[s * split_stride + j];
    if (summed) summed[(size_t)blockIdx.x * V + j] = v;
    if (v > best || (v == best && j < bi)) { best = v; bi = j; }
  }
  for (int o = 16; o > 0; o >>= 1) {
    float ov = __shfl_xor_sync(0xffffffffu, best, o);
    int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
  }
  int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
  if (l == 0) { sv[w] = best; si[w] = bi; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < nw; ++i)
      if (sv[i] > best || (sv[i] == best && si[i] < bi)) { best = sv[i]; bi = si[i]; }
    out[blockIdx.x] = (bi == 0x7fffffff) ? 0 : bi;
  }
}

// mode 0: n_active[b] = a.  mode 1 (prefill chunk): n_active[b] = clamp(lens_in[b] - a, 0, b_).
__global__ void set_nactive_kernel(int32_t* n_active, const int32_t* lens_in, int B, int mode, int a, int b_) {
  int b = threadIdx.x;
  if (b >= B) return;
  if (mode == 0) n_active[b] = a;
  else {
    int r = lens_in[b] - a;
    n_active[b] = r < 0 ? 0 : (r > b_ ? b_ : r);
  }
}

// After a chain-shaped prefill chunk: everything is accepted in place.
template <typename T>
__global__ void prefill_commit_kernel(const int32_t* __restrict__ n_active, int32_t* __restrict__ len,
                                      const T* __restrict__ hidden, T* __restrict__ h_last, int n, int d) {
  int b = blockIdx.x, na = n_active[b];
  if (na <= 0) return;
  const T* src = hidden + ((size_t)b * n + na - 1) * d;
  for (int j = threadIdx.x; j < d; j += blockDim.x) h_last[(size_t)b * d + j] = src[j];
  __syncthreads();
  if (threadIdx.x == 0) len[b] += na;
}

int launch_rope_table(cerb_ctx* c, cudaStream_t st) {
  int half = c->cfg.head_dim / 2, total = c->max_pos * half;
  rope_table_kernel<<<(total + 255) / 256, 256, 0, st>>>(c->d_rope, c->max_pos, half, (double)c->cfg.rope_base);
  CERB_LAUNCH_CHECK(c);
  return CERB_OK;
}

int launch_embed(cerb_ctx* c, const int32_t* tok, int tok_stride, int tok_off, int B, int n, cudaStream_t st) {
  int d = c->cfg.d_model;
  if (c->bf16)
    embed_kernel<bf16><<<B * n, 128, 0, st>>>((const bf16*)c->embed, tok, tok_stride, tok_off, c->d_nactive, n, d,
                                              c->cfg.vocab, (bf16*)c->d_x);
  else
    embed_kernel<float><<<B * n, 128, 0, st>>>((const float*)c->embed, tok, tok_stride, tok_off, c->d_nactive, n, d,
                                               c->cfg.vocab, (float*)c->d_x);
  CERB_LAUNCH_CHECK(c);
  return CERB_OK;
}

int launch_rmsnorm(cerb_ctx* c, const void* x, const void* gain, void* out, int rows, cudaStream_t st) {
  int d = c->cfg.d_model;
  if (c->bf16)
    rmsnorm_kernel<bf16><<<rows, 256, 0, st>>>((const bf16*)x, (const bf16*)gain, (bf16*)out, d, c->cfg.rms_eps);
  else
    rmsnorm_kernel<float><<<rows, 256, 0, st>>>((const float*)x, (const float*)gain, (float*)out, d, c->cfg.rms_eps);
  CERB_LAUNCH_CHECK(c);
  return CERB_OK;
}

int launch_rope_append(cerb_ctx* c, int layer, const TreeDev& t, const float* part, int nsplit, size_t split_stride,
                       int B, int n, cudaStream_t st) {
  const cerb_config& g = c->cfg;
  char* kp = c->k_pool + (size_t)layer * c->pool_layer_bytes;
  char* vp = c->v_pool + (size_t)layer * c->pool_layer_bytes;
  if (c->bf16)
    rope_append_kernel<bf16><<<B * n, 256, 0, st>>>(part, nsplit, split_stride, c->d_len, c->d_nactive, t.depth,
                                                    c->page_table, g.max_pages, c->d_rope, c->max_pos, n, g.n_heads,
                                                    g.head_dim, (bf16*)c->d_q, (bf16*)kp, (bf16*)vp);
  else
    rope_append_kernel<float><<<B * n, 256, 0, st>>>(part, nsplit, split_stride, c->d_len, c->d_nactive, t.depth,
                                                     c->page_table, g.max_pages, c->d_rope, c->max_pos, n, g.n_heads,
                                                     g.head_dim, (float*)c->d_q, (float*)kp, (float*)vp);
  CERB_LAUNCH_CHECK(c);
  return CERB_OK;
}

int launch_residual(cerb_ctx* c, void* x, const float* part, int nsplit, size_t split_stride, int rows, int N,
                    cudaStream_t st) {
  size_t total = (size_t)rows * N;
  unsigned blocks = (unsigned)((total + 255) / 256);
  if (c->bf16) residual_kernel<bf16><<<blocks, 256, 0, st>>>((bf16*)x, part, nsplit, split_stride, total);
  else residual_kernel<float><<<blocks, 256, 0, st>>>((float*)x, part, nsplit, split_stride, total);
  CERB_LAUNCH_CHECK(c);
  return CERB_OK;
}

int launch_swiglu(cerb_ctx* c, const float* part, int nsplit, size_t split_stride, void* act, int rows, cudaStream_t st) {
  int F = c->cfg.mlp_dim;
  size_t total = (size_t)rows * F;
  unsigned blocks = (unsigned)((total + 255) / 256);
  if (c->bf16) swiglu_kernel<bf16><<<blocks, 256, 0, st>>>(part, nsplit, split_stride, (bf16*)act, rows, F);
  else swiglu_kernel<float><<<blocks, 256, 0, st>>>(part, nsplit, split_stride, (float*)act, rows, F);
  CERB_LAUNCH_CHECK(c);
  return CERB_OK;
}

int launch_argmax_rows(cerb_ctx* c, const float* part, int nsplit, size_t split_stride, int rows, int V, int32_t* out,
                       float* summed, cudaStream_t st) {
  argmax_rows_kernel<<<rows, 1024, 0, st>>>(part, nsplit, split_stride, V, out, summed);
  CERB_LAUNCH_CHECK(c);
  return CERB_OK;
}

int launch_set_nactive(cerb_ctx* c, int mode, int a, int b, cudaStream_t st) {
  set_nactive_kernel<<<1, 32, 0, st>>>(c->d_nactive, c->d_lens_in, c->B, mode, a, b);
  CERB_LAUNCH_CHECK(c);
  return CERB_OK;
}

int launch_prefill_commit(cerb_ctx* c, int n, cudaStream_t st) {
  int d = c->cfg.d_model;
  if (c->bf16)
    prefill_commit_kernel<bf16><<<c->B, 256, 0, st>>>(c->d_nactive, c->d_len, (const bf16*)c->d_hidden,
                                                      (bf16*)c->d_hlast, n, d);
  else
    prefill_commit_kernel<float><<<c->B, 256, 0, st>>>(c->d_nactive, c->d_len, (const float*)c->d_hidden,
                                                       (float*)c->d_hlast, n, d);
  CERB_LAUNCH_CHECK(c);
  return CERB_OK;
}

}  // namespace cerb
