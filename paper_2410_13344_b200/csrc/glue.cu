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

template <typename T> __device__ __forceinline__ void ld4(const T* p, float* f);
template <> __device__ __forceinline__ void ld4<float>(const float* p, float* f) {
  float4 v = *reinterpret_cast<const float4*>(p);
  f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}
template <> __device__ __forceinline__ void ld4<bf16>(const bf16* p, float* f) {
  uint2 v = *reinterpret_cast<const uint2*>(p);
  float2 a = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&v.x)), b = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&v.y));
  f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
}
template <typename T> __device__ __forceinline__ void st4(T* p, const float* f);
template <> __device__ __forceinline__ void st4<float>(float* p, const float* f) {
  *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
}
template <> __device__ __forceinline__ void st4<bf16>(bf16* p, const float* f) {
  __nv_bfloat162 a = __floats2bfloat162_rn(f[0], f[1]), b = __floats2bfloat162_rn(f[2], f[3]);
  uint2 v;
  v.x = *reinterpret_cast<uint32_t*>(&a);
  v.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = v;
}
// One row per CTA, four consecutive columns per thread:
//   x <- (embedding row | x | x + sum of GEMM partial slots), kept in fp32 (the residual stream is never rounded);
//   out <- RMSNorm(x) * gain, in the model's storage type.
// Fusing the residual add (and the first layer's embedding gather) with the norm that always follows
// it halves the element-wise launches; the slot loads of a thread are independent 16-byte loads.
constexpr int NORM_THREADS = 1024;
constexpr int NORM_MAX_ITER = 4;          // d_model up to 16384
template <typename T>
__global__ void __launch_bounds__(NORM_THREADS) fused_norm_kernel(float* __restrict__ x, const float* __restrict__ part, int nsplit,
                                                                   size_t split_stride, const T* __restrict__ embed,
                                                                   const int32_t* __restrict__ tok, int tok_stride, int tok_off,
                                                                   const int32_t* __restrict__ n_active, int n, int V,
                                                                   const T* __restrict__ gain, T* __restrict__ out, int d, float eps,
                                                                   const int32_t* __restrict__ row_off, int B) {
  __shared__ float red[32];
  const int row = blockIdx.x;
  float* xr = x + (size_t)row * d;
  // The residual stream was last written by the previous norm (at least two kernels ago) and the gains
  // never change: both are fetched before waiting for the kernel in front (a GEMM, or whatever produced
  // the token ids), so that after the wait only that kernel's output remains to be read.
  float keep[NORM_MAX_ITER][4], gv[NORM_MAX_ITER][4];
#pragma unroll
  for (int it = 0; it < NORM_MAX_ITER; ++it) {
    const int j = (it * NORM_THREADS + threadIdx.x) * 4;
    if (j < d) {
      if (!embed) ld4(xr + j, keep[it]);
      if (out) ld4(gain + j, gv[it]);
    }
  }
  griddep_wait();
  griddep_launch();
  const T* src = nullptr;
  if (embed) {
    int b, v, t = 0;
    locate_row(row, row_off, B, n, b, v);
    if (v < n_active[b]) t = tok[(size_t)b * tok_stride + tok_off + v];
    if (t < 0 || t >= V) t = 0;
    src = embed + (size_t)t * d;
  }
  float ss = 0.f;
#pragma unroll
  for (int it = 0; it < NORM_MAX_ITER; ++it) {
    const int j = (it * NORM_THREADS + threadIdx.x) * 4;
    if (j < d) {
      float v[4];
      if (src) ld4(src + j, v);
      else {
#pragma unroll
        for (int e = 0; e < 4; ++e) v[e] = keep[it][e];
      }
      if (nsplit > 0) {
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        const float* pr = part + (size_t)row * d + j;
#pragma unroll 4
        for (int s = 0; s < nsplit; ++s) {
          float4 t4 = *reinterpret_cast<const float4*>(pr + s * split_stride);
          a.x += t4.x; a.y += t4.y; a.z += t4.z; a.w += t4.w;
        }
        v[0] += a.x; v[1] += a.y; v[2] += a.z; v[3] += a.w;
      }
      if (embed || nsplit > 0) st4(xr + j, v);
#pragma unroll
      for (int e = 0; e < 4; ++e) { keep[it][e] = v[e]; ss += v[e] * v[e]; }
    }
  }
  ss = block_sum(ss, red);
  if (!out) return;
  const float r = 1.0f / sqrtf(ss / (float)d + eps);
  T* o = out + (size_t)row * d;
#pragma unroll
  for (int it = 0; it < NORM_MAX_ITER; ++it) {
    const int j = (it * NORM_THREADS + threadIdx.x) * 4;
    if (j < d) {
      float ov[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) ov[e] = keep[it][e] * r * gv[it][e];
      st4(o + j, ov);
    }
  }
}

// q,k rotated at position len + depth; k,v stored at slot len + node of the paged pools; q kept dense.
// One CTA per (row, head), one thread per rotation pair.
template <typename T>
__global__ void rope_append_kernel(const float* __restrict__ part, int nsplit, size_t split_stride,
                                   const int32_t* __restrict__ len, const int32_t* __restrict__ n_active,
                                   const int32_t* __restrict__ depth, const int32_t* __restrict__ page_table,
                                   int max_pages, const float2* __restrict__ rope, int max_pos, int n, int H, int Dh,
                                   T* __restrict__ q, T* __restrict__ kpool, T* __restrict__ vpool,
                                   const int32_t* __restrict__ row_off, int B) {
  // Lengths, live node counts, the tree, the page table and the rotation table are at least two kernels
  // old: the chain of dependent index loads runs before the wait for the QKV GEMM in front.
  const int row = blockIdx.x, h = blockIdx.y;
  int b, v;
  locate_row(row, row_off, B, n, b, v);          // (the row offsets come from the host, before the step's first kernel)
  const int HD = H * Dh, half = Dh >> 1;
  const bool active = v < n_active[b];
  const int L = len[b];
  const int pos = L + depth[v], slot = L + v;
  const bool ok = active && pos < max_pos && slot < max_pos;
  const int page = ok ? page_table[(size_t)b * max_pages + slot / CERB_PAGE] : 0;
  const float2 cs0 = (ok && (int)threadIdx.x < half) ? rope[(size_t)pos * half + threadIdx.x] : make_float2(1.f, 0.f);
  griddep_wait();
  griddep_launch();
  if (!ok) return;
  const size_t kv = (((size_t)page * H + h) * CERB_PAGE + (size_t)(slot % CERB_PAGE)) * Dh;
  const float* pr = part + (size_t)row * 3 * HD + h * Dh;
  for (int i = threadIdx.x; i < half; i += blockDim.x) {
    float2 cs = i == (int)threadIdx.x ? cs0 : rope[(size_t)pos * half + i];
    float q1 = 0.f, q2 = 0.f, k1 = 0.f, k2 = 0.f, v1 = 0.f, v2 = 0.f;
    for (int s = 0; s < nsplit; ++s) {
      const float* p = pr + s * split_stride + i;
      q1 += p[0]; q2 += p[half]; k1 += p[HD]; k2 += p[HD + half]; v1 += p[2 * HD]; v2 += p[2 * HD + half];
    }
    T* qo = q + (size_t)row * HD + h * Dh + i;
    stf(qo, q1 * cs.x - q2 * cs.y);
    stf(qo + half, q2 * cs.x + q1 * cs.y);
    stf(kpool + kv + i, k1 * cs.x - k2 * cs.y);
    stf(kpool + kv + i + half, k2 * cs.x + k1 * cs.y);
    stf(vpool + kv + i, v1);
    stf(vpool + kv + i + half, v2);
  }
}

template <typename T>
__global__ void swiglu_kernel(const float* __restrict__ part, int nsplit, size_t split_stride, T* __restrict__ act,
                              int rows, int F) {
  griddep_wait();
  griddep_launch();
  const int F4 = F >> 2;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (size_t)rows * F4) return;
  size_t row = i / F4, j = (i % F4) * 4;
  float4 g = make_float4(0.f, 0.f, 0.f, 0.f), u = g;
  for (int s = 0; s < nsplit; ++s) {
    const float* p = part + s * split_stride + row * 2 * F;
    float4 a = *reinterpret_cast<const float4*>(p + j), c = *reinterpret_cast<const float4*>(p + F + j);
    g.x += a.x; g.y += a.y; g.z += a.z; g.w += a.w;
    u.x += c.x; u.y += c.y; u.z += c.z; u.w += c.w;
  }
  T* o = act + row * F + j;
  stf(o, g.x / (1.0f + expf(-g.x)) * u.x);
  stf(o + 1, g.y / (1.0f + expf(-g.y)) * u.y);
  stf(o + 2, g.z / (1.0f + expf(-g.z)) * u.z);
  stf(o + 3, g.w / (1.0f + expf(-g.w)) * u.w);
}

// Row argmax over logits given as split-K partial sums; ties go to the lower index.  When
// `summed` is not null the summed logits are also written there ([rows][V]).
__global__ void argmax_rows_kernel(const float* __restrict__ part, int nsplit, size_t split_stride, int V,
                                   int32_t* __restrict__ out, float* __restrict__ summed) {
  __shared__ float sv[32];
  __shared__ int si[32];
  griddep_wait();
  griddep_launch();
  const float* r = part + (size_t)blockIdx.x * V;
  float best = -INFINITY;
  int bi = 0x7fffffff;
  if ((V & 3) == 0 && (split_stride & 3) == 0) {
    // 16-byte loads, two column groups per thread in flight: the kernel is pure load latency
    const int V4 = V >> 2;
#pragma unroll 2
    for (int j4 = threadIdx.x; j4 < V4; j4 += blockDim.x) {
      float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
      for (int s = 0; s < nsplit; ++s) {
        const float4 t = *reinterpret_cast<const float4*>(r + s * split_stride + 4 * j4);
        a.x += t.x; a.y += t.y; a.z += t.z; a.w += t.w;
      }
      if (summed) *reinterpret_cast<float4*>(summed + (size_t)blockIdx.x * V + 4 * j4) = a;
      const int j = 4 * j4;                       // ascending ids: a later equal value never replaces an earlier one
      if (a.x > best) { best = a.x; bi = j; }
      if (a.y > best) { best = a.y; bi = j + 1; }
      if (a.z > best) { best = a.z; bi = j + 2; }
      if (a.w > best) { best = a.w; bi = j + 3; }
    }
  } else {
    for (int j = threadIdx.x; j < V; j += blockDim.x) {
      float v = 0.f;
      for (int s = 0; s < nsplit; ++s) v += r[s * split_stride + j];
      if (summed) summed[(size_t)blockIdx.x * V + j] = v;
      if (v > best || (v == best && j < bi)) { best = v; bi = j; }
    }
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
  griddep_wait();
  griddep_launch();
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
  griddep_wait();
  griddep_launch();
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

// x <- embedding rows (tok != null) | x + partials (nsplit > 0) | x;  out <- RMSNorm(x) * gain (out may be null).
int launch_fused_norm(cerb_ctx* c, const float* part, int nsplit, size_t split_stride, const int32_t* tok, int tok_stride,
                      int tok_off, int n, const void* gain, void* out, int rows, cudaStream_t st, const int32_t* row_off) {
  const cerb_config& g = c->cfg;
  const int d = g.d_model;
  if (d % 4 || d > NORM_THREADS * NORM_MAX_ITER * 4) return CERB_E_SHAPE;
  if (c->bf16)
    launch_pdl(fused_norm_kernel<bf16>, dim3(rows), dim3(NORM_THREADS), 0, st, (float*)c->d_x, part, nsplit, split_stride,
               tok ? (const bf16*)c->embed : (const bf16*)nullptr, tok, tok_stride, tok_off, (const int32_t*)c->d_nactive, n,
               g.vocab, (const bf16*)gain, (bf16*)out, d, g.rms_eps, row_off, c->B);
  else
    launch_pdl(fused_norm_kernel<float>, dim3(rows), dim3(NORM_THREADS), 0, st, (float*)c->d_x, part, nsplit, split_stride,
               tok ? (const float*)c->embed : (const float*)nullptr, tok, tok_stride, tok_off, (const int32_t*)c->d_nactive, n,
               g.vocab, (const float*)gain, (float*)out, d, g.rms_eps, row_off, c->B);
  CERB_LAUNCH_CHECK(c);
  return CERB_OK;
}

int launch_rope_append(cerb_ctx* c, int layer, const TreeDev& t, const float* part, int nsplit, size_t split_stride,
                       int B, int n, int rows, cudaStream_t st, const int32_t* row_off) {
  const cerb_config& g = c->cfg;
  char* kp = c->k_pool + (size_t)layer * c->pool_layer_bytes;
  char* vp = c->v_pool + (size_t)layer * c->pool_layer_bytes;
  if (c->bf16)
    launch_pdl(rope_append_kernel<bf16>, dim3(rows, g.n_heads), dim3(64), 0, st, part, nsplit, split_stride,
               (const int32_t*)c->d_len, (const int32_t*)c->d_nactive, (const int32_t*)t.depth, c->page_table, g.max_pages,
               (const float2*)c->d_rope, c->max_pos, n, g.n_heads, g.head_dim, (bf16*)c->d_q, (bf16*)kp, (bf16*)vp, row_off, B);
  else
    launch_pdl(rope_append_kernel<float>, dim3(rows, g.n_heads), dim3(64), 0, st, part, nsplit, split_stride,
               (const int32_t*)c->d_len, (const int32_t*)c->d_nactive, (const int32_t*)t.depth, c->page_table, g.max_pages,
               (const float2*)c->d_rope, c->max_pos, n, g.n_heads, g.head_dim, (float*)c->d_q, (float*)kp, (float*)vp, row_off, B);
  CERB_LAUNCH_CHECK(c);
  return CERB_OK;
}

int launch_swiglu(cerb_ctx* c, const float* part, int nsplit, size_t split_stride, void* act, int rows, cudaStream_t st) {
  int F = c->cfg.mlp_dim;
  size_t total = (size_t)rows * (F / 4);
  unsigned blocks = (unsigned)((total + 255) / 256);
  if (c->bf16) launch_pdl(swiglu_kernel<bf16>, dim3(blocks), dim3(256), 0, st, part, nsplit, split_stride, (bf16*)act, rows, F);
  else launch_pdl(swiglu_kernel<float>, dim3(blocks), dim3(256), 0, st, part, nsplit, split_stride, (float*)act, rows, F);
  CERB_LAUNCH_CHECK(c);
  return CERB_OK;
}

int launch_argmax_rows(cerb_ctx* c, const float* part, int nsplit, size_t split_stride, int rows, int V, int32_t* out,
                       float* summed, cudaStream_t st) {
  launch_pdl(argmax_rows_kernel, dim3(rows), dim3(1024), 0, st, part, nsplit, split_stride, V, out, summed);
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
