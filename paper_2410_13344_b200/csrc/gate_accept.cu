// Entropy gate (Section 4.2) and greedy acceptance with KV compaction (Section 3.1).
#include "cerb_internal.cuh"

namespace cerb {

namespace {

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<bf16>(const bf16* p) { return __bfloat162float(*p); }

__device__ __forceinline__ float block_reduce(float v, float* red, bool is_max) {
  for (int o = 16; o > 0; o >>= 1) {
    float t = __shfl_xor_sync(0xffffffffu, v, o);
    v = is_max ? fmaxf(v, t) : v + t;
  }
  int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  float r = red[0];
  for (int i = 1; i < nw; ++i) r = is_max ? fmaxf(r, red[i]) : r + red[i];
  return r;
}

// P = Softmax(h_last) over the d_model components; S = -sum P log2 P.
// With m = max h, Z = sum e^(h-m), A = sum e^(h-m) (h-m):  S = (ln Z - A / Z) / ln 2.
// mode = S > T ? auto-regressive : parallel (Algorithm 1).
template <typename T>
__global__ void __launch_bounds__(256) gate_kernel(const T* __restrict__ h_last, int d, float thr, float* __restrict__ S,
                                                   int32_t* __restrict__ mode, int32_t* __restrict__ n_active, int n_par) {
  __shared__ float red[32];
  griddep_wait();
  griddep_launch();
  const T* h = h_last + (size_t)blockIdx.x * d;
  float m = -INFINITY;
  for (int j = threadIdx.x; j < d; j += blockDim.x) m = fmaxf(m, ldf(h + j));
  m = block_reduce(m, red, true);
  float z = 0.f, a = 0.f;
  for (int j = threadIdx.x; j < d; j += blockDim.x) {
    float t = ldf(h + j) - m, e = expf(t);
    z += e;
    a += e * t;
  }
  z = block_reduce(z, red, false);
  a = block_reduce(a, red, false);
  if (threadIdx.x == 0) {
    float s = (logf(z) - a / z) * 1.4426950408889634f;
    int md = s > thr ? CERB_MODE_AR : CERB_MODE_PAR;
    S[blockIdx.x] = s;
    mode[blockIdx.x] = md;
    if (n_active) n_active[blockIdx.x] = md == CERB_MODE_AR ? 1 : n_par;
  }
}

// One CTA of 192 threads (CERB_MAX_NODES) per sequence, thread v <-> node v.
//   match[v] = token of v equals the model's argmax at v's parent   (root: always)
//   v is accepted-reachable iff every node on its root path matches: (anc[v] & ~match) == 0
//   winner = deepest reachable node, lowest index among equals; its ancestors, ascending, are the path.
template <typename T>
__global__ void __launch_bounds__(CERB_MAX_NODES) accept_kernel(const int32_t* __restrict__ tok, const int32_t* __restrict__ argmax,
                                                     const int32_t* __restrict__ n_active,
                                                     const int32_t* __restrict__ parent, const int32_t* __restrict__ depth,
                                                     const uint64_t* __restrict__ anc, int n, int32_t* __restrict__ len,
                                                     int32_t* __restrict__ len_old, int32_t* __restrict__ root,
                                                     const T* __restrict__ hidden, T* __restrict__ h_last, int d,
                                                     int32_t* __restrict__ n_accept, int32_t* __restrict__ path,
                                                     int32_t* __restrict__ out_tok, const int32_t* __restrict__ row_off) {
  constexpr int NWARP = CERB_MAX_NODES / 32;
  __shared__ uint32_t mword[NWARP];
  __shared__ int skey[NWARP];
  __shared__ int best_s;
  griddep_wait();
  griddep_launch();
  const int b = blockIdx.x, v = threadIdx.x;
  const int na = min(n_active[b], n);
  const int32_t* tk = tok + (size_t)b * n;
  const size_t row0 = row_off ? (size_t)row_off[b] : (size_t)b * n;      // this sequence's first row of argmax / hidden
  const int32_t* am = argmax + row0;
  bool match = v < na && (v == 0 || tk[v] == am[parent[v]]);
  uint32_t bal = __ballot_sync(0xffffffffu, match);
  if ((v & 31) == 0) mword[v >> 5] = bal;
  __syncthreads();
  uint64_t mm[CERB_ANC_WORDS];
#pragma unroll
  for (int w = 0; w < CERB_ANC_WORDS; ++w) mm[w] = (uint64_t)mword[2 * w] | ((uint64_t)mword[2 * w + 1] << 32);
  int key = -1;
  if (v < na) {
    bool reach = true;
#pragma unroll
    for (int w = 0; w < CERB_ANC_WORDS; ++w) reach = reach && (anc[v * CERB_ANC_WORDS + w] & ~mm[w]) == 0;
    if (reach) key = depth[v] * 256 + (255 - v);
  }
  for (int o = 16; o > 0; o >>= 1) key = max(key, __shfl_xor_sync(0xffffffffu, key, o));
  if ((v & 31) == 0) skey[v >> 5] = key;
  __syncthreads();
  if (v == 0) {
    int k = skey[0];
#pragma unroll
    for (int w = 1; w < NWARP; ++w) k = max(k, skey[w]);
    int best = k < 0 ? 0 : 255 - (k & 255);
    best_s = best;
    int cnt = 0;
    for (int w = 0; w < CERB_ANC_WORDS; ++w) {
      uint64_t bits = anc[best * CERB_ANC_WORDS + w];
      while (bits && cnt < kPathMax) {
        int j = __ffsll((long long)bits) - 1;
        bits &= bits - 1;
        path[(size_t)b * kPathMax + cnt] = w * 64 + j;
        out_tok[(size_t)b * kPathMax + cnt] = tk[w * 64 + j];
        ++cnt;
      }
    }
    for (int j = cnt; j < kPathMax; ++j) { path[(size_t)b * kPathMax + j] = -1; out_tok[(size_t)b * kPathMax + j] = -1; }
    n_accept[b] = cnt;
    root[b] = am[best];
    int L = len[b];
    len_old[b] = L;
    len[b] = L + cnt;
  }
  __syncthreads();
  const T* src = hidden + (row0 + best_s) * d;
  for (int j = threadIdx.x; j < d; j += blockDim.x) h_last[(size_t)b * d + j] = src[j];
}

// Move the accepted nodes' K/V from slot L + path[j] to slot L + j in every layer.  One thread owns
// one 16-byte column chunk of one (layer, K|V, head) and loads all path rows before storing any:
// path[j] >= j, so a destination may be a later source.
__global__ void kv_compact_kernel(char* __restrict__ kpool, char* __restrict__ vpool, size_t layer_bytes,
                                  const int32_t* __restrict__ page_table, int max_pages,
                                  const int32_t* __restrict__ len_old, const int32_t* __restrict__ n_accept,
                                  const int32_t* __restrict__ path, int H, int row_bytes) {
  griddep_wait();
  griddep_launch();
  const int b = blockIdx.z, layer = blockIdx.y >> 1;
  char* pool = ((blockIdx.y & 1) ? vpool : kpool) + (size_t)layer * layer_bytes;
  const int chunks = row_bytes / 16;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= H * chunks) return;
  const int h = idx / chunks, ch = idx % chunks;
  const int cnt = n_accept[b], L = len_old[b];
  const int32_t* pt = page_table + (size_t)b * max_pages;
  uint4 regs[kPathMax];
  bool moved[kPathMax];
#pragma unroll
  for (int j = 0; j < kPathMax; ++j) {
    moved[j] = false;
    if (j < cnt) {
      int pj = path[(size_t)b * kPathMax + j];
      if (pj != j) {
        int slot = L + pj;
        size_t off = (((size_t)pt[slot / CERB_PAGE] * H + h) * CERB_PAGE + slot % CERB_PAGE) * row_bytes + (size_t)ch * 16;
        regs[j] = *reinterpret_cast<const uint4*>(pool + off);
        moved[j] = true;
      }
    }
  }
#pragma unroll
  for (int j = 0; j < kPathMax; ++j) {
    if (moved[j]) {
      int slot = L + j;
      size_t off = (((size_t)pt[slot / CERB_PAGE] * H + h) * CERB_PAGE + slot % CERB_PAGE) * row_bytes + (size_t)ch * 16;
      *reinterpret_cast<uint4*>(pool + off) = regs[j];
    }
  }
}

}  // namespace

int launch_gate(cerb_ctx* c, float T, float* S, int32_t* mode, int32_t* nactive_or_null, int n_par, cudaStream_t st) {
  int d = c->cfg.d_model;
  if (c->bf16) gate_kernel<bf16><<<c->B, 256, 0, st>>>((const bf16*)c->d_hlast, d, T, S, mode, nactive_or_null, n_par);
  else gate_kernel<float><<<c->B, 256, 0, st>>>((const float*)c->d_hlast, d, T, S, mode, nactive_or_null, n_par);
  CERB_LAUNCH_CHECK(c);
  return CERB_OK;
}

int launch_accept(cerb_ctx* c, const cerb_tree* tree, const int32_t* tree_tok, const int32_t* n_active,
                  const int32_t* node_argmax, int32_t* n_accept, int32_t* path, int32_t* out_tok, cudaStream_t st,
                  const int32_t* row_off) {
  const cerb_config& g = c->cfg;
  const TreeDev& t = tree->dev;
  if (c->bf16)
    accept_kernel<bf16><<<c->B, CERB_MAX_NODES, 0, st>>>(tree_tok, node_argmax, n_active, t.parent, t.depth, t.anc, tree->n, c->d_len,
                                              c->d_len_old, c->d_root, (const bf16*)c->d_hidden, (bf16*)c->d_hlast,
                                              g.d_model, n_accept, path, out_tok, row_off);
  else
    accept_kernel<float><<<c->B, CERB_MAX_NODES, 0, st>>>(tree_tok, node_argmax, n_active, t.parent, t.depth, t.anc, tree->n, c->d_len,
                                               c->d_len_old, c->d_root, (const float*)c->d_hidden, (float*)c->d_hlast,
                                               g.d_model, n_accept, path, out_tok, row_off);
  CERB_LAUNCH_CHECK(c);
  if (tree->n > 1) {
    int row_bytes = g.head_dim * (int)c->esize;
    int threads = g.n_heads * (row_bytes / 16);
    dim3 grid((threads + 127) / 128, g.n_layers * 2, c->B);
    kv_compact_kernel<<<grid, 128, 0, st>>>(c->k_pool, c->v_pool, c->pool_layer_bytes, c->page_table, g.max_pages,
                                            c->d_len_old, n_accept, path, g.n_heads, row_bytes);
    CERB_LAUNCH_CHECK(c);
  }
  return CERB_OK;
}

}  // namespace cerb
