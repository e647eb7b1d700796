// C ABI of the Cerberus decoding-step library: context set-up, workspace carve-out and the host
// controller that strings the kernels together (Algorithm 1).
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "cerb_internal.cuh"

using namespace cerb;

namespace cerb {
bool pdl_enabled() {
  static int v = -1;
  if (v < 0) {
    const char* e = getenv("CERB_PDL");
    v = e ? (atoi(e) != 0) : 1;
  }
  return v != 0;
}
namespace {
long long g_wait_cycles = 4000000000ll;       // about 2 s of SM clock: far beyond any legitimate wait
}
long long wait_cycles() { return g_wait_cycles; }
}  // namespace cerb

namespace {

struct Bump {
  char* base;
  size_t off;
  template <typename T>
  T* take(size_t count) {
    off = (off + 255) & ~(size_t)255;
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += count * sizeof(T);
    return p;
  }
};

inline int round_up(int v, int m) { return (v + m - 1) / m * m; }

enum { K_GEMM = 0, K_ATTN = 1, K_HEADS = 2, K_GLUE = 3, K_GATE = 4, K_ACCEPT = 5 };
constexpr size_t kProfMaxPairs = 1 << 15;

// Brackets a group of launches with two events when profiling is on; free otherwise.
struct ProfScope {
  cerb_ctx* c;
  cudaStream_t st;
  long idx;
  ProfScope(cerb_ctx* c_, int kind, cudaStream_t st_) : c(c_), st(st_), idx(-1) {
    if (!c->prof_on || c->prof_mode != 1 || c->prof_used >= kProfMaxPairs) return;
    if (c->prof_used * 2 >= c->prof_ev.size()) {
      cudaEvent_t a, b;
      if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) return;
      c->prof_ev.push_back(a);
      c->prof_ev.push_back(b);
      c->prof_kind.push_back(kind);
    }
    idx = (long)c->prof_used++;
    c->prof_kind[idx] = kind;
    cudaEventRecord(c->prof_ev[2 * idx], st);
  }
  ~ProfScope() {
    if (idx >= 0) cudaEventRecord(c->prof_ev[2 * idx + 1], st);
  }
};

int validate_config(const cerb_config* g) {
  if (!g) return CERB_E_ARG;
  if (g->dtype != CERB_F32 && g->dtype != CERB_BF16) return CERB_E_ARG;
  if (g->n_layers < 1 || g->d_model < 8 || g->n_heads < 1 || g->mlp_dim < 8 || g->vocab < 2) return CERB_E_SHAPE;
  if (g->head_dim != 64 && g->head_dim != 128) return CERB_E_SHAPE;
  if (g->d_model % 8 || g->mlp_dim % 8) return CERB_E_SHAPE;
  if (g->max_batch < 1 || g->max_batch > CERB_MAX_BATCH) return CERB_E_SHAPE;
  if (g->max_nodes < 1 || g->max_nodes > CERB_MAX_NODES) return CERB_E_SHAPE;
  if (g->max_pages < 1 || g->n_pool_pages < 1) return CERB_E_SHAPE;
  if (g->n_cheads < 0 || g->n_cheads > CERB_MAX_HEADS) return CERB_E_SHAPE;
  if (g->n_cheads > 0 && (g->n_levels < 1 || g->n_levels > CERB_MAX_LEVELS)) return CERB_E_SHAPE;
  for (int h = 0; h < g->n_cheads; ++h) {
    if (g->topk[h] < 1 || g->topk[h] > CERB_MAX_TOPK || g->topk[h] > g->vocab) return CERB_E_SHAPE;
    for (int j = 0; j < g->n_levels; ++j) {
      int s = g->concat_src[h][j];
      if (s < -1 || s >= g->n_cheads || s == h) return CERB_E_ARG;
    }
  }
  return CERB_OK;
}

void head_widths(const cerb_config* g, int w[CERB_MAX_HEADS][CERB_MAX_LEVELS + 1], int* wmax) {
  int mx = g->d_model;
  for (int h = 0; h < g->n_cheads; ++h) w[h][0] = g->d_model;
  for (int j = 0; j < g->n_levels; ++j)
    for (int h = 0; h < g->n_cheads; ++h) {
      int s = g->concat_src[h][j];
      w[h][j + 1] = w[h][j] + (s >= 0 ? w[s][j] : 0);
      if (w[h][j + 1] > mx) mx = w[h][j + 1];
    }
  *wmax = mx;
}

size_t part_floats_needed(const cerb_config* g, int Mmax, int sm_count) {
  const int HD = g->n_heads * g->head_dim;
  const int shapes[5][2] = {{3 * HD, g->d_model}, {g->d_model, HD}, {2 * g->mlp_dim, g->d_model},
                            {g->d_model, g->mlp_dim}, {g->vocab, g->d_model}};
  size_t best = 0;
  for (int i = 0; i < 5; ++i)
    for (int M = 1; M <= Mmax; ++M) {
      int ns = g->dtype == CERB_BF16 ? gemm_plan_split(sm_count, M, shapes[i][0], shapes[i][1]) : 1;
      size_t f = (size_t)ns * M * shapes[i][0];
      if (f > best) best = f;
    }
  return best;
}

// Lays the workspace out; with ctx->... pointers null-based when base == nullptr it only measures.
size_t carve(cerb_ctx* c, char* base) {
  const cerb_config& g = c->cfg;
  Bump b{base, 0};
  const int MB = CERB_MAX_BATCH, Mr = round_up(c->Mmax, 256), HD = g.n_heads * g.head_dim;
  const size_t es = c->esize;
  c->d_len = b.take<int32_t>(MB);
  c->d_len_old = b.take<int32_t>(MB);
  c->d_root = b.take<int32_t>(MB);
  c->d_nactive = b.take<int32_t>(MB);
  c->d_status = b.take<int32_t>(4);
  c->d_lens_in = b.take<int32_t>(MB);
  c->d_mode = b.take<int32_t>(MB);
  c->d_naccept = b.take<int32_t>(MB);
  c->d_kper = b.take<int32_t>(CERB_MAX_HEADS);
  c->d_rowoff = b.take<int32_t>(CERB_MAX_BATCH + 1);
  c->d_S = b.take<float>(MB);
  c->d_path = b.take<int32_t>(MB * kPathMax);
  c->d_outtok = b.take<int32_t>(MB * kPathMax);
  c->d_argmax = b.take<int32_t>(Mr);
  c->d_treetok = b.take<int32_t>(MB * CERB_MAX_NODES);
  c->d_topk = b.take<int32_t>(MB * CERB_MAX_HEADS * CERB_MAX_TOPK);
  c->d_topk_cv = b.take<float>((size_t)MB * CERB_MAX_HEADS * kTopkChunks * CERB_MAX_TOPK);
  c->d_topk_ci = b.take<int32_t>((size_t)MB * CERB_MAX_HEADS * kTopkChunks * CERB_MAX_TOPK);
  c->d_gemm_tickets = b.take<unsigned int>(kGemmTickets);
  c->d_gemm_clock = b.take<unsigned long long>(2 * kGemmClockSlots);
  c->d_hlast = b.take<char>((size_t)MB * g.d_model * es);
  c->d_x = b.take<char>((size_t)Mr * g.d_model * sizeof(float));     // residual stream, always fp32
  c->d_xn = b.take<char>((size_t)Mr * g.d_model * es);
  c->d_hidden = b.take<char>((size_t)Mr * g.d_model * es);
  c->d_q = b.take<char>((size_t)Mr * HD * es);
  c->d_attn = b.take<char>((size_t)Mr * HD * es);
  c->d_act = b.take<char>((size_t)Mr * g.mlp_dim * es);
  c->d_part = b.take<float>(c->part_floats);
  int Hc = g.n_cheads > 0 ? g.n_cheads : 1;
  c->d_hstate[0] = b.take<float>((size_t)MB * Hc * c->head_wmax);
  c->d_hstate[1] = b.take<float>((size_t)MB * Hc * c->head_wmax);
  c->d_hlogits = b.take<float>((size_t)g.max_batch * Hc * g.vocab);
  c->d_rope = b.take<float2>((size_t)c->max_pos * (g.head_dim / 2));
  c->d_attn_scratch = b.take<char>(c->attn_scratch_bytes);
  c->d_tree_store = b.take<char>((size_t)(CERB_MAX_TREES + 2) * kTreeSlotBytes);
  return (b.off + 255) & ~(size_t)255;
}

void init_sizes(cerb_ctx* c, const cerb_config* g, int sm_count) {
  c->cfg = *g;
  c->bf16 = g->dtype == CERB_BF16;
  c->esize = c->bf16 ? 2 : 4;
  // rows per sequence of one forward: the widest tree, or a prefill chunk (128 prompt tokens whatever max_nodes is)
  const int rows_seq = g->max_nodes > kPrefillChunkMax ? g->max_nodes : kPrefillChunkMax;
  c->Mmax = g->max_batch * rows_seq;
  c->max_pos = g->max_pages * CERB_PAGE;
  c->sm_count = sm_count;
  head_widths(g, c->head_w, &c->head_wmax);
  c->part_floats = part_floats_needed(g, c->Mmax, sm_count);
  c->attn_scratch_bytes = attn_scratch_bytes(g->max_batch, rows_seq, g->n_heads, g->head_dim);
}

int tree_build(cerb_ctx* c, const int32_t* parent, const int32_t* head_of, const int32_t* rank_of, int n, int slot,
               bool check_heads, bool enforce_depth, cerb_tree** out) {
  if (!parent || n < 1 || n > CERB_MAX_NODES) return CERB_E_ARG;
  cerb_tree* t = new (std::nothrow) cerb_tree();
  if (!t) return CERB_E_NOMEM;
  t->n = n;
  t->slot = slot;
  t->parent.assign(parent, parent + n);
  t->depth.assign(n, 0);
  std::vector<int32_t> hv(CERB_MAX_NODES, 0), rv(CERB_MAX_NODES, 0), pv(CERB_MAX_NODES, 0), dv(CERB_MAX_NODES, 0);
  std::vector<uint64_t> anc(CERB_MAX_NODES * CERB_ANC_WORDS, 0);
  int rc = cerb_tree_ancestors(parent, n, anc.data());
  if (rc != CERB_OK) { delete t; return rc; }
  t->max_depth = 0;
  for (int v = 0; v < n; ++v) {
    t->depth[v] = v == 0 ? 0 : t->depth[parent[v]] + 1;
    if (enforce_depth && t->depth[v] > CERB_MAX_DEPTH) { delete t; return CERB_E_ARG; }
    if (t->depth[v] > t->max_depth) t->max_depth = t->depth[v];
    pv[v] = parent[v];
    dv[v] = t->depth[v];
    if (v > 0 && check_heads) {
      if (!head_of || !rank_of) { delete t; return CERB_E_ARG; }
      int h = head_of[v], r = rank_of[v];
      if (h < 0 || h >= c->cfg.n_cheads || r < 0 || r >= c->cfg.topk[h]) { delete t; return CERB_E_ARG; }
      hv[v] = h;
      rv[v] = r;
    }
  }
  char* base = c->d_tree_store + (size_t)slot * kTreeSlotBytes;
  t->dev.parent = reinterpret_cast<int32_t*>(base);
  t->dev.depth = t->dev.parent + CERB_MAX_NODES;
  t->dev.head_of = t->dev.depth + CERB_MAX_NODES;
  t->dev.rank_of = t->dev.head_of + CERB_MAX_NODES;
  t->dev.anc = reinterpret_cast<uint64_t*>(t->dev.rank_of + CERB_MAX_NODES);
  const size_t ib = CERB_MAX_NODES * sizeof(int32_t);
  bool ok = cudaMemcpy(t->dev.parent, pv.data(), ib, cudaMemcpyHostToDevice) == cudaSuccess &&
            cudaMemcpy(t->dev.depth, dv.data(), ib, cudaMemcpyHostToDevice) == cudaSuccess &&
            cudaMemcpy(t->dev.head_of, hv.data(), ib, cudaMemcpyHostToDevice) == cudaSuccess &&
            cudaMemcpy(t->dev.rank_of, rv.data(), ib, cudaMemcpyHostToDevice) == cudaSuccess &&
            cudaMemcpy(t->dev.anc, anc.data(), CERB_MAX_NODES * CERB_ANC_WORDS * sizeof(uint64_t), cudaMemcpyHostToDevice) == cudaSuccess;
  if (!ok) { delete t; return CERB_E_CUDA; }
  *out = t;
  return CERB_OK;
}

// Device-clock profiling (mode 2): the next GEMM launch stamps its span into the next free slot.
unsigned long long* gemm_clock_slot(cerb_ctx* c) {
  if (!c->prof_on || c->prof_mode != 2 || c->gemm_clock_used >= kGemmClockSlots) return nullptr;
  return c->d_gemm_clock + c->gemm_clock_used++;
}

// out = X . W^T as fp32 split partials in d_part; returns the split count.
int gemm(cerb_ctx* c, const void* X, const ActMaps* xm, const void* W, const CUtensorMap* wm, int M, int N, int K,
         int* nsplit, cudaStream_t st) {
  if (c->bf16) {
    int ns = gemm_plan_split(c->sm_count, M, N, K);
    if ((size_t)ns * M * N > c->part_floats) return CERB_E_NOMEM;
    *nsplit = ns;
    return launch_gemm_bf16(c, wm, xm, c->d_part, M, N, K, ns, c->d_status, st, nullptr, gemm_clock_slot(c));
  }
  if ((size_t)M * N > c->part_floats) return CERB_E_NOMEM;
  *nsplit = 1;
  return launch_gemm_f32(c, (const float*)X, (const float*)W, c->d_part, M, N, K, st);
}

// Steps through the layer sequence of launch_order.cu while forward_rows launches: a kernel announced out of
// turn means the table of pre-wait reads no longer describes the code.
struct OrderCheck {
  const int* ids;
  int n, pos;
  explicit OrderCheck(int variant) : pos(0) { n = launch_order_layer(variant, &ids); }
  bool next(int id) {
    if (id == LO_NORM_FINAL) return pos == 0;
    const bool ok = ids[pos] == id;
    pos = (pos + 1) % n;
    return ok;
  }
};
#define CERB_ORDER(oc, id) do { if (!(oc).next(id)) return CERB_E_STATE; } while (0)

// The base-model forward over B*n rows (tokens tok[b*stride + off + v]); ends with the final norm
// in d_hidden.  d_nactive must already hold the live node count of every sequence.
// rows / row_off: with ragged rows (cerb_step on a batch whose sequences chose different modes) sequence b owns the
// rows row_off[b] .. row_off[b] + n_active[b] - 1 of every activation buffer and `rows` is their total; otherwise
// row_off is null and sequence b owns rows b * n .. b * n + n - 1.
// need: per sequence, how many of the n rows are live (host; a prefill chunk near the end of a prompt), or null = n.
int forward_rows(cerb_ctx* c, const cerb_tree* tree, const int32_t* tok, int tok_stride, int tok_off, int n,
                 cudaStream_t st, int rows = 0, const int32_t* row_off = nullptr, const int* need = nullptr) {
  const cerb_config& g = c->cfg;
  const int B = c->B, M = row_off ? rows : B * n, d = g.d_model, HD = g.n_heads * g.head_dim, F = g.mlp_dim;
  c->last_rows = M;
  // The host knows an upper bound of every committed length (cerb_accept adds the deepest possible path).  When
  // that bound reaches the end of the page table, the true lengths are fetched once before giving up.
  bool refreshed = false;
  int max_len = 0;
  for (int b = 0; b < B; ++b) {
    const int nb = need ? need[b] : n;
    if (c->h_len[b] + nb > c->max_pos && !refreshed) {
      int32_t tmp[CERB_MAX_BATCH];
      CERB_CUDA_OK(cudaStreamSynchronize(st));
      CERB_CUDA_OK(cudaMemcpy(tmp, c->d_len, B * sizeof(int32_t), cudaMemcpyDeviceToHost));
      for (int i = 0; i < B; ++i) c->h_len[i] = tmp[i];
      refreshed = true;
      max_len = 0;
      b = -1;
      continue;
    }
    if (c->h_len[b] + nb > c->max_pos) return CERB_E_STATE;
    if (c->h_len[b] + nb > max_len) max_len = c->h_len[b] + nb;
  }
  // Steps of up to 16 rows: SwiGLU runs in the gate-up GEMM's epilogue and (head_dim 128) RoPE + cache append in the
  // QKV GEMM's.
  const bool fuse_swiglu = c->bf16 && gemm_swiglu_fusable(M, F);
  const bool fuse_rope = fuse_swiglu && gemm_rope_fusable(M, g.head_dim);
  OrderCheck oc(fuse_rope ? 2 : fuse_swiglu ? 1 : 0);
  // embedding gather fused with the first layer's attention norm
  CERB_ORDER(oc, LO_NORM_ATTN);
  { ProfScope ps(c, K_GLUE, st);
    CERB_TRY(launch_fused_norm(c, nullptr, 0, 0, tok, tok_stride, tok_off, n, c->attn_norm[0], c->d_xn, M, st, row_off)); }
  cerb_attn_args a;
  memset(&a, 0, sizeof(a));
  a.dtype = g.dtype; a.B = B; a.n = n; a.n_heads = g.n_heads; a.head_dim = g.head_dim; a.max_pages = g.max_pages;
  a.q = c->d_q; a.page_table = c->page_table; a.len = c->d_len; a.n_active = c->d_nactive; a.anc = tree->dev.anc;
  a.out = c->d_attn; a.lse = nullptr; a.scale = 1.0f / sqrtf((float)g.head_dim); a.max_len = max_len;
  a.n_pool_pages = g.n_pool_pages; a.scratch = c->d_attn_scratch; a.scratch_bytes = c->attn_scratch_bytes;
  int ns = 1;
  for (int l = 0; l < g.n_layers; ++l) {
    a.k_pool = c->k_pool + (size_t)l * c->pool_layer_bytes;
    a.v_pool = c->v_pool + (size_t)l * c->pool_layer_bytes;
    CERB_ORDER(oc, LO_GEMM_QKV);
    if (fuse_rope) {
      // q, k and v leave the GEMM rotated and in place: no separate kernel, no second pass over the partial sums
      ProfScope ps(c, K_GEMM, st);
      const int nsl = gemm_plan_split(c->sm_count, M, 3 * HD, d);
      if ((size_t)nsl * M * 3 * HD > c->part_floats) return CERB_E_NOMEM;
      const RopeEpilogue re{c->d_len, c->d_nactive, tree->dev.depth, c->page_table, row_off, c->d_rope, c->d_q,
                            (void*)a.k_pool, (void*)a.v_pool, g.max_pages, c->max_pos, n, g.n_heads, B};
      const GemmEpilogue epi{2, nullptr, c->d_gemm_tickets, &re};
      CERB_TRY(launch_gemm_bf16(c, &c->tm_wqkv[l], &c->tm_xn, c->d_part, M, 3 * HD, d, nsl, c->d_status, st, &epi, gemm_clock_slot(c)));
    } else {
      { ProfScope ps(c, K_GEMM, st);
        CERB_TRY(gemm(c, c->d_xn, &c->tm_xn, c->wqkv[l], c->bf16 ? &c->tm_wqkv[l] : nullptr, M, 3 * HD, d, &ns, st)); }
      CERB_ORDER(oc, LO_ROPE);
      { ProfScope ps(c, K_GLUE, st); CERB_TRY(launch_rope_append(c, l, tree->dev, c->d_part, ns, (size_t)M * 3 * HD, B, n, M, st, row_off)); }
    }
    CERB_ORDER(oc, LO_ATTN);
    { ProfScope ps(c, K_ATTN, st);
      CERB_TRY(launch_tree_attention(c, &a, c->bf16 ? &c->tm_kpool[l] : nullptr, c->bf16 ? &c->tm_vpool[l] : nullptr,
                                     c->sm_count, c->d_status, st, row_off)); }
    CERB_ORDER(oc, LO_GEMM_WO);
    { ProfScope ps(c, K_GEMM, st);
      CERB_TRY(gemm(c, c->d_attn, &c->tm_attn, c->wo[l], c->bf16 ? &c->tm_wo[l] : nullptr, M, d, HD, &ns, st)); }
    // residual add fused with the MLP norm
    CERB_ORDER(oc, LO_NORM_MLP);
    { ProfScope ps(c, K_GLUE, st);
      CERB_TRY(launch_fused_norm(c, c->d_part, ns, (size_t)M * d, nullptr, 0, 0, n, c->mlp_norm[l], c->d_xn, M, st)); }
    CERB_ORDER(oc, LO_GEMM_GU);
    if (fuse_swiglu) {
      // SwiGLU runs in the GEMM's epilogue: no separate kernel, no second pass over the partial sums
      ProfScope ps(c, K_GEMM, st);
      const int nsl = gemm_plan_split(c->sm_count, M, 2 * F, d);
      if ((size_t)nsl * M * 2 * F > c->part_floats) return CERB_E_NOMEM;
      const GemmEpilogue epi{1, c->d_act, c->d_gemm_tickets};
      CERB_TRY(launch_gemm_bf16(c, &c->tm_wgu[l], &c->tm_xn, c->d_part, M, 2 * F, d, nsl, c->d_status, st, &epi, gemm_clock_slot(c)));
    } else {
      { ProfScope ps(c, K_GEMM, st);
        CERB_TRY(gemm(c, c->d_xn, &c->tm_xn, c->wgu[l], c->bf16 ? &c->tm_wgu[l] : nullptr, M, 2 * F, d, &ns, st)); }
      CERB_ORDER(oc, LO_SWIGLU);
      { ProfScope ps(c, K_GLUE, st); CERB_TRY(launch_swiglu(c, c->d_part, ns, (size_t)M * 2 * F, c->d_act, M, st)); }
    }
    CERB_ORDER(oc, LO_GEMM_DOWN);
    { ProfScope ps(c, K_GEMM, st);
      CERB_TRY(gemm(c, c->d_act, &c->tm_act, c->wd[l], c->bf16 ? &c->tm_wd[l] : nullptr, M, d, F, &ns, st)); }
    // residual add fused with the next layer's attention norm, or with the final norm
    CERB_ORDER(oc, l + 1 == g.n_layers ? LO_NORM_FINAL : LO_NORM_ATTN);
    { ProfScope ps(c, K_GLUE, st);
      const bool last = l + 1 == g.n_layers;
      CERB_TRY(launch_fused_norm(c, c->d_part, ns, (size_t)M * d, nullptr, 0, 0, n, last ? c->final_norm : c->attn_norm[l + 1],
                                 last ? c->d_hidden : c->d_xn, M, st)); }
  }
  return CERB_OK;
}

// LM head over `rows` rows of X, then row argmax (and the summed logits if asked for).
int lm_head_argmax(cerb_ctx* c, const void* X, const ActMaps* xm, int rows, int32_t* argmax_out, float* logits_out,
                   cudaStream_t st) {
  int ns = 1;
  { ProfScope ps(c, K_GEMM, st);
    CERB_TRY(gemm(c, X, xm, c->lm_head, c->bf16 ? &c->tm_lm_head : nullptr, rows, c->cfg.vocab, c->cfg.d_model, &ns, st)); }
  ProfScope ps(c, K_GLUE, st);
  return launch_argmax_rows(c, c->d_part, ns, (size_t)rows * c->cfg.vocab, rows, c->cfg.vocab, argmax_out, logits_out, st);
}

int set_active(cerb_ctx* c, const int32_t* n_active_dev, int n, cudaStream_t st) {
  if (n_active_dev) {
    CERB_CUDA_OK(cudaMemcpyAsync(c->d_nactive, n_active_dev, c->B * sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
    return CERB_OK;
  }
  return launch_set_nactive(c, 0, n, 0, st);
}

}  // namespace

extern "C" {

const char* cerb_strerror(int code) {
  switch (code) {
    case CERB_OK: return "ok";
    case CERB_E_ARG: return "invalid argument";
    case CERB_E_SHAPE: return "unsupported shape";
    case CERB_E_NOMEM: return "workspace too small or host allocation failed";
    case CERB_E_STATE: return "call out of order or sequence capacity exceeded";
    case CERB_E_NONFINITE: return "gate entropy is not finite";
    case CERB_E_TIMEOUT: return "a bounded device-side wait ran out";
    case CERB_E_CUDA: return "CUDA call failed";
    default: return "unknown error";
  }
}

int cerb_tree_ancestors(const int32_t* parent, int32_t n, uint64_t* anc_out) {
  if (!parent || !anc_out || n < 1 || n > CERB_MAX_NODES) return CERB_E_ARG;
  if (parent[0] != -1) return CERB_E_ARG;
  for (int v = 0; v < n; ++v) {
    uint64_t* mine = anc_out + (size_t)v * CERB_ANC_WORDS;
    for (int w = 0; w < CERB_ANC_WORDS; ++w) mine[w] = 0;
    if (v > 0) {
      int p = parent[v];
      if (p < 0 || p >= v) return CERB_E_ARG;
      for (int w = 0; w < CERB_ANC_WORDS; ++w) mine[w] = anc_out[(size_t)p * CERB_ANC_WORDS + w];
    }
    mine[v >> 6] |= 1ull << (v & 63);
  }
  return CERB_OK;
}

int cerb_workspace_bytes(const cerb_config* cfg, size_t* bytes_out) {
  if (!bytes_out) return CERB_E_ARG;
  CERB_TRY(validate_config(cfg));
  cerb_ctx* c = new (std::nothrow) cerb_ctx();
  if (!c) return CERB_E_NOMEM;
  init_sizes(c, cfg, 148);
  *bytes_out = carve(c, nullptr);
  delete c;
  return CERB_OK;
}

int cerb_load(const cerb_config* cfg, const cerb_weights* w, void* workspace_dev, size_t ws_bytes, cerb_ctx** out) {
  if (!w || !workspace_dev || !out) return CERB_E_ARG;
  CERB_TRY(validate_config(cfg));
  if (!w->embed || !w->final_norm || !w->lm_head || !w->attn_norm || !w->wqkv || !w->wo || !w->mlp_norm || !w->wgu ||
      !w->wd || !w->k_pool || !w->v_pool || !w->page_table)
    return CERB_E_ARG;
  if (cfg->n_cheads > 0 && (!w->head_W || !w->head_b || !w->head_fc)) return CERB_E_ARG;
  if ((uintptr_t)workspace_dev & 255) return CERB_E_ARG;
  cerb_ctx* c = new (std::nothrow) cerb_ctx();
  if (!c) return CERB_E_NOMEM;
  // The split plan (and with it the workspace size) is fixed for a 148-SM part so that
  // cerb_workspace_bytes needs no device; the launch plan uses the same number.
  init_sizes(c, cfg, 148);
  size_t need = carve(c, nullptr);
  if (ws_bytes < need) { delete c; return CERB_E_NOMEM; }
  carve(c, (char*)workspace_dev);
  const cerb_config& g = c->cfg;
  const int L = g.n_layers, HD = g.n_heads * g.head_dim;
  c->embed = w->embed; c->final_norm = w->final_norm; c->lm_head = w->lm_head;
  c->attn_norm.assign(w->attn_norm, w->attn_norm + L);
  c->wqkv.assign(w->wqkv, w->wqkv + L);
  c->wo.assign(w->wo, w->wo + L);
  c->mlp_norm.assign(w->mlp_norm, w->mlp_norm + L);
  c->wgu.assign(w->wgu, w->wgu + L);
  c->wd.assign(w->wd, w->wd + L);
  if (g.n_cheads > 0) {
    c->head_W.assign(w->head_W, w->head_W + g.n_cheads * g.n_levels);
    c->head_b.assign(w->head_b, w->head_b + g.n_cheads * g.n_levels);
    c->head_fc.assign(w->head_fc, w->head_fc + g.n_cheads);
  }
  c->k_pool = (char*)w->k_pool;
  c->v_pool = (char*)w->v_pool;
  c->pool_layer_bytes = (size_t)g.n_pool_pages * g.n_heads * CERB_PAGE * g.head_dim * c->esize;
  c->page_table = w->page_table;
  c->B = 0;
  c->verified_tree = nullptr;
  c->launches = 0;
  c->last_rows = 0;
  c->prof_on = false;
  c->prof_mode = 0;
  c->gemm_clock_used = 0;
  c->prof_used = 0;
  memset(c->tree_used, 0, sizeof(c->tree_used));
  memset(c->h_len, 0, sizeof(c->h_len));
  c->chain = c->single = nullptr;
  c->h_stage = nullptr;
  int rc = CERB_OK;
  do {
    if (cudaMallocHost((void**)&c->h_stage, 8 * CERB_MAX_BATCH * sizeof(int32_t)) != cudaSuccess) { rc = CERB_E_NOMEM; break; }
    if (cudaMemset(workspace_dev, 0, (size_t)((char*)c->d_hlast - (char*)workspace_dev)) != cudaSuccess) { rc = CERB_E_CUDA; break; }
    if (cudaMemset(c->d_attn_scratch, 0, 4096) != cudaSuccess) { rc = CERB_E_CUDA; break; }
    if (cudaMemcpy(c->d_kper, g.topk, CERB_MAX_HEADS * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess) { rc = CERB_E_CUDA; break; }
    if (c->bf16) {
      const int Mr = round_up(c->Mmax, 256);
      c->tm_wqkv.resize(L); c->tm_wo.resize(L); c->tm_wgu.resize(L); c->tm_wd.resize(L);
      c->tm_kpool.resize(L); c->tm_vpool.resize(L);
      for (int l = 0; l < L && rc == CERB_OK; ++l) {
        if ((rc = make_weight_map(&c->tm_wqkv[l], c->wqkv[l], 3 * HD, g.d_model)) != CERB_OK) break;
        if ((rc = make_weight_map(&c->tm_wo[l], c->wo[l], g.d_model, HD)) != CERB_OK) break;
        if ((rc = make_weight_map(&c->tm_wgu[l], c->wgu[l], 2 * g.mlp_dim, g.d_model)) != CERB_OK) break;
        if ((rc = make_weight_map(&c->tm_wd[l], c->wd[l], g.d_model, g.mlp_dim)) != CERB_OK) break;
        if ((rc = make_pool_map(&c->tm_kpool[l], c->k_pool + (size_t)l * c->pool_layer_bytes, g.n_pool_pages, g.n_heads, g.head_dim)) != CERB_OK) break;
        if ((rc = make_pool_map(&c->tm_vpool[l], c->v_pool + (size_t)l * c->pool_layer_bytes, g.n_pool_pages, g.n_heads, g.head_dim)) != CERB_OK) break;
      }
      if (rc != CERB_OK) break;
      if ((rc = make_weight_map(&c->tm_lm_head, c->lm_head, g.vocab, g.d_model)) != CERB_OK) break;
      if ((rc = make_act_maps(&c->tm_xn, c->d_xn, Mr, g.d_model)) != CERB_OK) break;
      if ((rc = make_act_maps(&c->tm_hidden, c->d_hidden, Mr, g.d_model)) != CERB_OK) break;
      if ((rc = make_act_maps(&c->tm_attn, c->d_attn, Mr, HD)) != CERB_OK) break;
      if ((rc = make_act_maps(&c->tm_act, c->d_act, Mr, g.mlp_dim)) != CERB_OK) break;
      if ((rc = make_act_maps(&c->tm_hlast, c->d_hlast, CERB_MAX_BATCH, g.d_model)) != CERB_OK) break;
    }
    if ((rc = launch_rope_table(c, 0)) != CERB_OK) break;
    const int chunk = kPrefillChunkMax;
    std::vector<int32_t> par(chunk);
    for (int v = 0; v < chunk; ++v) par[v] = v - 1;
    // the prefill chain is deeper than an acceptable path may be: no depth limit for it
    if ((rc = tree_build(c, par.data(), nullptr, nullptr, chunk, CERB_MAX_TREES, false, false, &c->chain)) != CERB_OK) break;
    int32_t one = -1;
    if ((rc = tree_build(c, &one, nullptr, nullptr, 1, CERB_MAX_TREES + 1, false, true, &c->single)) != CERB_OK) break;
    if (cudaDeviceSynchronize() != cudaSuccess) { rc = CERB_E_CUDA; break; }
  } while (0);
  if (rc != CERB_OK) { cerb_free(c); return rc; }
  *out = c;
  return CERB_OK;
}

int cerb_free(cerb_ctx* c) {
  if (!c) return CERB_E_ARG;
  if (c->h_stage) cudaFreeHost(c->h_stage);
  for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
  delete c->chain;
  delete c->single;
  delete c;
  return CERB_OK;
}

int cerb_tree_create(cerb_ctx* c, const int32_t* parent, const int32_t* head_of, const int32_t* rank_of, int32_t n,
                     cerb_tree** out) {
  if (!c || !out) return CERB_E_ARG;
  if (n > c->cfg.max_nodes) return CERB_E_ARG;
  int slot = -1;
  for (int i = 0; i < CERB_MAX_TREES; ++i)
    if (!c->tree_used[i]) { slot = i; break; }
  if (slot < 0) return CERB_E_NOMEM;
  CERB_TRY(tree_build(c, parent, head_of, rank_of, n, slot, c->cfg.n_cheads > 0 && n > 1, true, out));
  c->tree_used[slot] = true;
  return CERB_OK;
}

int cerb_tree_free(cerb_ctx* c, cerb_tree* t) {
  if (!c || !t) return CERB_E_ARG;
  if (t->slot >= 0 && t->slot < CERB_MAX_TREES) c->tree_used[t->slot] = false;
  if (c->verified_tree == t) c->verified_tree = nullptr;
  delete t;
  return CERB_OK;
}

int cerb_reset(cerb_ctx* c, void* stream) {
  if (!c) return CERB_E_ARG;
  CERB_CUDA_OK(cudaMemsetAsync(c->d_len, 0, CERB_MAX_BATCH * sizeof(int32_t), (cudaStream_t)stream));
  memset(c->h_len, 0, sizeof(c->h_len));
  c->verified_tree = nullptr;
  return CERB_OK;
}

int cerb_prefill(cerb_ctx* c, const int32_t* tokens_dev, const int32_t* lens_host, int32_t B, int32_t max_len,
                 void* stream) {
  if (!c || !tokens_dev || !lens_host) return CERB_E_ARG;
  if (B < 1 || B > c->cfg.max_batch || max_len < 1) return CERB_E_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  int longest = 0;
  for (int b = 0; b < B; ++b) {
    if (lens_host[b] < 1 || lens_host[b] > max_len) return CERB_E_ARG;
    if (lens_host[b] + c->cfg.max_nodes > c->max_pos) return CERB_E_STATE;
    if (lens_host[b] > longest) longest = lens_host[b];
  }
  c->B = B;
  CERB_TRY(cerb_reset(c, stream));
  // the staging buffer may still be in flight from an earlier call on this stream
  CERB_CUDA_OK(cudaStreamSynchronize(st));
  for (int b = 0; b < B; ++b) c->h_stage[b] = lens_host[b];
  CERB_CUDA_OK(cudaMemcpyAsync(c->d_lens_in, c->h_stage, B * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  const int C = c->chain->n;          // 128 tokens per chunk
  for (int off = 0; off < longest; off += C) {
    int need[CERB_MAX_BATCH];
    for (int b = 0; b < B; ++b) {
      c->h_len[b] = lens_host[b] < off ? lens_host[b] : off;
      const int left = lens_host[b] - off;
      need[b] = left < 0 ? 0 : left < C ? left : C;
    }
    CERB_TRY(launch_set_nactive(c, 1, off, C, st));
    CERB_TRY(forward_rows(c, c->chain, tokens_dev, max_len, off, C, st, 0, nullptr, need));
    CERB_TRY(launch_prefill_commit(c, C, st));
  }
  for (int b = 0; b < B; ++b) c->h_len[b] = lens_host[b];
  // root = argmax LH(h_last)
  CERB_TRY(lm_head_argmax(c, c->d_hlast, &c->tm_hlast, B, c->d_root, nullptr, st));
  c->verified_tree = nullptr;
  return CERB_OK;
}

int cerb_gate(cerb_ctx* c, float T, float* S_dev, int32_t* mode_dev, void* stream) {
  if (!c || !S_dev || !mode_dev) return CERB_E_ARG;
  if (c->B < 1) return CERB_E_STATE;
  return launch_gate(c, T, S_dev, mode_dev, nullptr, 0, (cudaStream_t)stream);
}

int cerb_draft(cerb_ctx* c, const cerb_tree* tree, int32_t* tree_tok_dev, int32_t* topk_dev, float* head_logits_dev,
               void* stream) {
  if (!c || !tree || !tree_tok_dev) return CERB_E_ARG;
  if (c->B < 1 || c->cfg.n_cheads < 1) return CERB_E_STATE;
  return launch_heads(c, tree, tree_tok_dev, nullptr, topk_dev, head_logits_dev, (cudaStream_t)stream);
}

int cerb_verify(cerb_ctx* c, const cerb_tree* tree, const int32_t* tree_tok_dev, const int32_t* n_active_dev,
                int32_t* node_argmax_dev, float* logits_dev, void* hidden_dev, void* stream) {
  if (!c || !tree || !tree_tok_dev || !node_argmax_dev) return CERB_E_ARG;
  if (c->B < 1) return CERB_E_STATE;
  cudaStream_t st = (cudaStream_t)stream;
  const int n = tree->n, M = c->B * n;
  CERB_TRY(set_active(c, n_active_dev, n, st));
  CERB_TRY(forward_rows(c, tree, tree_tok_dev, n, 0, n, st));
  CERB_TRY(lm_head_argmax(c, c->d_hidden, &c->tm_hidden, M, node_argmax_dev, logits_dev, st));
  if (hidden_dev)
    CERB_CUDA_OK(cudaMemcpyAsync(hidden_dev, c->d_hidden, (size_t)M * c->cfg.d_model * c->esize, cudaMemcpyDeviceToDevice, st));
  c->verified_tree = tree;
  return CERB_OK;
}

int cerb_accept(cerb_ctx* c, const cerb_tree* tree, const int32_t* tree_tok_dev, const int32_t* n_active_dev,
                const int32_t* node_argmax_dev, int32_t* n_accept_dev, int32_t* path_dev, int32_t* out_tok_dev,
                void* stream) {
  if (!c || !tree || !tree_tok_dev || !node_argmax_dev || !n_accept_dev || !path_dev || !out_tok_dev) return CERB_E_ARG;
  if (c->B < 1 || c->verified_tree != tree) return CERB_E_STATE;
  CERB_TRY(launch_accept(c, tree, tree_tok_dev, n_active_dev ? n_active_dev : c->d_nactive, node_argmax_dev,
                         n_accept_dev, path_dev, out_tok_dev, (cudaStream_t)stream));
  for (int b = 0; b < c->B; ++b) c->h_len[b] += tree->max_depth + 1;     // upper bound until the next read-back
  c->verified_tree = nullptr;
  return CERB_OK;
}

int cerb_step(cerb_ctx* c, const cerb_tree* tree, float T, const int32_t* plant_tok_dev, cerb_step_out* out,
              void* stream) {
  if (!c || !tree || !out || !out->S_dev || !out->mode_dev || !out->n_accept_dev || !out->tokens_dev) return CERB_E_ARG;
  if (c->B < 1) return CERB_E_STATE;
  if (tree->n > 1 && c->cfg.n_cheads < 1) return CERB_E_STATE;
  cudaStream_t st = (cudaStream_t)stream;
  const int B = c->B;
  // gate; it also writes each sequence's live node count (1 for an auto-regressive sequence)
  { ProfScope ps(c, K_GATE, st); CERB_TRY(launch_gate(c, T, out->S_dev, out->mode_dev, c->d_nactive, tree->n, st)); }
  int32_t* hs = c->h_stage;
  CERB_CUDA_OK(cudaMemcpyAsync(hs, out->mode_dev, B * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  CERB_CUDA_OK(cudaMemcpyAsync(hs + CERB_MAX_BATCH, c->d_len, B * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  CERB_CUDA_OK(cudaMemcpyAsync(hs + 2 * CERB_MAX_BATCH, out->S_dev, B * sizeof(float), cudaMemcpyDeviceToHost, st));
  CERB_CUDA_OK(cudaStreamSynchronize(st));
  bool any_par = false;
  for (int b = 0; b < B; ++b) {
    float S;
    memcpy(&S, hs + 2 * CERB_MAX_BATCH + b, sizeof(float));
    if (!isfinite(S)) return CERB_E_NONFINITE;
    if (hs[b] == CERB_MODE_PAR) any_par = true;
    c->h_len[b] = hs[CERB_MAX_BATCH + b];
    if (out->S_host) out->S_host[b] = S;
    if (out->mode_host) out->mode_host[b] = hs[b];
  }
  int n_ar = 0;
  for (int b = 0; b < B; ++b) n_ar += hs[b] == CERB_MODE_AR;
  const cerb_tree* used = (any_par && tree->n > 1) ? tree : c->single;
  const int32_t* tok = c->d_root;                       // [B][1]: the root tokens
  if (used != c->single) {
    ProfScope ps(c, K_HEADS, st);
    CERB_TRY(launch_heads(c, tree, c->d_treetok, plant_tok_dev, nullptr, nullptr, st));
    tok = c->d_treetok;
  }
  const int n = used->n;
  // A batch whose sequences chose different modes: an auto-regressive sequence contributes one row, a drafting one
  // n rows.  The row offsets go to the device ahead of the forward's first kernel (the staging words are free:
  // this call has just waited for the stream).
  int M = B * n;
  const int32_t* row_off = nullptr;
  if (used != c->single && n_ar > 0) {
    int32_t* ro = hs + 3 * CERB_MAX_BATCH;
    M = 0;
    for (int b = 0; b < B; ++b) { ro[b] = M; M += hs[b] == CERB_MODE_AR ? 1 : n; }
    ro[B] = M;
    CERB_CUDA_OK(cudaMemcpyAsync(c->d_rowoff, ro, (B + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    row_off = c->d_rowoff;
  }
  CERB_TRY(forward_rows(c, used, tok, n, 0, n, st, M, row_off));
  CERB_TRY(lm_head_argmax(c, c->d_hidden, &c->tm_hidden, M, c->d_argmax, nullptr, st));
  { ProfScope ps(c, K_ACCEPT, st);
    CERB_TRY(launch_accept(c, used, tok, c->d_nactive, c->d_argmax, out->n_accept_dev, c->d_path, out->tokens_dev, st, row_off)); }
  for (int b = 0; b < B; ++b) c->h_len[b] += used->max_depth + 1;
  if (out->n_accept_host)
    CERB_CUDA_OK(cudaMemcpyAsync(out->n_accept_host, out->n_accept_dev, B * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  if (out->tokens_host)
    CERB_CUDA_OK(cudaMemcpyAsync(out->tokens_host, out->tokens_dev, (size_t)B * kPathMax * sizeof(int32_t),
                                 cudaMemcpyDeviceToHost, st));
  c->verified_tree = nullptr;
  return CERB_OK;
}

int cerb_attn_scratch_bytes(int32_t B, int32_t n, int32_t n_heads, int32_t head_dim, size_t* bytes_out) {
  if (!bytes_out || B < 1 || n < 1 || n > CERB_MAX_NODES || n_heads < 1 || (head_dim != 64 && head_dim != 128)) return CERB_E_ARG;
  *bytes_out = attn_scratch_bytes(B, n, n_heads, head_dim);
  return CERB_OK;
}

int cerb_tree_attention(const cerb_attn_args* a, void* stream) {
  if (!a || !a->q || !a->k_pool || !a->v_pool || !a->page_table || !a->len || !a->anc || !a->out) return CERB_E_ARG;
  if (a->B < 1 || a->n < 1 || a->n > CERB_MAX_NODES || a->n_heads < 1) return CERB_E_ARG;
  if (a->head_dim != 64 && a->head_dim != 128) return CERB_E_SHAPE;
  if (a->dtype == CERB_F32) return launch_tree_attention(nullptr, a, nullptr, nullptr, 148, nullptr, (cudaStream_t)stream);
  if (a->dtype != CERB_BF16) return CERB_E_ARG;
  if (!a->scratch || a->n_pool_pages < 1) return CERB_E_ARG;
  CUtensorMap tk, tv;
  CERB_TRY(make_pool_map(&tk, a->k_pool, a->n_pool_pages, a->n_heads, a->head_dim));
  CERB_TRY(make_pool_map(&tv, a->v_pool, a->n_pool_pages, a->n_heads, a->head_dim));
  // the status word lives at the end of the counter block of the scratch
  int32_t* status = reinterpret_cast<int32_t*>((char*)a->scratch + 4096 - 16);
  return launch_tree_attention(nullptr, a, &tk, &tv, 148, status, (cudaStream_t)stream);
}

int cerb_gemm_scratch_bytes(int32_t M, int32_t N, int32_t K, size_t* bytes_out) {
  if (!bytes_out || M < 1 || N < 1 || K < 1) return CERB_E_ARG;
  *bytes_out = 256 + (size_t)gemm_plan_split(148, M, N, K) * M * N * sizeof(float);
  return CERB_OK;
}

// Sums split partials into the output (used only by the stand-alone GEMM entry point).
__global__ void sum_splits_kernel(const float* __restrict__ part, int nsplit, size_t stride, float* __restrict__ out,
                                  size_t total) {
  griddep_wait();
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  float a = 0.f;
  for (int s = 0; s < nsplit; ++s) a += part[s * stride + i];
  out[i] = a;
}

int cerb_gemm(int32_t dtype, const void* X_dev, const void* W_dev, float* out_dev, int32_t M, int32_t N, int32_t K,
              void* scratch_dev, size_t scratch_bytes, void* stream) {
  if (!X_dev || !W_dev || !out_dev || M < 1 || N < 1 || K < 1) return CERB_E_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (dtype == CERB_F32) return launch_gemm_f32(nullptr, (const float*)X_dev, (const float*)W_dev, out_dev, M, N, K, st);
  if (dtype != CERB_BF16) return CERB_E_ARG;
  if (K % 8) return CERB_E_SHAPE;
  size_t need;
  CERB_TRY(cerb_gemm_scratch_bytes(M, N, K, &need));
  if (!scratch_dev || scratch_bytes < need || ((uintptr_t)scratch_dev & 255)) return CERB_E_NOMEM;
  int ns = gemm_plan_split(148, M, N, K);
  CUtensorMap tw;
  ActMaps tx;
  CERB_TRY(make_weight_map(&tw, W_dev, N, K));
  CERB_TRY(make_act_maps(&tx, X_dev, M, K));
  int32_t* status = reinterpret_cast<int32_t*>(scratch_dev);
  float* part = reinterpret_cast<float*>((char*)scratch_dev + 256);
  CERB_CUDA_OK(cudaMemsetAsync(status, 0, 4, st));
  CERB_TRY(launch_gemm_bf16(nullptr, &tw, &tx, part, M, N, K, ns, status, st));
  size_t total = (size_t)M * N;
  sum_splits_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(part, ns, total, out_dev, total);
  if (cudaGetLastError() != cudaSuccess) return CERB_E_CUDA;
  return CERB_OK;
}

int cerb_read_state(cerb_ctx* c, int32_t* len_host, int32_t* root_host, void* h_last_host, void* stream) {
  if (!c) return CERB_E_ARG;
  if (c->B < 1) return CERB_E_STATE;
  cudaStream_t st = (cudaStream_t)stream;
  CERB_CUDA_OK(cudaStreamSynchronize(st));
  int32_t tmp[CERB_MAX_BATCH];
  CERB_CUDA_OK(cudaMemcpy(tmp, c->d_len, c->B * sizeof(int32_t), cudaMemcpyDeviceToHost));
  for (int b = 0; b < c->B; ++b) {
    c->h_len[b] = tmp[b];
    if (len_host) len_host[b] = tmp[b];
  }
  if (root_host) CERB_CUDA_OK(cudaMemcpy(root_host, c->d_root, c->B * sizeof(int32_t), cudaMemcpyDeviceToHost));
  if (h_last_host)
    CERB_CUDA_OK(cudaMemcpy(h_last_host, c->d_hlast, (size_t)c->B * c->cfg.d_model * c->esize, cudaMemcpyDeviceToHost));
  return CERB_OK;
}

int cerb_device_status(cerb_ctx* c, void* stream) {
  if (!c) return CERB_E_ARG;
  CERB_CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
  int32_t s = 0;
  CERB_CUDA_OK(cudaMemcpy(&s, c->d_status, sizeof(s), cudaMemcpyDeviceToHost));
  if (s != 0) {
    // a launch that gave up may have left the arrival counters of the GEMM's fused epilogue half-way
    CERB_CUDA_OK(cudaMemset(c->d_status, 0, 4 * sizeof(int32_t)));
    CERB_CUDA_OK(cudaMemset(c->d_gemm_tickets, 0, kGemmTickets * sizeof(unsigned int)));
  }
  return s;
}

int cerb_wait_diagnosis(cerb_ctx* c, int32_t* out4_host, void* stream) {
  if (!c || !out4_host) return CERB_E_ARG;
  CERB_CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
  CERB_CUDA_OK(cudaMemcpy(out4_host, c->d_status, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost));
  return CERB_OK;
}

int cerb_profile_enable(cerb_ctx* c, int32_t on) {
  if (!c || on < 0 || on > 2) return CERB_E_ARG;
  c->prof_on = on != 0;
  c->prof_mode = on;
  if (on == 2) {
    // starts collect a minimum, ends a maximum
    CERB_CUDA_OK(cudaMemset(c->d_gemm_clock, 0xFF, kGemmClockSlots * sizeof(unsigned long long)));
    CERB_CUDA_OK(cudaMemset(c->d_gemm_clock + kGemmClockSlots, 0, kGemmClockSlots * sizeof(unsigned long long)));
    c->gemm_clock_used = 0;
  }
  return CERB_OK;
}

int cerb_profile_read(cerb_ctx* c, double* ms_out, int64_t* groups_out, void* stream) {
  if (!c || !ms_out || !groups_out) return CERB_E_ARG;
  CERB_CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
  for (int k = 0; k < CERB_PROF_KINDS; ++k) { ms_out[k] = 0.0; groups_out[k] = 0; }
  if (c->prof_mode == 2) {
    const int n = c->gemm_clock_used;
    std::vector<unsigned long long> h(2 * (size_t)kGemmClockSlots);
    CERB_CUDA_OK(cudaMemcpy(h.data(), c->d_gemm_clock, h.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
    for (int i = 0; i < n; ++i) {
      const unsigned long long t0 = h[i], t1 = h[kGemmClockSlots + i];
      if (t1 > t0) { ms_out[0] += (double)(t1 - t0) * 1e-6; groups_out[0] += 1; }
    }
    CERB_CUDA_OK(cudaMemset(c->d_gemm_clock, 0xFF, kGemmClockSlots * sizeof(unsigned long long)));
    CERB_CUDA_OK(cudaMemset(c->d_gemm_clock + kGemmClockSlots, 0, kGemmClockSlots * sizeof(unsigned long long)));
    c->gemm_clock_used = 0;
    return CERB_OK;
  }
  for (size_t i = 0; i < c->prof_used; ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->prof_ev[2 * i], c->prof_ev[2 * i + 1]) != cudaSuccess) continue;
    ms_out[c->prof_kind[i]] += ms;
    groups_out[c->prof_kind[i]] += 1;
  }
  c->prof_used = 0;
  return CERB_OK;
}

int64_t cerb_launch_count(const cerb_ctx* c) { return c ? c->launches : -1; }

int32_t cerb_last_forward_rows(const cerb_ctx* c) { return c ? c->last_rows : -1; }

int cerb_set_wait_cycles(int64_t cycles) {
  if (cycles < 1000) return CERB_E_ARG;
  cerb::g_wait_cycles = cycles;
  return CERB_OK;
}

}  // extern "C"
