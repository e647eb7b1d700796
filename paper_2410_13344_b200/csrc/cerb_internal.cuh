// Internal declarations shared by the translation units of libcerb.so.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "cerb.h"

#define CERB_CUDA_OK(expr)                         \
  do {                                             \
    cudaError_t e__ = (expr);                      \
    if (e__ != cudaSuccess) return CERB_E_CUDA;    \
  } while (0)

#define CERB_TRY(expr)                 \
  do {                                 \
    int rc__ = (expr);                 \
    if (rc__ != CERB_OK) return rc__;  \
  } while (0)

#define CERB_LAUNCH_CHECK(c)                                   \
  do {                                                         \
    if (c) (c)->launches++;                                    \
    if (cudaGetLastError() != cudaSuccess) return CERB_E_CUDA; \
  } while (0)

namespace cerb {

typedef __nv_bfloat16 bf16;

// Programmatic dependent launch: a kernel launched through launch_pdl may begin while its
// predecessor in the stream is still running; it must execute griddep_wait() before it touches
// anything the predecessor writes (or anything the predecessor may still be reading and this
// kernel overwrites).  griddep_launch() lets the next kernel in the stream be scheduled early.
#ifdef __CUDACC__
// Which sequence and which node a row of the step's activation buffers belongs to: with ragged rows (sequences that
// verify a one-node tree next to sequences that verify the whole tree) sequence b starts at row_off[b], otherwise at
// b * n.
__device__ __forceinline__ void locate_row(int row, const int32_t* __restrict__ row_off, int B, int n, int& b, int& v) {
  if (!row_off) { b = row / n; v = row - b * n; return; }
  b = 0;
  while (b + 1 < B && row_off[b + 1] <= row) ++b;
  v = row - row_off[b];
}
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif
bool pdl_enabled();
// Budget of every bounded device-side wait, in SM clock cycles (cerb_set_wait_cycles; about 2 s by default).
long long wait_cycles();

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Same, for a kernel whose CTAs form clusters of `cluster_x` along x.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                      unsigned cluster_x, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cluster_x;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

constexpr int kPathMax = CERB_MAX_DEPTH + 1;
constexpr int kPrefillChunkMax = 128;   // prompt tokens per prefill chunk (a chain-shaped tree), whatever max_nodes is
constexpr int kGemmRowsPerPass = 256;   // activation rows one tcgen05 pass covers at most (the MMA's N extent; CTA pairs)
constexpr int kGemmMaxSplit = 16;

// Device-side copy of a tree, living in the workspace.
struct TreeDev {
  int32_t* parent;   // [CERB_MAX_NODES]
  int32_t* depth;
  int32_t* head_of;
  int32_t* rank_of;
  uint64_t* anc;     // [CERB_MAX_NODES][CERB_ANC_WORDS]
};
constexpr size_t kTreeSlotBytes = 4 * CERB_MAX_NODES * sizeof(int32_t) + CERB_MAX_NODES * CERB_ANC_WORDS * sizeof(uint64_t);

// Tensor maps for one activation buffer used as the MMA's B operand, one per row bucket.
constexpr int kRowBuckets = 5;          // 16, 32, 64, 128, 256 rows
struct ActMaps {
  CUtensorMap m[kRowBuckets];
};

}  // namespace cerb

struct cerb_tree {
  int32_t n;
  int32_t slot;
  int32_t max_depth;
  cerb::TreeDev dev;
  std::vector<int32_t> parent, depth;
};

struct cerb_ctx {
  cerb_config cfg;
  bool bf16;
  size_t esize;                       // bytes per model element
  int Mmax;                           // max rows of one forward (max_batch * max_nodes)
  int max_pos;                        // 16 * max_pages
  int head_w[CERB_MAX_HEADS][CERB_MAX_LEVELS + 1];   // state width entering each level
  int head_wmax;

  // weights (device pointers, host arrays)
  const void *embed, *final_norm, *lm_head;
  std::vector<const void*> attn_norm, wqkv, wo, mlp_norm, wgu, wd, head_W, head_b, head_fc;
  char *k_pool, *v_pool;
  size_t pool_layer_bytes;
  const int32_t* page_table;

  // tensor maps (bf16 only)
  std::vector<CUtensorMap> tm_wqkv, tm_wo, tm_wgu, tm_wd;
  CUtensorMap tm_lm_head;
  cerb::ActMaps tm_xn, tm_attn, tm_act, tm_hidden, tm_hlast;
  std::vector<CUtensorMap> tm_kpool, tm_vpool;        // per layer

  // workspace carve-out
  int32_t *d_len, *d_len_old, *d_root, *d_nactive, *d_status, *d_lens_in, *d_mode, *d_naccept;
  int32_t *d_path, *d_outtok, *d_argmax, *d_treetok, *d_topk, *d_kper;
  int32_t* d_rowoff;                  // [CERB_MAX_BATCH + 1] first row of every sequence when the rows of a step are ragged
  float* d_S;
  void *d_hlast, *d_x, *d_xn, *d_q, *d_attn, *d_act, *d_hidden;
  float *d_part, *d_logits, *d_hlogits;
  float* d_topk_cv;       // per-chunk top-k candidates of the heads' logits: values [B][Hc][kTopkChunks][MAX_TOPK]
  int32_t* d_topk_ci;     // ... and their token ids
  unsigned int* d_gemm_tickets;   // kGemmTickets arrival counters of the GEMM's fused epilogue (zero between launches)
  size_t part_floats;
  float* d_hstate[2];
  float2* d_rope;
  char* d_attn_scratch;
  size_t attn_scratch_bytes;
  char* d_tree_store;
  bool tree_used[CERB_MAX_TREES];
  cerb_tree* chain;                   // chain tree of max_nodes for the prefill
  cerb_tree* single;                  // one-node tree for auto-regressive steps

  // pinned host staging
  int32_t* h_stage;                   // [8 * CERB_MAX_BATCH]

  // host-side state
  int B;
  int h_len[CERB_MAX_BATCH];          // upper bound of the committed length per sequence
  const cerb_tree* verified_tree;     // tree of the last cerb_verify not yet accepted
  int64_t launches;
  int last_rows;                      // rows of the last forward (for accounting)
  int sm_count;

  // optional per-family timing (cerb_profile_*)
  bool prof_on;
  int prof_mode;                      // 1: CUDA-event brackets per family; 2: the GEMM kernels stamp their own span
  unsigned long long* d_gemm_clock;   // [2][kGemmClockSlots]: first CTA past its dependency wait, last CTA done (ns)
  int gemm_clock_used;
  std::vector<cudaEvent_t> prof_ev;   // begin/end pairs
  std::vector<int> prof_kind;         // family of each pair
  size_t prof_used;                   // pairs recorded since the last read
};

namespace cerb {

inline int row_bucket(int rows) {
  int b = 0, r = 16;
  while (r < rows && b < kRowBuckets - 1) { r <<= 1; ++b; }
  return b;
}
inline int bucket_rows(int b) { return 16 << b; }
constexpr int kGemmTickets = 4096;
constexpr int kGemmClockSlots = 4096;
constexpr int kTopkChunks = 16;     // the vocabulary is cut into this many chunks for the heads' top-k

// launch_order.cu: the forward's launch sequence and what each kernel reads ahead of its dependency wait
enum { LO_SET_ACTIVE = 0, LO_NORM_ATTN, LO_GEMM_QKV, LO_ROPE, LO_ATTN, LO_GEMM_WO, LO_NORM_MLP, LO_GEMM_GU, LO_SWIGLU,
       LO_GEMM_DOWN, LO_NORM_FINAL, LO_GEMM_LM, LO_ARGMAX };
int launch_order_layer(int variant, const int** ids_out);     // variant 0: separate SwiGLU and RoPE kernels, 1: SwiGLU fused
                                                               // into the gate-up GEMM, 2: RoPE + append fused into the QKV GEMM too
int launch_order_violations(int variant);

// ---- launch wrappers implemented across the .cu files (all asynchronous on `st`) ----

// glue.cu
int launch_rope_table(cerb_ctx* c, cudaStream_t st);
int launch_fused_norm(cerb_ctx* c, const float* part, int nsplit, size_t split_stride, const int32_t* tok, int tok_stride,
                      int tok_off, int n, const void* gain, void* out, int rows, cudaStream_t st,
                      const int32_t* row_off = nullptr);
int launch_rope_append(cerb_ctx* c, int layer, const TreeDev& t, const float* part, int nsplit, size_t split_stride,
                       int B, int n, int rows, cudaStream_t st, const int32_t* row_off = nullptr);
int launch_swiglu(cerb_ctx* c, const float* part, int nsplit, size_t split_stride, void* act, int rows, cudaStream_t st);
int launch_argmax_rows(cerb_ctx* c, const float* part, int nsplit, size_t split_stride, int rows, int V, int32_t* out,
                       float* summed, cudaStream_t st);
int launch_set_nactive(cerb_ctx* c, int mode, int a, int b, cudaStream_t st);
int launch_prefill_commit(cerb_ctx* c, int n, cudaStream_t st);

// gemm_f32.cu / gemm_bf16.cu : out[split][M][N] fp32 partial sums of X[M][K] . W[N][K]^T
int launch_gemm_f32(cerb_ctx* c, const float* X, const float* W, float* out, int M, int N, int K, cudaStream_t st);
int gemm_plan_split(int sm_count, int M, int N, int K);
// Optional fused epilogue of the bf16 GEMM.  kind 1 (SwiGLU): W is [gate rows F][up rows F]; the GEMM
// pairs gate tile t with up tile t in one unit and the CTA that completes a tile last writes
// act[row][f] = SiLU(gate) * up (bf16) instead of leaving the partial slots to a separate kernel.
// kind 2 (RoPE + cache append): W is the QKV matrix [q rows | k rows | v rows] of a model with head_dim 128; the CTA
// that completes a 256-row tile (two heads' worth of q, k or v) last sums the tile's slots in index order, rotates q
// and k at position len + depth and writes q dense and k, v into the paged pools -- what rope_append_kernel does,
// with the same arithmetic in the same order.  Both pay for steps of up to 16 rows only.
struct RopeEpilogue {
  const int32_t *len, *n_active, *depth, *page_table, *row_off;    // as for rope_append_kernel (row_off may be null)
  const float2* rope;       // rotation table [max_pos][64]
  void *q, *kpool, *vpool;  // bf16: q [rows][H * 128]; this layer's pools
  int max_pages, max_pos, n, H, B;
};
struct GemmEpilogue {
  int kind;                 // 0 none, 1 SwiGLU, 2 RoPE + cache append
  void* act;                // kind 1: [M][F] bf16
  unsigned int* tickets;    // kGemmTickets counters, zero on entry and on exit
  const RopeEpilogue* rope; // kind 2
};
bool gemm_swiglu_fusable(int M, int F);
bool gemm_rope_fusable(int M, int head_dim);
int launch_gemm_bf16(cerb_ctx* c, const CUtensorMap* tmW, const ActMaps* tmX, float* out, int M, int N, int K,
                     int nsplit, int32_t* status, cudaStream_t st, const GemmEpilogue* epi = nullptr,
                     unsigned long long* clock_slot = nullptr);
int make_weight_map(CUtensorMap* out, const void* W, int N, int K);
int make_act_maps(ActMaps* out, const void* X, int rows_alloc, int K);
int init_driver_api();

// attention.cu
size_t attn_scratch_bytes(int B, int n, int H, int Dh);
int make_pool_map(CUtensorMap* out, const void* pool, int n_pool_pages, int H, int Dh);
// row_off: first row of every sequence in q / out when the rows of a batch are ragged (device, [B]); null = b * n
int launch_tree_attention(cerb_ctx* c, const cerb_attn_args* a, const CUtensorMap* tmK, const CUtensorMap* tmV,
                          int sm_count, int32_t* status, cudaStream_t st, const int32_t* row_off = nullptr);

// heads.cu
int launch_heads(cerb_ctx* c, const cerb_tree* tree, int32_t* tree_tok, const int32_t* plant, int32_t* topk_out,
                 float* logits_out, cudaStream_t st);

// gate_accept.cu
int launch_gate(cerb_ctx* c, float T, float* S, int32_t* mode, int32_t* nactive_or_null, int n_par, cudaStream_t st);
int launch_accept(cerb_ctx* c, const cerb_tree* tree, const int32_t* tree_tok, const int32_t* n_active,
                  const int32_t* node_argmax, int32_t* n_accept, int32_t* path, int32_t* out_tok, cudaStream_t st,
                  const int32_t* row_off = nullptr);

}  // namespace cerb
