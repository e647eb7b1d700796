/*
 * cerb.h -- C ABI of the Cerberus decoding-step library (sm_100a, one GPU).
 *
 * One decoding step of Cerberus (arxiv 2410.13344, Algorithm 1) has four parts:
 * the Cerberus heads draft candidate tokens in parallel (Section 4.1), an entropy
 * gate on the last hidden state picks parallel or auto-regressive decoding
 * (Section 4.2), the base model verifies the candidate tree in one forward pass
 * with tree-masked attention over the KV cache (Sections 1 and 3.1, "tree
 * verification"), and the longest greedily matching path is accepted and its KV
 * entries are moved into place.
 *
 * Conventions for every call
 *   - returns an int status: CERB_OK (0) or a negative CERB_E_* code; nothing
 *     throws across this boundary; cerb_strerror() names a code.
 *   - "dev" pointers are device memory, "host" pointers are host memory.  All
 *     device memory is CALLER-OWNED (weights, KV pools, page table, workspace,
 *     outputs), must outlive the context and is never freed here.  The library
 *     allocates only its host-side context / tree structs.
 *   - `stream` is a cudaStream_t passed as void*.  Calls are asynchronous on it
 *     unless stated otherwise and allocate no device memory.
 *   - dtype CERB_BF16: weights, activations and KV cache are bf16; accumulation,
 *     softmax, logits, head states and the entropy are fp32.  dtype CERB_F32:
 *     everything fp32.
 *   - batch: B sequences, each with its own committed length `len[b]`, last
 *     hidden state, next root token and page-table row.
 *
 * Row / slot conventions (shared by verify, accept and the KV cache)
 *   - a tree has n nodes, node 0 is the root (the LM head's own greedy token),
 *     parent[v] < v; rows of a step are ordered [b][v];
 *   - node v is evaluated at RoPE position len[b] + depth[v];
 *   - node v's K/V are written at logical slot len[b] + v; after acceptance the
 *     j-th accepted node is moved to slot len[b] + j and len[b] += n_accept[b].
 *   - logical slot s of sequence b lives in physical page page_table[b][s / 16],
 *     row s % 16.  Pool layout per layer: [page][head][16][head_dim].
 */
#ifndef CERB_H_
#define CERB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CERB_OK            0
#define CERB_E_ARG        -1   /* null pointer, negative size, unknown enum          */
#define CERB_E_SHAPE      -2   /* a dimension the kernels do not support             */
#define CERB_E_NOMEM      -3   /* workspace too small / host allocation failed       */
#define CERB_E_STATE      -4   /* call out of order, sequence would exceed its pages */
#define CERB_E_NONFINITE  -5   /* gate entropy is not finite                         */
#define CERB_E_TIMEOUT    -6   /* a bounded device-side wait ran out                 */
#define CERB_E_CUDA       -7   /* a CUDA runtime / driver call failed                */

#define CERB_F32   0
#define CERB_BF16  1

#define CERB_MODE_PAR 0        /* parallel decoding: draft + tree verification */
#define CERB_MODE_AR  1        /* auto-regressive step: one-node tree          */

#define CERB_PAGE        16    /* tokens per KV page                                  */
#define CERB_MAX_NODES   192   /* tree nodes per sequence; Sec. 5.1 uses up to 150 candidates + the root */
#define CERB_ANC_WORDS   3     /* 64-bit words of one node's ancestor mask (CERB_MAX_NODES / 64)       */
#define CERB_MAX_DEPTH   8     /* deepest node; an accepted path has <= 9 nodes       */
#define CERB_MAX_HEADS   8     /* decoding heads                                      */
#define CERB_MAX_LEVELS  8     /* Resblocks per decoding head                         */
#define CERB_MAX_TOPK    16    /* candidates kept per decoding head                   */
#define CERB_MAX_BATCH   16
#define CERB_MAX_TREES   8     /* trees alive per context                             */

typedef struct cerb_ctx cerb_ctx;
typedef struct cerb_tree cerb_tree;

/* Model and head configuration (Algorithm 1 "Require": N layers, TL, LH, CH). */
typedef struct cerb_config {
  int32_t dtype;                 /* CERB_F32 | CERB_BF16 */
  int32_t n_layers;              /* N */
  int32_t d_model;
  int32_t n_heads;               /* attention heads (= KV heads) */
  int32_t head_dim;              /* 64 or 128 */
  int32_t mlp_dim;
  int32_t vocab;
  float   rope_base;             /* 10000 */
  float   rms_eps;               /* 1e-5 */
  int32_t max_pages;             /* page-table columns per sequence: capacity = 16 * max_pages tokens */
  int32_t n_pool_pages;          /* physical pages per layer in each pool */
  int32_t max_batch;             /* <= CERB_MAX_BATCH */
  int32_t max_nodes;             /* <= CERB_MAX_NODES (prefill runs in chunks of 128 tokens whatever this is) */
  int32_t n_cheads;              /* Cerberus heads CH_0 .. CH_{n_cheads-1} */
  int32_t n_levels;              /* Resblocks per head */
  /* Section 4.1 wiring: concat_src[h][j] = -1 for the plain Resblock
   * SiLU(W h + b + h); otherwise the two-input Resblock, whose input is
   * Concat(state of head h, state of head concat_src[h][j]), both taken as they
   * enter level j.  The block's width is the concatenated width and stays so for
   * the rest of that head. */
  int32_t concat_src[CERB_MAX_HEADS][CERB_MAX_LEVELS];
  int32_t topk[CERB_MAX_HEADS];  /* candidates kept per head (<= CERB_MAX_TOPK) */
} cerb_config;

/* Caller-owned device tensors, row-major [out][in], dtype as in the config.
 * The arrays of pointers themselves are HOST arrays and are copied at load. */
typedef struct cerb_weights {
  const void* embed;             /* dev [vocab][d_model]  */
  const void* final_norm;        /* dev [d_model]         */
  const void* lm_head;           /* dev [vocab][d_model]  */
  const void* const* attn_norm;  /* host [n_layers] -> dev [d_model] */
  const void* const* wqkv;       /* host [n_layers] -> dev [3*H*Dh][d_model], q rows, k rows, v rows */
  const void* const* wo;         /* host [n_layers] -> dev [d_model][H*Dh] */
  const void* const* mlp_norm;   /* host [n_layers] -> dev [d_model] */
  const void* const* wgu;        /* host [n_layers] -> dev [2*mlp_dim][d_model], gate rows then up rows */
  const void* const* wd;         /* host [n_layers] -> dev [d_model][mlp_dim] */
  const void* const* head_W;     /* host [n_cheads*n_levels] (index h*n_levels+j) -> dev [w][w] */
  const void* const* head_b;     /* host [n_cheads*n_levels] -> dev [w] */
  const void* const* head_fc;    /* host [n_cheads] -> dev [vocab][w_final] */
  void* k_pool;                  /* dev [n_layers][n_pool_pages][H][16][Dh] */
  void* v_pool;                  /* dev, same layout */
  const int32_t* page_table;     /* dev [max_batch][max_pages]; entries for slots < len + max_nodes must be valid */
} cerb_weights;

/* Bytes of device workspace cerb_load needs for this configuration (256-byte aligned base). */
int cerb_workspace_bytes(const cerb_config* cfg, size_t* bytes_out);

/* Validates the configuration, records the pointers, builds TMA descriptors and
 * the RoPE table inside the workspace.  Synchronous (it runs small set-up kernels
 * on the default stream and waits).  CERB_E_SHAPE for unsupported dimensions,
 * CERB_E_NOMEM if ws_bytes < cerb_workspace_bytes. */
int cerb_load(const cerb_config* cfg, const cerb_weights* w, void* workspace_dev, size_t ws_bytes, cerb_ctx** out);
int cerb_free(cerb_ctx* ctx);

/* Candidate tree ("tree paths", Section 5.1 Tree Settings): parent[0] = -1,
 * parent[v] < v.  head_of[v] / rank_of[v] name the decoding head and the rank in
 * its top-k that fills node v (ignored for the root).  Depths and ancestor
 * bitmasks are derived here.  Host arrays, copied; synchronous.  CERB_E_ARG if the
 * order is not topological, depth > CERB_MAX_DEPTH, n > max_nodes, or a
 * head / rank is outside the configuration; CERB_E_NOMEM when CERB_MAX_TREES
 * trees are alive. */
int cerb_tree_create(cerb_ctx* ctx, const int32_t* parent, const int32_t* head_of, const int32_t* rank_of,
                     int32_t n, cerb_tree** out);
int cerb_tree_free(cerb_ctx* ctx, cerb_tree* tree);

/* Forget all sequences (len = 0). */
int cerb_reset(cerb_ctx* ctx, void* stream);

/* Process the prompts: tokens_dev [B][max_len] int32, lens_host [B] (1 <= len).
 * Runs the base model over the prompt in chain-shaped chunks (a chain tree is
 * ordinary causal attention), fills the KV cache, sets len, the last hidden state
 * (final-norm output at the last position) and the root token
 * argmax LH(h_last) (Algorithm 1, LH).  Sets the batch size B for later calls. */
int cerb_prefill(cerb_ctx* ctx, const int32_t* tokens_dev, const int32_t* lens_host, int32_t B, int32_t max_len,
                 void* stream);

/* Entropy gate (Section 4.2; Algorithm 1: P = Softmax(h_last), S = Entropy(P),
 * S > T selects auto-regressive decoding).  The softmax runs over the d_model
 * components of each sequence's last hidden state; S is in bits.
 * S_dev [B] float, mode_dev [B] int32 (CERB_MODE_*).
 * The call only enqueues work and never reads S back, so it cannot return
 * CERB_E_NONFINITE: a non-finite S (from a non-finite hidden state) is left in
 * S_dev for the caller to see (a NaN compares false with T and so selects
 * CERB_MODE_PAR); cerb_step, which reads S on the host anyway, reports it. */
int cerb_gate(cerb_ctx* ctx, float T, float* S_dev, int32_t* mode_dev, void* stream);

/* Draft (Section 4.1; Algorithm 1: Candidates = (LH[h_last], CH_0[h_last], ...)):
 * runs every decoding head level by level from each sequence's last hidden
 * state, takes each head's top-k (ties: lower id) and fills the tree:
 * tree_tok[b][0] = root token, tree_tok[b][v] = topk[b][head_of[v]][rank_of[v]].
 * tree_tok_dev [B][n] int32; topk_dev optional [B][n_cheads][CERB_MAX_TOPK] int32;
 * head_logits_dev optional [B][n_cheads][vocab] float. */
int cerb_draft(cerb_ctx* ctx, const cerb_tree* tree, int32_t* tree_tok_dev, int32_t* topk_dev,
               float* head_logits_dev, void* stream);

/* Tree verification (Algorithm 1: O = Tree_Verify(Candidates)): one base-model
 * forward over all n nodes of every sequence.  Node v attends to the committed
 * prefix and to its own ancestors.  Writes the nodes' K/V at slots len + v (not
 * committed until cerb_accept).  n_active_dev: optional [B] int32, nodes
 * 0 .. n_active[b]-1 are live (NULL = all n); inactive rows are ignored.
 * node_argmax_dev [B][n] int32 = argmax of the LM head at each node (ties: lower
 * id).  logits_dev optional [B][n][vocab] float; hidden_dev optional [B][n][d_model]
 * (model dtype) = final-norm output per node. */
int cerb_verify(cerb_ctx* ctx, const cerb_tree* tree, const int32_t* tree_tok_dev, const int32_t* n_active_dev,
                int32_t* node_argmax_dev, float* logits_dev, void* hidden_dev, void* stream);

/* Greedy acceptance and commit (Section 3.1: candidates are verified to find the
 * tokens to accept).  A root-to-node path is accepted when every non-root token
 * equals node_argmax at its parent; the longest path wins, ties go to the lowest
 * end node; the root is always accepted.  Then the path's K/V move to slots
 * len .. len + n_accept - 1 in every layer, len += n_accept, the last hidden
 * state becomes the last accepted node's, and that node's argmax becomes the next
 * root.  Must follow a cerb_verify of the same tree (else CERB_E_STATE).
 * n_accept_dev [B]; path_dev [B][CERB_MAX_DEPTH+1] node indices (-1 padded);
 * out_tok_dev [B][CERB_MAX_DEPTH+1] accepted tokens (-1 padded). */
int cerb_accept(cerb_ctx* ctx, const cerb_tree* tree, const int32_t* tree_tok_dev, const int32_t* n_active_dev,
                const int32_t* node_argmax_dev, int32_t* n_accept_dev, int32_t* path_dev, int32_t* out_tok_dev,
                void* stream);

/* Results of one whole step.  Device buffers are required; the host mirrors are
 * optional (pinned memory recommended) and are valid once `stream` is synchronised. */
typedef struct cerb_step_out {
  float*   S_dev;          /* [B] */
  int32_t* mode_dev;       /* [B] */
  int32_t* n_accept_dev;   /* [B] */
  int32_t* tokens_dev;     /* [B][CERB_MAX_DEPTH+1] */
  float*   S_host;         /* optional [B] */
  int32_t* mode_host;      /* optional [B] */
  int32_t* n_accept_host;  /* optional [B] */
  int32_t* tokens_host;    /* optional [B][CERB_MAX_DEPTH+1] */
} cerb_step_out;

/* One decoding step, Algorithm 1: gate; sequences with S > T verify a one-node
 * tree (their root token), the others draft and verify `tree` (the rows of a batch
 * are ragged: one row for an auto-regressive sequence, n for a drafting one); then
 * accept and commit.  Waits once inside, after the gate, to learn whether any sequence
 * drafts; everything else is asynchronous on `stream`.  plant_tok_dev: optional
 * [B][n] int32 with -1 = keep the drafted token, used to exercise acceptance with
 * untrained heads; NULL in normal use. */
int cerb_step(cerb_ctx* ctx, const cerb_tree* tree, float T, const int32_t* plant_tok_dev, cerb_step_out* out,
              void* stream);

/* Stand-alone tree-verification attention (what cerb_verify runs per layer).
 * For each sequence b, node i < n and head h: softmax over the len[b] prefix keys
 * and the tree keys j with bit j of anc[i] set, of scale * q_i . k, times V;
 * lse = natural log of the softmax denominator (scaled scores). */
typedef struct cerb_attn_args {
  int32_t dtype;                /* CERB_BF16 | CERB_F32 */
  int32_t B, n, n_heads, head_dim;
  int32_t max_pages;            /* page-table row stride */
  const void* q;                /* dev [B][n][H][Dh] */
  const void* k_pool;           /* dev [pages][H][16][Dh] (one layer) */
  const void* v_pool;
  const int32_t* page_table;    /* dev [B][max_pages] */
  const int32_t* len;           /* dev [B] prefix lengths; tree keys sit at slots len .. len+n-1 */
  const int32_t* n_active;      /* dev [B] or NULL (= n) */
  const uint64_t* anc;          /* dev [n][CERB_ANC_WORDS]: bit j (word j/64) set iff j is an ancestor of i or i itself */
  void* out;                    /* dev [B][n][H][Dh] */
  float* lse;                   /* dev [B][H][n] or NULL */
  float scale;
  int32_t max_len;              /* host upper bound of len[b] + n, sizes the launch */
  int32_t n_pool_pages;         /* pages in the pool (bounds the TMA descriptor) */
  void* scratch;                /* dev scratch for split-KV partials, cerb_attn_scratch_bytes(); first 4 KB zero before first use */
  size_t scratch_bytes;
} cerb_attn_args;

/* Errors found on the device (a bounded wait that ran out: CERB_E_TIMEOUT; max_len smaller than a
 * sequence's len + n: CERB_E_SHAPE) are written to the four int32 status words at bytes 4080..4095 of
 * the scratch ([0] code, [1] which wait, [2] which block, [3] which launch); the call itself only
 * enqueues and returns CERB_OK.  A launch that finds word [0] set runs with its waits shortened to
 * microseconds, produces nothing useful and leaves the word as it is; the caller reads the words after
 * synchronising and clears the first 4 KB before the next use. */
int cerb_attn_scratch_bytes(int32_t B, int32_t n, int32_t n_heads, int32_t head_dim, size_t* bytes_out);
int cerb_tree_attention(const cerb_attn_args* args, void* stream);

/* cerb_tree_attention for callers that cannot allocate device memory (the paper has no
 * counterpart; this is a packaging variant of the same kernels).  Typical cases: code running
 * inside an allocator or memory-pool callback, a plug-in that only receives fixed buffers from its
 * host application, a process whose device-memory budget is fixed at start-up.  The split-KV
 * scratch that the caller would otherwise provide lives in a static device array inside the
 * library, CERB_STATIC_ATTN_SCRATCH_BYTES large; every GPU that loads the library holds it until
 * the process exits.  args->scratch and args->scratch_bytes are ignored; inputs and outputs are
 * still the caller's.  bf16 only.  This call never allocates or frees device memory.
 *
 * Limit.  CERB_E_NOMEM when cerb_attn_scratch_bytes() for the problem exceeds the static array.
 * That size is 4096 + (328 + B * n_heads) * P * (head_dim + 4) * 4 bytes with P = the tree's node
 * count padded to 16 / 32 / 64 / 128 (every tree above 64 nodes counts as 128).  With 16 MiB:
 *   head_dim 128: trees of up to 16 nodes B * n_heads <= 1020 (the ticket counters' limit, CERB_E_SHAPE
 *                 beyond it, as for the ordinary entry); up to 32 nodes <= 664; up to 64
 *                 nodes <= 168 (batch 5 at 32 heads); trees above 64 nodes are always rejected;
 *   head_dim  64: up to 64 nodes B * n_heads <= 635; above 64 nodes <= 153.
 *
 * Set-up.  The first call on each device looks up the array's device address (one runtime query,
 * with that device current); make that first call outside any stream capture.
 * Sharing.  All calls share the one array and each call clears, on `stream`, the part that must
 * start at zero, so two calls that may overlap on the GPU (different streams, no dependency) race
 * with each other: serialise them.
 * Errors found on the device (a bounded wait that ran out, max_len smaller than a sequence's
 * len + n) land in status words inside the array, which no call clears:
 * cerb_tree_attention_noalloc_status synchronises `stream`, returns the first word (CERB_OK,
 * CERB_E_TIMEOUT or CERB_E_SHAPE; the output of the call that raised it is undefined) and clears
 * it.  Until it has been read, later calls through this entry run with shortened waits. */
#define CERB_STATIC_ATTN_SCRATCH_BYTES (16u << 20)
int cerb_tree_attention_noalloc(const cerb_attn_args* args, void* stream);
int cerb_tree_attention_noalloc_status(void* stream);

/* Ancestor bitmasks of a tree, the form cerb_tree_attention takes: anc_out host [n][CERB_ANC_WORDS]. */
int cerb_tree_ancestors(const int32_t* parent, int32_t n, uint64_t* anc_out);

/* Stand-alone dense GEMM as the verification forward runs it (Algorithm 1, TL_i / LH):
 * out[M][N] (fp32) = X[M][K] . W[N][K]^T, X and W in `dtype`, fp32 accumulation.
 * bf16 runs on the tcgen05 tensor-core path (weights streamed once, split along K
 * when few weight tiles exist); scratch holds the split-K partial sums,
 * cerb_gemm_scratch_bytes().  K must be a multiple of 8. */
int cerb_gemm_scratch_bytes(int32_t M, int32_t N, int32_t K, size_t* bytes_out);
int cerb_gemm(int32_t dtype, const void* X_dev, const void* W_dev, float* out_dev, int32_t M, int32_t N, int32_t K,
              void* scratch_dev, size_t scratch_bytes, void* stream);

/* Synchronous read-back of the per-sequence state (any pointer may be NULL):
 * len_host [B], root_host [B], h_last_host [B][d_model] in the model dtype. */
int cerb_read_state(cerb_ctx* ctx, int32_t* len_host, int32_t* root_host, void* h_last_host, void* stream);

/* Status word written by bounded device-side waits since the last call of this
 * function: CERB_OK, or CERB_E_TIMEOUT.  Synchronises `stream`. */
int cerb_device_status(cerb_ctx* ctx, void* stream);

/* Diagnosis of a CERB_E_TIMEOUT (the paper has no counterpart): copies the four status words to out4_host
 * without clearing them: [0] the status cerb_device_status reports, [1] a number naming the wait inside the
 * kernel that ran out first, [2] the block that waited (x + 1000 y + 1000000 z), [3] a number naming the
 * launch (GEMM: output columns + 100000 x rows).  Synchronises
 * `stream`. */
int cerb_wait_diagnosis(cerb_ctx* ctx, int32_t* out4_host, void* stream);

/* Per-kernel-family device timing, for measurement only (the paper has no counterpart).  While
 * enabled, the host controller brackets each family's launches with CUDA events on the caller's
 * stream; cerb_profile_read synchronises the stream, adds up the elapsed times and launch-group
 * counts per family since the last read, and clears them.  Families: 0 dense GEMMs, 1 tree
 * attention, 2 decoding heads + top-k + tree fill, 3 element-wise glue (embedding, norms, RoPE
 * and KV append, residual, SwiGLU, argmax), 4 gate, 5 acceptance + KV compaction.
 * ms_out and groups_out are host arrays of CERB_PROF_KINDS entries.  Event recording costs a few
 * microseconds per bracket and keeps neighbouring kernels from overlapping, so time whole steps with
 * profiling off.  cerb_profile_enable(ctx, 2) selects a second mode that leaves the launch sequence
 * untouched: every bf16 GEMM launch records, in the device's nanosecond timer, when its first CTA got past
 * the wait for the previous kernel and when its last CTA finished; cerb_profile_read then returns the sum of
 * those spans in ms_out[0] and their number in groups_out[0] (other families 0; at most 4096 launches
 * between reads).  on = 0 switches profiling off, 1 selects the event brackets. */
#define CERB_PROF_KINDS 6
int cerb_profile_enable(cerb_ctx* ctx, int32_t on);
int cerb_profile_read(cerb_ctx* ctx, double* ms_out, int64_t* groups_out, void* stream);

/* Budget of every bounded device-side wait (mbarrier and cluster waits inside the kernels), in SM clock
 * cycles, for all later launches of this process; the paper has no counterpart.  The default, 4e9 (about two
 * seconds), is far beyond any legitimate wait.  A wait that runs out makes its CTA raise CERB_E_TIMEOUT in the
 * status word, leave its loops, wait (bounded) for its own copies in flight, free its tensor memory and
 * return; the results of that launch are then undefined and cerb_device_status reports the code.  Meant for
 * testing that exit; CERB_E_ARG below 1000 cycles. */
int cerb_set_wait_cycles(int64_t cycles);

/* The launch sequence of the base-model forward with, per kernel, the buffers it writes and the buffers it reads
 * ahead of its dependency wait (bit masks; the paper has no counterpart, this documents the library's use of
 * programmatic dependent launch).  Writes one line per launch, "id|name|writes|reads-before-wait", for one set-up
 * launch, three layers and the tail, into buf (host).  variant 0: separate SwiGLU and RoPE kernels; 1: SwiGLU inside the
 * gate-up GEMM (steps of at most 16 rows); 2: RoPE + cache append inside the QKV GEMM as well (such steps at
 * head_dim 128).  Returns CERB_OK when no kernel reads, ahead of its wait, a buffer
 * that the kernel right in front of it writes, CERB_E_STATE otherwise, CERB_E_NOMEM when buf is too small. */
int cerb_launch_order_table(int32_t variant, char* buf_host, size_t cap);

/* Number of kernel launches issued by this context since load (for accounting). */
int64_t cerb_launch_count(const cerb_ctx* ctx);

/* Activation rows of the last base-model forward this context launched (for accounting): B * n for cerb_verify and
 * the prefill chunks; for cerb_step the sum over the sequences of n (drafting) or 1 (auto-regressive). */
int32_t cerb_last_forward_rows(const cerb_ctx* ctx);

const char* cerb_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* CERB_H_ */
