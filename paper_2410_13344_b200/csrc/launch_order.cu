// The launch sequence of the base-model forward and what each kernel touches before its dependency wait.
//
// Every kernel of the forward is launched programmatically dependent on its predecessor: it may start while the
// kernel in front is still running, and it executes griddepcontrol.wait before it touches what that kernel writes.
// Every kernel also releases its own dependents only AFTER its own wait.  So when kernel i runs, kernel i - 2 and
// everything older is complete, and kernel i may read, ahead of its wait, any buffer whose youngest writer is at
// least two launches older.  This file states, per kernel, what it writes and what it reads ahead of its wait;
// launch_order_violations() checks the rule over the cyclic layer sequence, and the host controller steps
// through the same table while it launches (forward_rows), so that the table cannot drift from the code.
#include <stdio.h>
#include <string.h>

#include "cerb_internal.cuh"

namespace cerb {

namespace {

// buffers (bits)
enum : unsigned {
  B_X = 1u << 0,       // residual stream (fp32)
  B_XN = 1u << 1,      // norm output = GEMM input
  B_PART = 1u << 2,    // fp32 partial slots of the last GEMM
  B_Q = 1u << 3,       // rotated queries
  B_KV = 1u << 4,      // this step's tree slots of the K/V pools
  B_ATTN = 1u << 5,    // attention output
  B_ACT = 1u << 6,     // SwiGLU output
  B_HIDDEN = 1u << 7,  // final-norm output
  B_STATE = 1u << 8,   // per-sequence state the step starts from: lengths, live node counts (written before the forward)
  B_CONST = 1u << 9,   // never written during a forward: weights, gains, tree arrays, page table, rotation table,
                       // committed (prefix) K/V
};

struct Entry {
  int id;
  const char* name;
  unsigned writes;
  unsigned prewait_reads;
};

// One layer, then the tail.  Ids are what forward_rows announces, in this order.
const Entry kSetActive = {LO_SET_ACTIVE, "set_active / gate (live node counts)", B_STATE, 0};
const Entry kLayer64[] = {
    {LO_NORM_ATTN, "fused_norm (embedding or residual add, attention norm)", B_X | B_XN, B_X | B_CONST},
    {LO_GEMM_QKV, "gemm qkv", B_PART, B_CONST},
    {LO_ROPE, "rope_append", B_Q | B_KV, B_STATE | B_CONST},
    {LO_ATTN, "tree attention", B_ATTN, B_STATE | B_CONST},
    {LO_GEMM_WO, "gemm wo", B_PART, B_CONST},
    {LO_NORM_MLP, "fused_norm (residual add, MLP norm)", B_X | B_XN, B_X | B_CONST},
    {LO_GEMM_GU, "gemm gate-up", B_PART, B_CONST},
    {LO_SWIGLU, "swiglu", B_ACT, 0},
    {LO_GEMM_DOWN, "gemm down", B_PART, B_CONST},
};
// Few-row steps: SwiGLU runs in the gate-up GEMM's epilogue (that GEMM writes the activations itself).
const Entry kLayer16[] = {
    kLayer64[0], kLayer64[1], kLayer64[2], kLayer64[3], kLayer64[4], kLayer64[5],
    {LO_GEMM_GU, "gemm gate-up + swiglu epilogue", B_PART | B_ACT, B_CONST},
    kLayer64[8],
};
// ... and (head_dim 128) RoPE + cache append in the QKV GEMM's epilogue.
const Entry kLayer16r[] = {
    kLayer64[0],
    {LO_GEMM_QKV, "gemm qkv + rope / append epilogue", B_PART | B_Q | B_KV, B_CONST},
    kLayer64[3], kLayer64[4], kLayer64[5],
    {LO_GEMM_GU, "gemm gate-up + swiglu epilogue", B_PART | B_ACT, B_CONST},
    kLayer64[8],
};
const Entry kTail[] = {
    {LO_NORM_FINAL, "fused_norm (residual add, final norm)", B_X | B_HIDDEN, B_X | B_CONST},
    {LO_GEMM_LM, "gemm lm_head", B_PART, B_CONST},
    {LO_ARGMAX, "argmax_rows", 0, 0},
};

int build(int variant, const Entry** out, int cap) {
  // set-up, three layers (enough to close the cycle between layers), tail
  const Entry* layer = variant == 2 ? kLayer16r : variant == 1 ? kLayer16 : kLayer64;
  const int nl = variant == 2   ? (int)(sizeof(kLayer16r) / sizeof(Entry))
                 : variant == 1 ? (int)(sizeof(kLayer16) / sizeof(Entry))
                                : (int)(sizeof(kLayer64) / sizeof(Entry));
  int n = 0;
  out[n++] = &kSetActive;
  for (int l = 0; l < 3; ++l)
    for (int i = 0; i < nl && n < cap; ++i) out[n++] = &layer[i];
  for (int i = 0; i < 3 && n < cap; ++i) out[n++] = &kTail[i];
  return n;
}

}  // namespace

int launch_order_layer(int variant, const int** ids_out) {
  static int ids64[16], ids16[16], ids16r[16];
  static int n64 = 0, n16 = 0, n16r = 0;
  if (!n64) {
    for (const Entry& e : kLayer64) ids64[n64++] = e.id;
    for (const Entry& e : kLayer16) ids16[n16++] = e.id;
    for (const Entry& e : kLayer16r) ids16r[n16r++] = e.id;
  }
  *ids_out = variant == 2 ? ids16r : variant == 1 ? ids16 : ids64;
  return variant == 2 ? n16r : variant == 1 ? n16 : n64;
}

// Number of (kernel, buffer) pairs that break the rule; the tail after the last layer counts as the "next layer"
// (its first kernel is a fused_norm as well).
int launch_order_violations(int variant) {
  const Entry* seq[64];
  const int n = build(variant, seq, 64);
  int bad = 0;
  for (int i = 1; i < n; ++i) {
    for (unsigned bit = 1; bit <= B_STATE; bit <<= 1) {
      if (!(seq[i]->prewait_reads & bit)) continue;
      int j = i - 1;
      while (j >= 0 && !(seq[j]->writes & bit)) --j;
      if (j >= 0 && i - j < 2) ++bad;           // the youngest writer is the kernel right in front
    }
  }
  return bad;
}

}  // namespace cerb

extern "C" int cerb_launch_order_table(int32_t variant, char* buf, size_t cap) {
  using namespace cerb;
  if (!buf || cap < 64 || variant < 0 || variant > 2) return CERB_E_ARG;
  const Entry* seq[64];
  const int n = build(variant, seq, 64);
  size_t off = 0;
  for (int i = 0; i < n; ++i) {
    int w = snprintf(buf + off, cap - off, "%d|%s|%u|%u\n", seq[i]->id, seq[i]->name, seq[i]->writes, seq[i]->prewait_reads);
    if (w < 0 || (size_t)w >= cap - off) return CERB_E_NOMEM;
    off += (size_t)w;
  }
  return launch_order_violations(variant) == 0 ? CERB_OK : CERB_E_STATE;
}
