// Internal declarations shared by the kernels and the host scheduler of the Amphista step.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "amph.h"

namespace amph {

typedef unsigned long long u64;

constexpr int kMaxRows = AMPH_MAX_NODES;   // rows one forward call may carry (tree nodes / prefill chunk)
constexpr int kMaxK = AMPH_MAX_HEADS_K;
constexpr int kTopkStride = AMPH_TOPK_STRIDE;   // row stride of the top-k id / value tables
constexpr int kPendMax = kMaxK + 1;        // rows the adaptation layers may have pending

// Per-call row table: where each row of a forward call sits and what it may see.
// Row r is at rotary position pos[r], writes its key / value to cache slot slot[r] and attends
// slots [0, base) plus slot base + m for every set bit m of mask[r] (Fig. 5: ancestors only).
struct RowMeta {
  int base;
  int n_rows;
  int pos[kMaxRows];
  int slot[kMaxRows];
  u64 mask[kMaxRows][2];
};

// Static tree tables built at init (Appendix A.1).
struct TreeDev {
  int n_nodes;
  int parent[kMaxRows];
  int depth[kMaxRows];
  int rank[kMaxRows];
  u64 anc[kMaxRows][2];     // bit m set <=> node m is on the root path of this node (itself included)
};

// Device-resident decoding state; every kernel reads lengths from here, so a step needs no
// host round trip.
struct DevState {
  int C;                    // committed tokens (cache slots 0..C-1)
  int root;                 // token chosen for position C
  int n_pending;            // rows queued for the adaptation layers (positions C-n_pending..C-1)
  int err;                  // sticky device-side error code (amph_status) or 0
  int pend_tok[16];         // token at position (row position + 1) for each pending row
  // result of the last acceptance
  int L;                    // accepted tokens (root included)
  int C_old;                // C before the acceptance
  int best;                 // deepest accepted node
  int next_root;
  int path[16];
  int out_tok[16];
  int step;                 // acceptances this sequence has seen (counter of the sampling generator)
};

// Programmatic dependent launch.  Every kernel of the step is launched with the attribute below, so it
// may become resident before its predecessor in the stream has finished; it must call pdl_wait() before
// touching anything the predecessor writes.  pdl_launch_dependents() lets the successor start launching.
// Rule used here: weight-streaming projections trigger at once, prefetch weights, then wait; every other
// kernel waits first and triggers right after, so at most two consecutive kernels ever overlap.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... P, typename... A>
inline cudaError_t launch_pdl(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, A... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...);
}
#endif

struct KvView {             // one layer's cache: K and V as [n_heads][max_ctx][head_dim]
  void* k;
  void* v;
};

// fp32 partial sums of a projection: value(row, col) = sum_{s < splits} p[s*split_stride + row*ld + col]
struct PartialView {
  const float* p;
  int splits;
  int ld;                   // row stride in floats (total output features of the launch)
  size_t split_stride;      // floats between consecutive splits
};

// Deferred RMSNorm: a projection may be fed g * x (not yet divided by the row's RMS); the kernel that
// consumes the projection's output multiplies by 1 / sqrt(sum_c ss[row][c] / d + eps).  ss == NULL: no scaling.
struct RowScale {
  const float* ss = nullptr;   // [rows][chunks] partial sums of squares of the row
  int chunks = 0;
  int d = 1;
  float eps = 0.f;
};
constexpr int kScaleChunkCols = 512;     // columns per block of resid_scale_kernel (128 threads x float4)

#ifdef __CUDACC__
// value(row, col .. col+3) of a projection left as split-K partial sums (fixed order: deterministic)
__device__ __forceinline__ float4 sum_partials4(const PartialView& P, int row, int col) {
  const float* p = P.p + (size_t)row * P.ld + col;
  float4 acc = *reinterpret_cast<const float4*>(p);
#pragma unroll 4
  for (int s = 1; s < P.splits; ++s) {
    const float4 v = *reinterpret_cast<const float4*>(p + (size_t)s * P.split_stride);
    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
  }
  return acc;
}
__device__ __forceinline__ float row_scale(const RowScale& rs, int row) {
  if (rs.ss == nullptr) return 1.0f;
  float tot = 0.f;
#pragma unroll 8
  for (int c = 0; c < rs.chunks; ++c) tot += rs.ss[row * rs.chunks + c];       // fixed order
  return 1.0f / sqrtf(tot / (float)rs.d + rs.eps);
}
#endif

// ---- launchers (one per kernel family); dtype = AMPH_DTYPE_* of weights / activations / cache
void launch_embed(const void* tok_emb, int dtype, const int* toks, int vocab, int rows, int d,
                  float* x, cudaStream_t st);

// x <- (mode 0: x, mode 1: x + sum P, mode 2: sum P); then, if gain != NULL, RMSNorm of the result
// into xn (storage dtype) and hid (fp32); with gain == NULL xn / hid receive the plain row.
// col_off selects the column window of P.
void launch_resid_norm(float* x, PartialView P, int col_off, int mode, const void* gain, int dtype,
                       void* xn, float* hid, float eps, int rows, int d, cudaStream_t st);

// Fully parallel variant for the inner layers: x <- x + sum P (mode 1) or sum P (mode 2); xn <- gain * x
// (not normalised) and ss_part[row][chunk] <- sum of squares of the chunk.  gain == NULL: x only.
// early != 0: let the next kernel (a projection, which only prefetches weights until its own wait) start
// launching before this kernel has waited for its predecessor.  The caller sets it only when the
// predecessor's grid is fully resident (one wave), so that the early starter cannot take its slots.
void launch_resid_scale(float* x, PartialView P, int col_off, int mode, const void* gain, int dtype, void* xn,
                        float* ss_part, int rows, int d, cudaStream_t st, int early = 0);

void launch_rope_table(const RowMeta* meta, const double* inv_freq, float2* table, int rows, int half,
                       cudaStream_t st);

// q <- rope(sum P[:, 0:d]); K cache <- rope(sum P[:, d:2d]); V cache <- sum P[:, 2d:3d]
void launch_qkv_rope(PartialView P, const RowMeta* meta, const float2* rope, void* q, KvView kv,
                     int dtype, int rows, int n_heads, int head_dim, int max_ctx, cudaStream_t st,
                     RowScale rs = RowScale());

struct RopeGroups {         // per row group: row table, rotary table, cache
  const RowMeta* meta[AMPH_MAX_BATCH];
  const float2* rope[AMPH_MAX_BATCH];
  void* kc[AMPH_MAX_BATCH];
  void* vc[AMPH_MAX_BATCH];
  int G, rpg;
};
void launch_qkv_rope_groups(PartialView P, const RopeGroups& gr, void* q, int dtype, int n_heads, int head_dim, int max_ctx,
                            cudaStream_t st, RowScale rs = RowScale());

struct AttnScratch {
  float* o;                 // [splits][heads][rows][head_dim]
  float* ml;                // [splits][heads][rows][2]  (running max, running sum)
};
void launch_tree_attention(const void* q, KvView kv, const RowMeta* meta, AttnScratch sc, void* out,
                           int dtype, int rows, int n_heads, int head_dim, int max_ctx, int ctx_hi,
                           int max_splits, cudaStream_t st, int early = 0, int separate_merge = 0);

// merged_out != NULL and splits <= 8: the splits of a head run as one cluster and write the final bf16 rows to
// merged_out themselves (returns true); otherwise partial results go to sc for attn_combine_kernel (returns false).
bool launch_tree_attention_mma(const void* q, KvView kv, const RowMeta* meta, AttnScratch sc, int rows, int n_heads,
                               int head_dim, int max_ctx, int splits, cudaStream_t st, void* merged_out);

void launch_attn_combine(AttnScratch sc, void* out, int dtype, int splits, int rows, int n_heads, int head_dim,
                         cudaStream_t st, int early);

// tcgen05 / TMA tree attention (bf16 caches).  An AttnTc holds the tensor maps of the caches it has seen.
struct AttnTc;
AttnTc* attn_tc_create();
void attn_tc_destroy(AttnTc* a);
int attn_tc_splits(const AttnTc* a, int keys_bound, int n_heads, int rows, int max_splits);
int attn_tc_stages(int keys_bound, int splits, int head_dim);
bool launch_tree_attention_tc(AttnTc* a, const void* q, int q_rows_cap, KvView kv, const RowMeta* meta, AttnScratch sc, int rows,
                              int n_heads, int head_dim, int max_ctx, int splits, int keys_bound, cudaStream_t st,
                              void* merged_out, int* err_flag);

bool launch_tree_attention_tc_groups(AttnTc* a, const void* q, int q_rows_cap, int G, const KvView* kv, const RowMeta* const* meta,
                                     int rows, int n_heads, int head_dim, int max_ctx, int splits, int keys_bound, cudaStream_t st,
                                     void* merged_out, int* err_flag);

void launch_swiglu(PartialView P, void* act, int dtype, int rows, int f, cudaStream_t st, RowScale rs = RowScale(),
                   int early = 0);

// cat[r] = [feat[r] ; tok_emb[next[r]]]   (Eq. 1's concatenation)
void launch_concat(const float* feat, const void* tok_emb, const int* next_tok, int vocab, void* cat,
                   int dtype, int rows, int d, cudaStream_t st);

struct GemmSeg { const void* w; };
// P[row][seg*out + o] = sum_k X[row][k] * W_seg[o][k]; plain CUDA-core kernel, one split.
void launch_gemm_generic(const void* x, int ldx, const GemmSeg* segs, int n_seg, int out, int in,
                         float* P, int ldp, int rows, int dtype, cudaStream_t st);

// ---- draft-module specific
void launch_gather_last(const float* h1, const float* h2, const DevState* st_dev, float* last /*[2][d]*/,
                        void* last_act /*[>=2][d]*/, int dtype, int d, cudaStream_t st);
// Hp[k] = src_k + silu(sum P[row_k][k*d + :] + b_k) + PE[k]   (Eq. 2-4)
void launch_mlp_heads(PartialView P, const float* last, const void* const* bias, const void* pe,
                      float* hp, float* ao, void* ao_act, int dtype, int K, int n_sal, int d, cudaStream_t st);
// unmasked attention across the K rows, one block per attention head (Eq. 5)
void launch_aeb_attention(PartialView P, void* out_act, int dtype, int K, int n_heads, int head_dim,
                          cudaStream_t st);
// out_act[k][j] = P(row k, column k * r + j): row k of the k-th low-rank projection, as the next projection's input
void launch_gather_diag(PartialView P, void* out_act, int dtype, int K, int r, cudaStream_t st);
// per head k: top-c_k of row k of segment k; also stores the row into d_logits[k]
// cand: scratch for the slices' candidates, kMaxK * kTopkCandChunks * kTopkStride (value, id) pairs
constexpr int kTopkCandChunks = 32;
void launch_topk_heads(PartialView P, int vocab, int K, const int* ck, int* ids, float* vals,
                       float* d_logits, float* cand, cudaStream_t st);
// cand: scratch for the slices' candidates, kMaxRows * 8 (value, id) pairs
void launch_argmax_rows(PartialView P, int vocab, int rows, int* amax, float* logits_out, float* cand, cudaStream_t st);

// ---- control kernels
void launch_meta_chain(RowMeta* meta, int base, int n_rows, cudaStream_t st);             // prefill chunk
void launch_meta_pending(RowMeta* meta, const DevState* s, cudaStream_t st);              // adaptation rows
void launch_tree_build(const TreeDev* tree, DevState* s, const int* topk_ids, const int* override_tok,
                       int* tok, RowMeta* meta, cudaStream_t st);
void launch_accept(const TreeDev* tree, DevState* s, const int* tok, const int* amax, cudaStream_t st);
// Sampling at temperature T > 0 (Table 2): choice[r] for rows row0 .. row0 + n_rows - 1 = the token the target draws after
// that row from softmax(logits / T) with the row's own uniform (Philox4x32-10 keyed by seed; counter = row - row0, the
// sequence's step count, seq, stream).  With a tree (tok != NULL) the vocabulary is walked in the order (tokens of the
// row's children in node order, then every other id ascending), so that a child is accepted iff its token is the choice:
// the rejection-sampling test of Section 2 for point-mass proposals.  uniforms_out (may be NULL) receives the uniforms.
void launch_sample_rows(const float* logits, int vocab, int row0, int n_rows, const TreeDev* tree, const int* tok,
                        const DevState* s, int seq, int stream_id, float temperature, unsigned long long seed, int* choice,
                        float* uniforms_out, cudaStream_t st);
void launch_compact(const DevState* s, const KvView* kv_layers, int n_layers, int dtype, int n_heads,
                    int head_dim, int max_ctx, const float* hidden, float* pend_h, int d, cudaStream_t st);
void launch_reduce_partials(PartialView P, float* y, int rows, int cols, cudaStream_t st);
void launch_kv_export(KvView kv, int which, int dtype, int row0, int rows, int n_heads, int head_dim, int max_ctx,
                      float* dst, cudaStream_t st);
void launch_prefill_tail(DevState* s, const int* amax, int last_row, const float* hidden, float* pend_h,
                         int d, int C, cudaStream_t st);

}  // namespace amph
