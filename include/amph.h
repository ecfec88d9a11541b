/*
 * amph.h - C ABI of the B200 (sm_100a) Amphista speculative-decoding step.
 *
 * One decoding step of Amphista (arXiv 2406.13170) for a Llama/Vicuna-shaped target at
 * batch 1:  draft module (Section 3, Eq. 1-6)  ->  candidate tree (Appendix A.1)  ->
 * target forward over all tree tokens under a tree-causal mask (Section 2 "Tree
 * Attention", Fig. 5)  ->  greedy longest-prefix acceptance and KV-cache compaction
 * (Section 2 "Speculative Decoding", Section 3.2 last paragraph).
 *
 * Conventions
 *   - Every function returns an amph_status; none throws, aborts or exits.
 *     amph_last_error() gives a human-readable message for the last failure on a context.
 *   - OWNERSHIP: the caller allocates and owns all device memory (weights, the KV region,
 *     the workspace) and passes raw device pointers; they must stay valid and unmoved
 *     until amph_destroy.  The library owns only the host-side amph_ctx.  The library
 *     never allocates device memory.
 *   - All device work is enqueued on the stream given to amph_init (a cudaStream_t passed
 *     as void*; NULL = the legacy default stream).
 *   - Pointers documented "host or device" may be pageable/pinned host memory or device
 *     memory; results are copied with a stream-ordered copy and are valid once the
 *     caller has synchronised the stream.  Pointers documented "host" are read or written
 *     before the call returns.
 *   - Linear weights are row-major [out_features, in_features]; vectors are contiguous.
 *   - Requires an sm_100a device.  There is no CPU path: without the device every call
 *     that needs one fails with AMPH_ERR_CUDA.
 */
#ifndef AMPH_H_
#define AMPH_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t amph_status;
enum {
  AMPH_OK = 0,
  AMPH_ERR_INVALID_ARG = 1,    /* NULL pointer, non-positive size, unknown name            */
  AMPH_ERR_SHAPE = 2,          /* unsupported model / tree shape, tensor shape mismatch     */
  AMPH_ERR_STATE = 3,          /* call order violated (see the state machine below)         */
  AMPH_ERR_CAPACITY = 4,       /* ctx_len + tree nodes would exceed max_ctx                 */
  AMPH_ERR_WORKSPACE = 5,      /* kv / workspace region too small or misaligned             */
  AMPH_ERR_MISSING_WEIGHT = 6, /* amph_load_weights did not receive every tensor           */
  AMPH_ERR_CUDA = 7,           /* a CUDA runtime / driver call failed                       */
  AMPH_ERR_TIMEOUT = 8         /* a bounded device-side wait gave up (pipeline barrier)     */
};

enum { AMPH_DTYPE_F32 = 0, AMPH_DTYPE_BF16 = 1 };

/* amph_config.flags */
enum {
  AMPH_FLAG_NO_TENSOR_CORE = 1, /* route every projection through the plain CUDA-core kernel */
  AMPH_FLAG_NO_GRAPH = 2,       /* launch kernels one by one instead of replaying a CUDA graph */
  AMPH_FLAG_SEPARATE_ROPE = 4,   /* rotary embedding + KV-cache write as a kernel of their own (bf16, up to 64 rows: the q / k / v projection does both otherwise) */
  AMPH_FLAG_SEPARATE_MERGE = 8,  /* merge the attention KV splits in a kernel of its own (bf16: a cluster does it otherwise) */
  AMPH_FLAG_SEPARATE_SWIGLU = 16, /* SwiGLU as a kernel of its own (bf16: the gate / up projection applies it otherwise) */
  AMPH_FLAG_NO_SAMPLED_TOKEN = 64, /* the "w/o Sampled-Token" ablation (Section 4.5): the adaptation layers are fed the
                                    * hidden state alone; draft.fc{s} is then [d, d] instead of [d, 2d]            */
  AMPH_FLAG_CHUNKED_PREFILL = 128, /* prefill one chunk of 128 prompt tokens per weight pass instead of four */
  AMPH_FLAG_MMA_SYNC_ATTENTION = 32, /* bf16 tree attention on the warp-level mma.sync kernel instead of the tcgen05 / TMA one */
  AMPH_FLAG_NO_SIDE_PREFETCH = 256  /* no helper stream: by default (bf16, a stream of the caller's own) every layer of the captured schedule of amph_step forks a small
                                     * kernel onto a second stream, created by amph_init, that pulls the head of the gate / up
                                     * weights into L2 while attention runs; it joins the caller's stream before amph_accept /
                                     * amph_step / amph_prefill return their work to it */
};

#define AMPH_MAX_HEADS_K 8
#define AMPH_MAX_NODES 128
#define AMPH_MAX_BATCH 8
#define AMPH_TOPK_STRIDE 16

typedef struct amph_ctx amph_ctx;

/* Shapes of the target model and of the draft module.
 * Target: Llama architecture (RMSNorm, rotary embedding on pairs (i, i + head_dim/2),
 * multi-head attention with n_heads * head_dim == d_model, SwiGLU FFN, untied lm_head).
 * Draft module (Section 3): n_sal staged adaptation layers, each one decoder layer of the
 * target's shape with its own KV cache and a preceding fc: 2d -> d; K head MLPs d -> d;
 * positional embedding PE [K, d]; aeb_layers unmasked self-attention layers with n_heads
 * heads; K vocabulary projections [vocab, d]; head k keeps its top topk[k] candidates. */
typedef struct {
  int32_t n_layers, d_model, n_heads, head_dim, d_ffn, vocab;
  float rms_eps, rope_theta;
  int32_t weight_dtype;   /* AMPH_DTYPE_*: storage type of every weight tensor             */
  int32_t kv_dtype;       /* AMPH_DTYPE_*: storage type of all KV caches (must equal weight_dtype) */
  int32_t max_ctx;        /* KV capacity in slots (committed tokens + tree nodes)           */
  int32_t max_batch;      /* sequences decoded side by side (Section 4.4), 1..AMPH_MAX_BATCH; max_batch * tree nodes
                           * (rounded up to 16) must not exceed 512.  Every sequence has its own KV caches, length
                           * and pending rows; one pass streams the weights once for all of them                 */
  int32_t K;              /* drafting heads, 1..AMPH_MAX_HEADS_K (the paper uses 4)         */
  int32_t n_sal;          /* staged adaptation layers: 2 (the paper's design), 1, or 0 (the  *
                           * heads then read the target's hidden state; Section 4.5)         */
  int32_t aeb_layers;     /* 1 (the paper's design), 2 (its "alpha" variant) or 0 (no        *
                           * Auto-embedding Block: independent heads; Section 4.5)           */
  int32_t topk[AMPH_MAX_HEADS_K]; /* candidates kept per head, each 1..AMPH_TOPK_STRIDE     */
  int32_t flags;          /* AMPH_FLAG_*                                                    */
  int32_t lm_rank;        /* 0: each drafting head owns a [vocab, d] matrix (Eq. 6); r > 0: it owns two
                           * low-rank factors a [r, d] and b [vocab, r], logits = b (a x) (Appendix A.2.4);
                           * r a multiple of 8, r <= d_model                                  */
  float temperature;      /* 0: greedy decoding (Table 1).  T > 0: random sampling (Table 2): the target draws every
                           * token from softmax(logits / T), and a drafted token is accepted by the rejection-sampling
                           * test of Section 2 for a point-mass proposal (see amph_accept)                        */
  uint32_t seed_lo, seed_hi; /* key of the counter-based generator (Philox4x32-10) that supplies the uniforms at T > 0 */
} amph_config;

/* Draft-tree topology (Appendix A.1): node 0 is the root (the token the target chose last);
 * a node of depth k >= 1 carries head k's candidate of rank `rank`.  Nodes must be sorted so
 * that parent[n] < n.  All three arrays are HOST pointers of n_nodes entries, copied by
 * amph_init.  n_nodes <= AMPH_MAX_NODES; depth <= K; rank[n] < topk[depth[n]-1]. */
typedef struct {
  int32_t n_nodes;
  const int16_t* parent;  /* parent[0] = -1 */
  const uint8_t* depth;   /* depth[0] = 0   */
  const uint8_t* rank;    /* rank[0] ignored */
} amph_tree;

/* One named weight tensor in device memory (borrowed, not copied). */
typedef struct {
  const char* name;
  const void* dev_ptr;    /* 16-byte aligned, contiguous row-major */
  int32_t dtype;          /* AMPH_DTYPE_*, must equal config.weight_dtype */
  int32_t ndim;           /* 1 or 2 */
  int64_t shape[4];
} amph_tensor;

/* State machine: amph_init -> amph_load_weights -> amph_prefill ->
 *   ( amph_draft -> amph_verify_tree -> amph_accept )*   or   amph_step*
 * A call out of order returns AMPH_ERR_STATE and changes nothing. */

/* Sizes of the two device regions the caller must provide for (config, tree).
 * kv_bytes: target KV cache + the adaptation layers' KV caches; ws_bytes: activations,
 * partial sums, state.  Host-only computation; no device needed. */
amph_status amph_workspace_bytes(const amph_config* cfg, const amph_tree* tree,
                                 size_t* kv_bytes, size_t* ws_bytes);

/* Creates a context.  kv_dev / ws_dev: device regions of at least the sizes above, 256-byte
 * aligned, owned by the caller.  Validates shapes, builds the tree tables (ancestor bitmasks,
 * positions: Fig. 5) and zeroes the state.  stream: cudaStream_t as void*. */
amph_status amph_init(const amph_config* cfg, const amph_tree* tree, void* kv_dev, size_t kv_bytes,
                      void* ws_dev, size_t ws_bytes, void* stream, amph_ctx** out);

/* Registers the weights.  Names (i = layer, s = 1..n_sal, k = 0..K-1, l = 0..aeb_layers-1):
 *   tok_emb [V,d]; layers.{i}.{attn_norm [d], wq, wk, wv, wo [d,d], ffn_norm [d],
 *   w_gate, w_up [F,d], w_down [d,F]}; final_norm [d]; lm_head [V,d];
 *   draft.fc{s} [d,2d] (Eq. 1; input order [hidden ; token embedding]; [d,d] with AMPH_FLAG_NO_SAMPLED_TOKEN);
 *   draft.sal{s}.<the nine per-layer names>; draft.mlp.{k}.w [d,d], draft.mlp.{k}.b [d] (Eq. 2);
 *   draft.pe [K,d] (Eq. 4); draft.aeb.{l}.{wq,wk,wv,wo} [d,d] (Eq. 5); draft.lm_head.{k} [V,d] (Eq. 6),
 *   or with lm_rank = r > 0: draft.lm_head.{k}.a [r,d] and draft.lm_head.{k}.b [V,r] (Appendix A.2.4).
 * May be called several times; AMPH_ERR_MISSING_WEIGHT is reported by amph_prefill if a tensor
 * was never given.  Pointers are borrowed. */
amph_status amph_load_weights(amph_ctx* ctx, const amph_tensor* tensors, int32_t n);

/* Causal forward of the prompt through the target (fills its KV cache), greedy choice of the
 * root token, and the adaptation layers over all prompt positions but the last, which stays
 * pending for the first draft (Eq. 1: their caches cover positions before t).
 * prompt_ids: HOST, n >= 1 ids in [0, vocab).  out_root: HOST, may be NULL.  Synchronises the
 * stream before returning.  Resets any previous sequence. */
amph_status amph_prefill(amph_ctx* ctx, const int32_t* prompt_ids, int32_t n, int32_t* out_root);

/* The same for sequence seq (0 .. max_batch - 1) of a context created with max_batch > 1 (Section 4.4: several
 * sequences of different lengths decoded side by side).  Every sequence must be prefilled before the first
 * amph_draft / amph_step; a sequence may be prefilled again later (between steps) to start a new text in its slot.
 * With max_batch = B the per-step calls take and return arrays with a leading sequence dimension:
 *   amph_draft        out_topk_ids / out_topk_vals [B][K][AMPH_TOPK_STRIDE]
 *   amph_verify_tree  tree_tokens / out_argmax [B][n_nodes]
 *   amph_accept       out_tokens / out_path [B][K+1], out_n / out_next_root [B]
 *   amph_step         out_tokens [B][K+1], out_n [B]
 * Sequences advance independently (own length, own accepted count); one pass streams the weights once for all. */
amph_status amph_prefill_seq(amph_ctx* ctx, int32_t seq, const int32_t* prompt_ids, int32_t n, int32_t* out_root);

/* Draft module (Section 3): adaptation layers over the pending rows (Eq. 1), K head MLPs on
 * the last row (Eq. 2), + PE (Eq. 3-4), bi-directional self-attention across the K rows (Eq. 5),
 * K vocabulary projections and top-k (Eq. 6), then tree tokens (Appendix A.1).
 * out_topk_ids [K][AMPH_TOPK_STRIDE] int32, out_topk_vals [K][AMPH_TOPK_STRIDE] float: host or
 * device, may be NULL; row k holds topk[k] entries ordered by value descending, equal values by
 * ascending id. */
amph_status amph_draft(amph_ctx* ctx, int32_t* out_topk_ids, float* out_topk_vals);

/* Target forward over the n_nodes tree tokens (Section 2, Fig. 5): node n at position
 * ctx_len + depth[n], its key / value in slot ctx_len + n, attending the ctx_len committed
 * slots and its ancestors.  tree_tokens: host or device [n_nodes] int32, or NULL to use the
 * tokens amph_draft built; entries < 0 keep the drafted token, entry 0 is always the root.
 * out_argmax: host or device [n_nodes] int32 (greedy choice after each node; ties -> lowest id),
 * may be NULL. */
amph_status amph_verify_tree(amph_ctx* ctx, const int32_t* tree_tokens, int32_t* out_argmax);

/* Greedy acceptance (Section 2): the deepest root path on which every drafted token equals the
 * target's greedy choice at its parent; compacts the accepted nodes' key / value rows to slots
 * ctx_len .. ctx_len + n - 1, advances ctx_len by n, and queues the accepted rows for the next draft.
 * With temperature T > 0 the "choice" after node n is drawn instead (amph_verify_tree computes it right after the
 * logits): with p = softmax(logits_n / T) and the node's uniform u_n, walk the vocabulary in the order (tokens of n's
 * children in node order, then every other id ascending) and take the first token whose cumulative probability
 * exceeds u_n.  Child i is thus accepted with probability p(x_i) / (1 - p(x_1) - .. - p(x_{i-1})) given that its elder
 * siblings were rejected, and a node whose children are all rejected hands on a token drawn from p with the
 * children's tokens removed: rejection sampling with point-mass proposals, which leaves the emitted tokens
 * distributed exactly as sampling from the target.  u_n = 2^-24 * (top 24 bits of word 0 of Philox4x32-10 with counter
 * (n, step, sequence, 0) and key (seed_lo, seed_hi)), step = acceptances the sequence has seen; the token after the
 * prompt uses counter (0, 0, sequence, 1).
 * out_tokens [K+1], out_n [1], out_path [K+1] (node ids), out_next_root [1]: host or device int32,
 * each may be NULL. */
amph_status amph_accept(amph_ctx* ctx, int32_t* out_tokens, int32_t* out_n, int32_t* out_path,
                        int32_t* out_next_root);

/* draft -> tree -> verify -> accept, enqueued back to back with no host synchronisation.
 * out_tokens [K+1], out_n [1]: host or device int32, may be NULL. */
amph_status amph_step(amph_ctx* ctx, int32_t* out_tokens, int32_t* out_n);

/* Debug taps (stream-ordered copy into dst, host or device).  A name may carry "#b" to select sequence b (default 0).
 * Names and element types:
 *   "hidden" f32 [rows,d] post-final-norm rows of the last target pass and "logits" f32 [rows,V] (rows =
 *   n_nodes after amph_verify_tree; after amph_prefill the rows of its last pass: a pass carries 4 * AMPH_MAX_NODES
 *   prompt tokens, so prompt token j is row j mod 512; AMPH_MAX_NODES with AMPH_FLAG_CHUNKED_PREFILL);
 *   "d_logits" f32 [K,V]; "hp" f32 [K,d] (Eq. 4); "attn_o" f32 [K,d] (Eq. 5);
 *   "sal_h" f32 [2,d] (Eq. 1: h^1_t, h^2_t of the last row); "tree_tokens", "argmax" i32 [n_nodes] (at T > 0
 *   "argmax" holds the sampled choices); "uniforms" f32 [n_nodes] (the uniforms of the last verification, T > 0);
 *   "kv.k.{i}", "kv.v.{i}", "sal{s}.k", "sal{s}.v": f32 [rows, d] for cache slots 0..rows-1,
 *   rows = bytes / (4 d), converted from the cache's storage type.
 * bytes must not exceed the tensor's size. */
amph_status amph_get_tensor(amph_ctx* ctx, const char* name, void* dst, size_t bytes);

/* Test hook: overwrites "tree_tokens" or "argmax" (i32 [n_nodes], host or device source) with a
 * stream-ordered copy, e.g. to run amph_accept on a chosen verification outcome.  Allowed after
 * amph_verify_tree only.  "logits" (f32 [n_nodes, vocab], T > 0 only) replaces the verified rows' logits and draws
 * the choices again from them with the same uniforms.  "root" (i32 [1]) replaces the root token; allowed right after amph_prefill only.
 * "#b" selects the sequence as for amph_get_tensor. */
amph_status amph_set_tensor(amph_ctx* ctx, const char* name, const void* src, size_t bytes);

/* Synchronises the stream and reports the committed length, the current root token and the
 * number of rows pending for the adaptation layers.  Any pointer may be NULL.  Also surfaces
 * device-side errors (AMPH_ERR_TIMEOUT).  amph_get_state reads sequence 0, amph_get_state_seq sequence seq. */
amph_status amph_get_state(amph_ctx* ctx, int32_t* ctx_len, int32_t* root, int32_t* n_pending);
amph_status amph_get_state_seq(amph_ctx* ctx, int32_t seq, int32_t* ctx_len, int32_t* root, int32_t* n_pending);

/* Teacher forcing (the counterpart of amph_get_state; sequence 0): replaces the decoding state of a prefilled sequence that has no
 * draft in flight.  ctx_len: committed tokens (the KV caches of the target and of the adaptation layers are NOT touched:
 * the caller vouches that their first ctx_len, resp. ctx_len - n_pending, slots belong to the sequence); root: the
 * token chosen for position ctx_len; the n_pending (1..K+1) rows queued for the adaptation layers (Eq. 1) sit at
 * positions ctx_len - n_pending .. ctx_len - 1: pend_hidden f32 [n_pending][d_model] (host or device) holds the
 * target's post-final-norm hidden rows h_j, pend_next (HOST, n_pending ids) the token at position j + 1 of each
 * (the last one is root).  Synchronises the stream. */
amph_status amph_set_state(amph_ctx* ctx, int32_t ctx_len, int32_t root, int32_t n_pending, const float* pend_hidden,
                           const int32_t* pend_next);

/* Per-kernel timing of the projections (the weight-streaming kernels that dominate a step).
 * Between amph_profile_begin and amph_profile_end every projection launch is bracketed by CUDA
 * events on the context's stream.  amph_profile_end synchronises the stream and reports, summed over
 * the bracketed launches: device time in milliseconds, number of launches, and weight bytes streamed
 * (each weight matrix counted once per launch).  HOST output pointers, each may be NULL.  At most
 * 16384 launches are recorded per begin / end pair; later ones run unrecorded. */
enum {
  AMPH_PROF_PROJECTION = 0,  /* weight-streaming projections                          */
  AMPH_PROF_NORM = 1,        /* split-K reduction + residual + RMSNorm               */
  AMPH_PROF_ROPE_KV = 2,     /* rotary embedding + KV-cache write                     */
  AMPH_PROF_ATTENTION = 3,   /* tree attention (+ merge of the KV splits), Eq. 5 attention */
  AMPH_PROF_SWIGLU = 4,
  AMPH_PROF_SELECT = 5,      /* top-k per drafting head, argmax per verified row       */
  AMPH_PROF_ACCEPT = 6,      /* acceptance + KV compaction                            */
  AMPH_PROF_OTHER = 7,       /* embedding, concatenation, row tables, head epilogues   */
  AMPH_PROF_CATEGORIES = 8
};
amph_status amph_profile_begin(amph_ctx* ctx);
amph_status amph_profile_end(amph_ctx* ctx, double* proj_ms, int64_t* proj_launches, int64_t* proj_weight_bytes);

/* The projection primitive on its own (the weight-streaming kernel every linear map of Eq. 1-6 and
 * of the target's layers goes through):  y[r][s*out + o] = sum_k x[r][k] * w[s][o][k]  for up to 8
 * weight matrices w[s] ([out, in] row-major, device) that share the activation rows x
 * ([x_rows_cap, in] row-major, device, same dtype as the weights; only the first `rows` are used).
 * w: HOST array of n_seg device pointers.  y: device fp32 [rows, n_seg*out].
 * use_tensor_core != 0 selects the tcgen05 kernel (bf16 only; out % 128 == 0, in % 64 == 0,
 * rows <= 512, x_rows_cap >= rows rounded up to 16, or to 128 beyond 128 rows: then every weight tile is streamed once
 * and multiplied with up to four 128-row blocks) and fails with AMPH_ERR_SHAPE if the shape is
 * not covered; 0 selects the plain CUDA-core kernel.  ws_dev: device scratch of ws_bytes >=
 * 256 + 16 * 128 * n_seg * out * 4 bytes, 256-byte aligned; its first int32 is zeroed by the call and is set to
 * AMPH_ERR_TIMEOUT if a bounded device-side wait gave up.  Stream-ordered; no context needed. */
amph_status amph_project(const void* x_dev, int32_t x_rows_cap, const void* const* w, int32_t n_seg,
                         int32_t out, int32_t in, int32_t rows, int32_t dtype, int32_t use_tensor_core,
                         float* y_dev, void* ws_dev, size_t ws_bytes, void* stream);

/* Failure-path self-test of the bounded device-side waits (no counterpart in the paper).  Runs the tensor-core
 * projection of amph_project (bf16, same arguments) with every pipeline wait limited to limit_us microseconds and the
 * first pipeline barrier of each CTA expecting 1 KB more than its copies deliver, so that this wait can never
 * complete.  Nothing faults and nothing hangs: each CTA gives up after the limit, lets its own copies land, frees its
 * tensor memory and returns; y_dev receives zeros.  After the stream has been synchronised the first int32 of ws_dev
 * reads AMPH_ERR_TIMEOUT.  The device context stays usable. */
amph_status amph_selftest_wait_timeout(const void* x_dev, int32_t x_rows_cap, const void* const* w, int32_t n_seg,
                                       int32_t out, int32_t in, int32_t rows, float* y_dev, void* ws_dev, size_t ws_bytes,
                                       void* stream, int32_t limit_us);

/* (No counterpart in the paper: a packaging variant of amph_project.)
 * The same projection for callers that cannot allocate device memory at the time of the call: for
 * example code running after a serving engine has taken all free GPU memory into its own pool, where
 * a cudaMalloc would fail, or a latency-critical loop that must not meet the implicit synchronisation
 * of an allocation.  Instead of caller-provided scratch, the split-K partial sums live in a fixed
 * array of AMPH_NOALLOC_SCRATCH_BYTES inside the library image; every GPU that loads the library
 * holds that array until the process exits.  The call allocates nothing (no cudaMalloc / cudaFree).
 * Arguments as for amph_project, except:
 *   status_dev : device int32, may be NULL; zeroed by the call, set to AMPH_ERR_TIMEOUT if a bounded
 *                device-side wait gave up (with NULL the flag is kept inside the scratch, unread);
 *   err_msg    : HOST buffer of err_len bytes that receives a message on failure, may be NULL.
 * Limit: 256 + (rows rounded up to 16) * n_seg * out * 4 bytes must not exceed
 * AMPH_NOALLOC_SCRATCH_BYTES, otherwise AMPH_ERR_WORKSPACE (nothing is launched).
 * The first call on each device looks up the array's device address (with that device current);
 * make that first call before starting any stream capture.  With CUDA's default lazy module loading the
 * library's device image, and with it the array's 16 MiB, is placed on a device the first time the
 * library is used there, which may be this first call: make it while the device still has that much
 * memory free (before another component takes all of it), or run the process with CUDA_MODULE_LOADING=EAGER;
 * otherwise the first call can fail with AMPH_ERR_CUDA.  All calls on a device share the one
 * array, which keeps the previous call's contents (the call clears what must start at zero): calls
 * whose kernels may overlap on the GPU (different streams, or several threads) race on it, so
 * serialise them.  Stream-ordered; y_dev is valid once the stream has been synchronised. */
#define AMPH_NOALLOC_SCRATCH_BYTES (16u << 20)
amph_status amph_project_noalloc(const void* x_dev, int32_t x_rows_cap, const void* const* w, int32_t n_seg,
                                 int32_t out, int32_t in, int32_t rows, int32_t dtype, int32_t use_tensor_core,
                                 float* y_dev, int32_t* status_dev, void* stream, char* err_msg, size_t err_len);

/* Per-category device time of the last amph_profile_begin / amph_profile_end pair: ms and launches are
 * HOST arrays of AMPH_PROF_CATEGORIES entries (either may be NULL).  While profiling, every kernel launch
 * (or pair: attention + merge) is bracketed by events, which serialises kernels that otherwise overlap. */
amph_status amph_profile_breakdown(amph_ctx* ctx, double* ms, int64_t* launches);

/* Forgets the sequence (caches are logically emptied); weights stay registered. */
amph_status amph_reset(amph_ctx* ctx);

void amph_destroy(amph_ctx* ctx);

/* Message of the last failure on ctx ("" if none); with ctx == NULL, of the last failed
 * amph_init / amph_workspace_bytes on this thread.  The string is owned by the library. */
const char* amph_last_error(const amph_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* AMPH_H_ */
