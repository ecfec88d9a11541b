// Host side of the Amphista step library: argument validation, workspace layout, weight
// registry and the kernel schedule of prefill / draft / verify / accept (declared in amph.h).
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <string>
#include <unordered_map>
#include <vector>

#include "amph_internal.cuh"
#include "gemm_tc.cuh"

using namespace amph;

namespace {

thread_local std::string g_last_error;

struct LayerW {
  const void *attn_norm, *wq, *wk, *wv, *wo, *ffn_norm, *w_gate, *w_up, *w_down;
};

struct TensorRec {
  const void* ptr;
  int ndim;
  int64_t shape[2];
};

constexpr int kPrefillRows = kMaxRows;           // rows of one prefill chunk (one row group)
constexpr int kMaxSeq = AMPH_MAX_BATCH;       // sequences of a context = row groups of a batched pass
constexpr int kPrefillGroups = 4;               // row groups (chunks of 128 prompt tokens) one prefill pass carries
constexpr int kSmallRows = 16;                  // rows one sequence contributes to the draft module's passes

// Offsets of every buffer inside the caller's workspace region.  A forward pass carries G row groups of equal
// height: the sequences of a batch (each with its own caches, row table and state) or consecutive chunks of one
// prompt.  Buffers marked "per group" hold kMaxSeq copies `*_stride` bytes apart; row buffers hold all groups'
// rows back to back (group g starts at row g * rows-per-group of that pass).
struct Layout {
  size_t total = 0;
  size_t take(size_t bytes) {
    const size_t off = total;
    total += (bytes + 255) / 256 * 256;
    return off;
  }
  size_t per_group(size_t bytes, size_t* stride) {
    *stride = (bytes + 255) / 256 * 256;
    return take(*stride * kMaxSeq);
  }
  // per group
  size_t state, meta_v, meta_s, kv_tab, rope_v, rope_s, topk_ids, topk_vals, topk_cand, last, d_logits, att_o, att_ml;
  size_t state_s, meta_s_, kv_tab_s, rope_s_, topk_ids_s, topk_vals_s, topk_cand_s, last_s, d_logits_s, att_o_s, att_ml_s;
  // shared
  size_t tree, inv_freq;
  size_t tok, amax, override_tok, next_tok, amax_cand, uniforms;        // [Rcap] ints / candidates / floats
  size_t x, hidden, h1, h2, pend_h, hp, attn_o;                           // fp32 rows
  size_t xn, q, att, act, cat, last_act, ao_act, aeb_act, lr_act;        // storage-type rows
  size_t partial, logits, ss_a, ss_b;
  size_t partial_floats;
  int attn_splits;
};

enum Phase { PH_CREATED = 0, PH_READY, PH_DRAFTED, PH_VERIFIED };

}  // namespace

struct amph_ctx {
  amph_config cfg;
  TreeDev tree_host;
  cudaStream_t stream;
  int dtype;
  size_t esz;
  int B;                    // sequences of this context (cfg.max_batch)
  int Mcap;                 // rows of one group at most = rows of a prefill chunk
  int Rcap;                 // rows of one pass at most (all groups)
  int Mver;                 // rows one sequence carries in a verification pass (tree nodes rounded up to 16)
  int rows_small;           // rows one sequence carries in the draft module's passes
  int small_cap;            // row capacity of the draft module's small activation buffers
  Layout lay;
  char* ws;
  char* kv;
  std::vector<KvView> kv_target[kMaxSeq];
  KvView kv_sal[kMaxSeq][2];
  std::unordered_map<std::string, TensorRec> tensors;
  bool resolved;
  const void *tok_emb, *final_norm, *lm_head, *fc[2], *pe;
  std::vector<LayerW> layers;
  LayerW sal[2];
  const void* mlp_w[kMaxK];
  const void* mlp_b[kMaxK];
  const void* aeb_w[2][4];
  const void* draft_lm[kMaxK];      // [V, d] heads, or with lm_rank > 0 the [V, r] factors
  const void* draft_lm_a[kMaxK];    // [r, d] factors (lm_rank > 0)
  Phase phase;
  bool prefilled[kMaxSeq] = {false};
  int ctx_hi[kMaxSeq] = {0};   // host-side upper bound of each sequence's committed length
  std::string err;
  TcGemm* tc;               // tensor-core projection plans (NULL when disabled / unsupported)
  AttnTc* attn_tc = nullptr; // tcgen05 tree attention (NULL: fp32 caches, disabled or unsupported)
  int sm_count = 148;
  bool last_proj_one_wave = false;   // the last projection ran on the tensor-core kernel with a fully resident grid
  cudaStream_t side = nullptr;            // forked stream of the gate / up prefetch helpers (NULL: disabled)
  std::vector<cudaEvent_t> fork_ev;       // one event per fork of a step, reused from step to step
  size_t fork_used = 0;
  cudaEvent_t join_ev = nullptr;
  bool side_dirty = false;                // helpers were launched since the last join
  cudaGraphExec_t graph_exec = nullptr;   // captured draft -> verify -> accept schedule of amph_step
  long long graph_key = -1; // attention split counts the captured grids were sized for
  bool graph_off = false;   // capture is not possible (legacy stream, flag) or failed once
  bool prof_on = false;     // bracket projection launches with events (amph_profile_begin / end)
  std::vector<cudaEvent_t> prof_ev;
  std::vector<int> prof_cat;
  size_t prof_used = 0;
  int64_t prof_bytes = 0;
  double prof_cat_ms[AMPH_PROF_CATEGORIES] = {0};
  int64_t prof_cat_n[AMPH_PROF_CATEGORIES] = {0};

  template <typename T> T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
  template <typename T> T* grp(size_t off, size_t stride, int g) const { return reinterpret_cast<T*>(ws + off + stride * g); }
  DevState* state(int b) const { return grp<DevState>(lay.state, lay.state_s, b); }
  RowMeta* meta_v(int g) const { return grp<RowMeta>(lay.meta_v, lay.meta_s_, g); }
  RowMeta* meta_s(int g) const { return grp<RowMeta>(lay.meta_s, lay.meta_s_, g); }
  int max_ctx_hi() const { int m = 0; for (int b = 0; b < B; ++b) m = ctx_hi[b] > m ? ctx_hi[b] : m; return m; }
};

namespace {

amph_status fail(amph_ctx* ctx, amph_status code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (ctx) ctx->err = buf;
  g_last_error = buf;
  return code;
}

// Brackets the launches issued during its lifetime with a pair of events (only while profiling).
struct ProfScope {
  amph_ctx* ctx;
  bool rec;
  ProfScope(amph_ctx* c, int cat) : ctx(c) {
    rec = c->prof_on && c->prof_used + 2 <= c->prof_ev.size();
    if (rec) {
      cudaEventRecord(c->prof_ev[c->prof_used], c->stream);
      c->prof_cat[c->prof_used / 2] = cat;
    }
  }
  ~ProfScope() {
    if (rec) {
      cudaEventRecord(ctx->prof_ev[ctx->prof_used + 1], ctx->stream);
      ctx->prof_used += 2;
    }
  }
};

amph_status cuda_check(amph_ctx* ctx, cudaError_t e, const char* what) {
  if (e == cudaSuccess) return AMPH_OK;
  return fail(ctx, AMPH_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

int round_up(int v, int m) { return (v + m - 1) / m * m; }

amph_status validate(const amph_config* c, const amph_tree* t, TreeDev* out) {
  if (!c || !t) return fail(nullptr, AMPH_ERR_INVALID_ARG, "config and tree must not be NULL");
  if (c->n_layers < 1 || c->d_model < 8 || c->n_heads < 1 || c->d_ffn < 8 || c->vocab < 2)
    return fail(nullptr, AMPH_ERR_SHAPE, "non-positive model dimension");
  if (c->n_heads * c->head_dim != c->d_model)
    return fail(nullptr, AMPH_ERR_SHAPE, "n_heads * head_dim (%d) != d_model (%d)", c->n_heads * c->head_dim, c->d_model);
  if (c->head_dim != 64 && c->head_dim != 128)
    return fail(nullptr, AMPH_ERR_SHAPE, "head_dim must be 64 or 128 (got %d)", c->head_dim);
  if (c->d_model % 8 || c->d_ffn % 8) return fail(nullptr, AMPH_ERR_SHAPE, "d_model and d_ffn must be multiples of 8");
  if (c->d_model > 12288) return fail(nullptr, AMPH_ERR_SHAPE, "d_model > 12288 is not supported");
  if (c->weight_dtype != AMPH_DTYPE_F32 && c->weight_dtype != AMPH_DTYPE_BF16)
    return fail(nullptr, AMPH_ERR_SHAPE, "unknown weight_dtype %d", c->weight_dtype);
  if (c->kv_dtype != c->weight_dtype) return fail(nullptr, AMPH_ERR_SHAPE, "kv_dtype must equal weight_dtype");
  if (c->max_batch < 1 || c->max_batch > kMaxSeq) return fail(nullptr, AMPH_ERR_SHAPE, "max_batch must be in 1..%d", kMaxSeq);
  if (c->K < 1 || c->K > kMaxK) return fail(nullptr, AMPH_ERR_SHAPE, "K must be in 1..%d", kMaxK);
  if (c->n_sal < 0 || c->n_sal > 2) return fail(nullptr, AMPH_ERR_SHAPE, "n_sal must be 0, 1 or 2");
  if (c->aeb_layers < 0 || c->aeb_layers > 2) return fail(nullptr, AMPH_ERR_SHAPE, "aeb_layers must be 0, 1 or 2");
  if (c->lm_rank < 0 || c->lm_rank > c->d_model || c->lm_rank % 8) return fail(nullptr, AMPH_ERR_SHAPE, "lm_rank must be 0 or a multiple of 8 up to d_model");
  for (int k = 0; k < c->K; ++k)
    if (c->topk[k] < 1 || c->topk[k] > kTopkStride || c->topk[k] > c->vocab)
      return fail(nullptr, AMPH_ERR_SHAPE, "topk[%d] = %d out of range 1..%d", k, c->topk[k], kTopkStride);
  if (!(c->rms_eps >= 0.f) || !(c->rope_theta > 1.f)) return fail(nullptr, AMPH_ERR_SHAPE, "bad rms_eps / rope_theta");
  if (!(c->temperature >= 0.f) || !(c->temperature < 1e6f)) return fail(nullptr, AMPH_ERR_SHAPE, "temperature must be 0 (greedy) or positive and finite");
  if (t->n_nodes < 1 || t->n_nodes > kMaxRows) return fail(nullptr, AMPH_ERR_SHAPE, "n_nodes must be in 1..%d", kMaxRows);
  if (!t->parent || !t->depth || !t->rank) return fail(nullptr, AMPH_ERR_INVALID_ARG, "tree arrays must not be NULL");
  if (c->max_batch * round_up(t->n_nodes < 16 ? 16 : t->n_nodes, 16) > kPrefillGroups * kMaxRows)
    return fail(nullptr, AMPH_ERR_SHAPE, "max_batch * tree nodes (rounded up to 16) must not exceed %d rows", kPrefillGroups * kMaxRows);
  if (c->max_ctx < t->n_nodes + 1) return fail(nullptr, AMPH_ERR_SHAPE, "max_ctx must exceed n_nodes");
  TreeDev td;
  memset(&td, 0, sizeof td);
  td.n_nodes = t->n_nodes;
  for (int n = 0; n < t->n_nodes; ++n) {
    const int p = t->parent[n], dep = t->depth[n];
    if (n == 0) {
      if (p != -1 || dep != 0) return fail(nullptr, AMPH_ERR_SHAPE, "node 0 must be the root (parent -1, depth 0)");
      td.anc[0][0] = 1ull;
    } else {
      if (p < 0 || p >= n) return fail(nullptr, AMPH_ERR_SHAPE, "parent[%d] = %d must be in 0..%d", n, p, n - 1);
      if (dep != td.depth[p] + 1) return fail(nullptr, AMPH_ERR_SHAPE, "depth[%d] must be depth[parent] + 1", n);
      if (dep > c->K) return fail(nullptr, AMPH_ERR_SHAPE, "depth[%d] = %d exceeds K = %d", n, dep, c->K);
      if (t->rank[n] >= c->topk[dep - 1])
        return fail(nullptr, AMPH_ERR_SHAPE, "rank[%d] = %d needs topk[%d] > %d", n, t->rank[n], dep - 1, t->rank[n]);
      td.anc[n][0] = td.anc[p][0];
      td.anc[n][1] = td.anc[p][1];
      td.anc[n][n >> 6] |= 1ull << (n & 63);
    }
    td.parent[n] = p;
    td.depth[n] = dep;
    td.rank[n] = t->rank[n];
  }
  if (out) *out = td;
  return AMPH_OK;
}

void make_layout(const amph_config& c, int n_nodes, Layout* L, int* Mcap_out, size_t* kv_bytes, int* Mver_out = nullptr,
                 int* Rcap_out = nullptr, int* small_cap_out = nullptr) {
  const int Mver = round_up(n_nodes < 16 ? 16 : n_nodes, 16);
  const int Mcap = Mver > kPrefillRows ? Mver : kPrefillRows;
  const int B = c.max_batch;
  int Rcap = kPrefillGroups * kPrefillRows;                   // a dense prefill pass
  if (B * Mver > Rcap) Rcap = B * Mver;
  const int small_cap = round_up(B * (c.K > 2 ? c.K : 2) > B * kSmallRows ? B * c.K : B * kSmallRows, 16);
  if (Mver_out) *Mver_out = Mver;
  if (Rcap_out) *Rcap_out = Rcap;
  if (small_cap_out) *small_cap_out = small_cap;
  const size_t esz = c.weight_dtype == AMPH_DTYPE_F32 ? 4 : 2;
  const size_t d = c.d_model, F = c.d_ffn, V = c.vocab, half = c.head_dim / 2;
  Layout l;
  l.state = l.per_group(sizeof(DevState), &l.state_s);
  l.meta_v = l.per_group(sizeof(RowMeta), &l.meta_s_);
  l.meta_s = l.per_group(sizeof(RowMeta), &l.meta_s_);
  l.kv_tab = l.per_group(sizeof(KvView) * c.n_layers, &l.kv_tab_s);
  l.rope_v = l.per_group(sizeof(float2) * Mcap * half, &l.rope_s_);
  l.rope_s = l.per_group(sizeof(float2) * Mcap * half, &l.rope_s_);
  l.topk_ids = l.per_group(sizeof(int) * kMaxK * kTopkStride, &l.topk_ids_s);
  l.topk_vals = l.per_group(sizeof(float) * kMaxK * kTopkStride, &l.topk_vals_s);
  l.topk_cand = l.per_group(2 * sizeof(float) * kMaxK * kTopkCandChunks * kTopkStride, &l.topk_cand_s);
  l.last = l.per_group(4 * 2 * d, &l.last_s);
  l.d_logits = l.per_group(4 * (size_t)kMaxK * V, &l.d_logits_s);
  l.tree = l.take(sizeof(TreeDev));
  l.inv_freq = l.take(sizeof(double) * half);
  l.tok = l.take(sizeof(int) * Rcap);
  l.amax = l.take(sizeof(int) * Rcap);
  l.override_tok = l.take(sizeof(int) * Rcap);
  l.next_tok = l.take(sizeof(int) * Rcap);
  l.amax_cand = l.take(2 * sizeof(float) * Rcap * 8);
  l.uniforms = l.take(sizeof(float) * Rcap);
  l.x = l.take(4 * Rcap * d);
  l.hidden = l.take(4 * Rcap * d);
  l.h1 = l.take(4 * Rcap * d);
  l.h2 = l.take(4 * Rcap * d);
  l.pend_h = l.take(4 * (size_t)kMaxSeq * kSmallRows * d);     // [sequence][16][d]: the rows of a draft pass back to back
  l.hp = l.take(4 * (size_t)kMaxSeq * kMaxK * d);               // [sequence][K][d]
  l.attn_o = l.take(4 * (size_t)small_cap * d);                 // [sequence * K + k][d]
  l.xn = l.take(esz * Rcap * d);
  l.q = l.take(esz * Rcap * d);
  l.att = l.take(esz * Rcap * d);
  l.act = l.take(esz * Rcap * F);
  l.cat = l.take(esz * Rcap * 2 * d);
  l.last_act = l.take(esz * small_cap * d);
  l.ao_act = l.take(esz * small_cap * d);
  l.aeb_act = l.take(esz * small_cap * d);
  l.lr_act = l.take(esz * small_cap * (size_t)(c.lm_rank > 0 ? c.lm_rank : 8));
  size_t big = 3 * d > 2 * F ? 3 * d : 2 * F;
  size_t pf = 4 * (size_t)Rcap * big;                       // room for 4 K-splits of the widest projection
  if (2 * (size_t)Rcap * V > pf) pf = 2 * (size_t)Rcap * V;
  if ((size_t)small_cap * c.K * V > pf) pf = (size_t)small_cap * c.K * V;
  l.partial_floats = pf;
  l.partial = l.take(4 * pf);
  int splits = (296 + c.n_heads - 1) / c.n_heads;
  if (splits > 8) splits = 8;                               // the KV splits of a head run as one thread-block cluster (<= 8 CTAs)
  l.attn_splits = splits;
  l.att_o = l.per_group(4 * (size_t)splits * c.n_heads * Mcap * c.head_dim, &l.att_o_s);
  l.att_ml = l.per_group(4 * (size_t)splits * c.n_heads * Mcap * 2, &l.att_ml_s);
  l.logits = l.take(4 * (size_t)Rcap * V);
  l.ss_a = l.take(4 * (size_t)Rcap * 32);
  l.ss_b = l.take(4 * (size_t)Rcap * 32);
  *L = l;
  *Mcap_out = Mcap;
  const size_t per_layer = 2 * (size_t)c.n_heads * c.max_ctx * c.head_dim * esz;
  *kv_bytes = per_layer * (c.n_layers + c.n_sal) * B;
}

// ---- weights ------------------------------------------------------------------------------
const void* find(amph_ctx* ctx, const std::string& name, int64_t s0, int64_t s1, bool* ok) {
  auto it = ctx->tensors.find(name);
  if (it == ctx->tensors.end()) {
    if (*ok) fail(ctx, AMPH_ERR_MISSING_WEIGHT, "weight '%s' was never loaded", name.c_str());
    *ok = false;
    return nullptr;
  }
  const TensorRec& t = it->second;
  const bool shape_ok = s1 == 0 ? (t.ndim == 1 && t.shape[0] == s0) : (t.ndim == 2 && t.shape[0] == s0 && t.shape[1] == s1);
  if (!shape_ok) {
    if (*ok) fail(ctx, AMPH_ERR_MISSING_WEIGHT, "weight '%s' has the wrong shape", name.c_str());
    *ok = false;
    return nullptr;
  }
  return t.ptr;
}

bool resolve_layer(amph_ctx* ctx, const std::string& pre, LayerW* w, bool* ok) {
  const int64_t d = ctx->cfg.d_model, F = ctx->cfg.d_ffn;
  w->attn_norm = find(ctx, pre + "attn_norm", d, 0, ok);
  w->wq = find(ctx, pre + "wq", d, d, ok);
  w->wk = find(ctx, pre + "wk", d, d, ok);
  w->wv = find(ctx, pre + "wv", d, d, ok);
  w->wo = find(ctx, pre + "wo", d, d, ok);
  w->ffn_norm = find(ctx, pre + "ffn_norm", d, 0, ok);
  w->w_gate = find(ctx, pre + "w_gate", F, d, ok);
  w->w_up = find(ctx, pre + "w_up", F, d, ok);
  w->w_down = find(ctx, pre + "w_down", d, F, ok);
  return *ok;
}

amph_status resolve(amph_ctx* ctx) {
  if (ctx->resolved) return AMPH_OK;
  const amph_config& c = ctx->cfg;
  const int64_t d = c.d_model, V = c.vocab;
  bool ok = true;
  ctx->tok_emb = find(ctx, "tok_emb", V, d, &ok);
  ctx->final_norm = find(ctx, "final_norm", d, 0, &ok);
  ctx->lm_head = find(ctx, "lm_head", V, d, &ok);
  ctx->layers.resize(c.n_layers);
  for (int i = 0; i < c.n_layers; ++i) resolve_layer(ctx, "layers." + std::to_string(i) + ".", &ctx->layers[i], &ok);
  for (int s = 0; s < c.n_sal; ++s) {
    ctx->fc[s] = find(ctx, "draft.fc" + std::to_string(s + 1), d, (c.flags & AMPH_FLAG_NO_SAMPLED_TOKEN) ? d : 2 * d, &ok);
    resolve_layer(ctx, "draft.sal" + std::to_string(s + 1) + ".", &ctx->sal[s], &ok);
  }
  for (int k = 0; k < c.K; ++k) {
    ctx->mlp_w[k] = find(ctx, "draft.mlp." + std::to_string(k) + ".w", d, d, &ok);
    ctx->mlp_b[k] = find(ctx, "draft.mlp." + std::to_string(k) + ".b", d, 0, &ok);
    if (c.lm_rank > 0) {
      ctx->draft_lm_a[k] = find(ctx, "draft.lm_head." + std::to_string(k) + ".a", c.lm_rank, d, &ok);
      ctx->draft_lm[k] = find(ctx, "draft.lm_head." + std::to_string(k) + ".b", V, c.lm_rank, &ok);
    } else {
      ctx->draft_lm[k] = find(ctx, "draft.lm_head." + std::to_string(k), V, d, &ok);
    }
  }
  ctx->pe = find(ctx, "draft.pe", c.K, d, &ok);
  static const char* names[4] = {"wq", "wk", "wv", "wo"};
  for (int l = 0; l < c.aeb_layers; ++l)
    for (int j = 0; j < 4; ++j)
      ctx->aeb_w[l][j] = find(ctx, "draft.aeb." + std::to_string(l) + "." + names[j], d, d, &ok);
  if (!ok) return AMPH_ERR_MISSING_WEIGHT;
  ctx->resolved = true;
  return AMPH_OK;
}

// ---- projections --------------------------------------------------------------------------
// Y = X W^T for up to four weight matrices that share X; the result is left as fp32 partial sums.
enum XBuf { XB_XN = 0, XB_ATT, XB_ACT, XB_CAT, XB_LAST, XB_AO, XB_AEB, XB_LR, XB_COUNT };

void* xbuf_ptr(amph_ctx* ctx, int xb) {
  const Layout& l = ctx->lay;
  const size_t off[XB_COUNT] = {l.xn, l.att, l.act, l.cat, l.last_act, l.ao_act, l.aeb_act, l.lr_act};
  return ctx->ws + off[xb];
}

PartialView project_impl(amph_ctx* ctx, int xb, const void* const* w, int n_seg, int out, int in, int rows);

PartialView project(amph_ctx* ctx, int xb, const void* const* w, int n_seg, int out, int in, int rows) {
  ProfScope ps(ctx, AMPH_PROF_PROJECTION);
  if (ps.rec) ctx->prof_bytes += (int64_t)n_seg * out * in * (int64_t)ctx->esz;
  return project_impl(ctx, xb, w, n_seg, out, in, rows);
}

PartialView project_impl(amph_ctx* ctx, int xb, const void* const* w, int n_seg, int out, int in, int rows) {
  float* P = ctx->at<float>(ctx->lay.partial);
  PartialView pv;
  ctx->last_proj_one_wave = false;
  if (ctx->tc) {
    int splits = 0;
    size_t stride = 0;
    if (tc_gemm_launch(ctx->tc, xb, w, n_seg, out, in, rows, P, ctx->lay.partial_floats, &splits, &stride,
                       ctx->stream)) {
      ctx->last_proj_one_wave = (long long)n_seg * (out / 128) * splits <= 2LL * ctx->sm_count;
      pv.p = P;
      pv.splits = splits;
      pv.ld = n_seg * out;
      pv.split_stride = stride;
      return pv;
    }
  }
  GemmSeg segs[kMaxK];
  for (int s = 0; s < n_seg; ++s) segs[s].w = w[s];
  launch_gemm_generic(xbuf_ptr(ctx, xb), in, segs, n_seg, out, in, P, n_seg * out, rows, ctx->dtype, ctx->stream);
  pv.p = P;
  pv.splits = 1;
  pv.ld = n_seg * out;
  pv.split_stride = 0;
  return pv;
}

RowScale row_scale_of(const amph_ctx* ctx, size_t off) {
  RowScale rs;
  rs.ss = ctx->at<float>(off);
  rs.chunks = (ctx->cfg.d_model + kScaleChunkCols - 1) / kScaleChunkCols;
  rs.d = ctx->cfg.d_model;
  rs.eps = ctx->cfg.rms_eps;
  return rs;
}

// A forward pass: G row groups of rpg rows each.  Group g uses row table meta[g], rotary table rope[g], the caches of
// sequence seq[g], and may see at most keys[g] cache slots (host-side bound: committed slots + the rows of the pass).
struct Pass {
  int G = 1;
  int rpg = 0;
  const RowMeta* meta[kMaxSeq];
  float2* rope[kMaxSeq];
  int seq[kMaxSeq];
  int keys[kMaxSeq];
  int rows() const { return G * rpg; }
};

PartialView rows_from(PartialView P, int row0) {
  P.p += (size_t)row0 * P.ld;
  return P;
}
RowScale rows_from(RowScale rs, int row0) {
  if (rs.ss) rs.ss += (size_t)row0 * rs.chunks;
  return rs;
}

void pass_rope_tables(amph_ctx* ctx, const Pass& ps) {
  for (int g = 0; g < ps.G; ++g) {
    ProfScope p(ctx, AMPH_PROF_OTHER);
    launch_rope_table(ps.meta[g], ctx->at<double>(ctx->lay.inv_freq), ps.rope[g], ps.rpg, ctx->cfg.head_dim / 2, ctx->stream);
  }
}

// While attention, the output projection and the residual kernel of a layer run, HBM is nearly idle (they are latency
// chains over L2-resident data).  A helper on a forked stream uses that window to pull the head of the layer's gate / up
// weights (kGateUpPrefetchBytes, about a third of them at 7B) into L2, so that the gate / up projection starts on L2 hits.
// Forked right after the q / k / v projection is launched: measured -1.5 % per step; forked after the attention or the output
// projection it costs 2-5 % (an event between two programmatically dependent launches), as does a larger budget.
constexpr size_t kGateUpPrefetchBytes = 56u << 20;

void fork_prefetch(amph_ctx* ctx, const LayerW& w, int rows) {
  if (!(ctx->side && ctx->tc && rows <= 64)) return;
  const amph_config& c = ctx->cfg;
  // a gate / up launch of about a full wave (two CTAs per SM) gains nothing: measured +0.3 % at d_ffn = 17920 (280 tiles)
  if (c.d_ffn / 64 > ctx->sm_count * 2 * 13 / 16) return;
  // only inside the captured schedule of amph_step: launched call by call, the host-side fork and join cost more than the
  // prefetch gains (measured +95 us per step on the draft / verify / accept path)
  cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(ctx->stream, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusActive) { cudaGetLastError(); return; }
  if (ctx->fork_used == ctx->fork_ev.size()) { cudaEvent_t e; cudaEventCreateWithFlags(&e, cudaEventDisableTiming); ctx->fork_ev.push_back(e); }
  cudaEvent_t e = ctx->fork_ev[ctx->fork_used++];
  cudaEventRecord(e, ctx->stream);
  cudaStreamWaitEvent(ctx->side, e, 0);
  tc_gemm_prefetch_swiglu(ctx->tc, w.w_gate, w.w_up, c.d_ffn, c.d_model, kGateUpPrefetchBytes, ctx->side);
  ctx->side_dirty = true;
}

// One decoder layer over the rows of the pass; cache_of(seq) gives the layer's cache of a sequence.
// Entry: xn holds the input of the q/k/v projections: attn_norm * x / rms(x) if !entry_deferred, else
// attn_norm * x with the row sums of squares in ss_a (the division is applied after the projection).
// Exit: x is updated.  With next_gain and no hid: xn = next_gain * x, sums of squares in ss_a (deferred form
// for the next layer; returns true).  With hid: xn and hid hold the normalised rows (returns false).
template <typename CacheOf>
bool layer_forward(amph_ctx* ctx, const LayerW& w, CacheOf cache_of, float* x, const Pass& ps, const void* next_gain,
                   float* hid, bool entry_deferred) {
  const amph_config& c = ctx->cfg;
  const Layout& l = ctx->lay;
  cudaStream_t st = ctx->stream;
  const int rows = ps.rows();
  const size_t d = c.d_model;
  const void* qkv[3] = {w.wq, w.wk, w.wv};
  const RowScale rs = entry_deferred ? row_scale_of(ctx, l.ss_a) : RowScale();
  PartialView P = {nullptr, 0, 0, 0};
  bool fused_rope = false;
  if (ctx->tc && ps.G == 1 && !(c.flags & AMPH_FLAG_SEPARATE_ROPE)) {   // q / k / v projection that rotates and writes the cache itself
    ProfScope p(ctx, AMPH_PROF_PROJECTION);
    fused_rope = tc_gemm_launch_qkv_rope(ctx->tc, XB_XN, w.wq, w.wk, w.wv, c.n_heads, c.head_dim, c.d_model, rows, ctx->ws + l.q,
                                         cache_of(ps.seq[0]), ps.meta[0], ps.rope[0], c.max_ctx, rs, st);
    if (fused_rope && p.rec) ctx->prof_bytes += 3LL * c.d_model * c.d_model * (int64_t)ctx->esz;
    if (!fused_rope) cudaGetLastError();
  }
  if (!fused_rope) P = project(ctx, XB_XN, qkv, 3, c.d_model, c.d_model, rows);
  if (fused_rope) fork_prefetch(ctx, w, rows);
  bool grouped_rope = false;
  if (!fused_rope && ps.G > 1) {                      // every group's rotary embedding + cache write in one launch
    ProfScope p(ctx, AMPH_PROF_ROPE_KV);
    RopeGroups gr;
    gr.G = ps.G;
    gr.rpg = ps.rpg;
    for (int g = 0; g < ps.G; ++g) {
      const KvView kv = cache_of(ps.seq[g]);
      gr.meta[g] = ps.meta[g]; gr.rope[g] = ps.rope[g]; gr.kc[g] = kv.k; gr.vc[g] = kv.v;
    }
    launch_qkv_rope_groups(P, gr, ctx->ws + l.q, ctx->dtype, c.n_heads, c.head_dim, c.max_ctx, st, rs);
    grouped_rope = true;
  }
  for (int g = 0; g < ps.G && !fused_rope && !grouped_rope; ++g) {     // rotary embedding + cache write, per group (its own cache and slots)
    ProfScope p(ctx, AMPH_PROF_ROPE_KV);
    launch_qkv_rope(rows_from(P, g * ps.rpg), ps.meta[g], ps.rope[g], ctx->ws + l.q + ctx->esz * g * ps.rpg * d, cache_of(ps.seq[g]),
                    ctx->dtype, ps.rpg, c.n_heads, c.head_dim, c.max_ctx, st, rows_from(rs, g * ps.rpg));
  }
  bool grouped_attn = false;
  if (ctx->attn_tc && ps.G > 1 && !(c.flags & AMPH_FLAG_SEPARATE_MERGE)) {   // every group's tree attention in one launch
    ProfScope p(ctx, AMPH_PROF_ATTENTION);
    KvView kvs[kMaxSeq];
    int keys = 0;
    for (int g = 0; g < ps.G; ++g) { kvs[g] = cache_of(ps.seq[g]); keys = ps.keys[g] > keys ? ps.keys[g] : keys; }
    const int splits = attn_tc_splits(ctx->attn_tc, keys, c.n_heads, ps.rpg, l.attn_splits);
    grouped_attn = launch_tree_attention_tc_groups(ctx->attn_tc, ctx->ws + l.q, ctx->Rcap, ps.G, kvs, ps.meta, ps.rpg, c.n_heads,
                                                   c.head_dim, c.max_ctx, splits, keys, st, ctx->ws + l.att, &ctx->state(0)->err);
    if (!grouped_attn) cudaGetLastError();
  }
  for (int g = 0; g < ps.G && !grouped_attn; ++g) {   // tree attention, per group
    ProfScope p(ctx, AMPH_PROF_ATTENTION);
    const KvView kv = cache_of(ps.seq[g]);
    AttnScratch sc = {ctx->grp<float>(l.att_o, l.att_o_s, g), ctx->grp<float>(l.att_ml, l.att_ml_s, g)};
    char* qg = ctx->ws + l.q + ctx->esz * g * ps.rpg * d;
    char* og = ctx->ws + l.att + ctx->esz * g * ps.rpg * d;
    const bool last_g = g + 1 == ps.G;
    bool done = false;
    if (ctx->attn_tc) {
      const int splits = attn_tc_splits(ctx->attn_tc, ps.keys[g], c.n_heads, ps.rpg, l.attn_splits);
      const bool merged = !(c.flags & AMPH_FLAG_SEPARATE_MERGE);
      done = launch_tree_attention_tc(ctx->attn_tc, qg, ctx->Rcap - g * ps.rpg, kv, ps.meta[g], sc, ps.rpg, c.n_heads, c.head_dim,
                                      c.max_ctx, splits, ps.keys[g], st, merged ? og : nullptr, &ctx->state(0)->err);
      if (done && !merged)
        launch_attn_combine(sc, og, ctx->dtype, splits, ps.rpg, c.n_heads, c.head_dim, st, last_g && ctx->tc != nullptr);
      if (!done) cudaGetLastError();
    }
    if (!done)
      launch_tree_attention(qg, kv, ps.meta[g], sc, og, ctx->dtype, ps.rpg, c.n_heads, c.head_dim, c.max_ctx, ps.keys[g],
                            l.attn_splits, st, last_g && ctx->tc != nullptr, (c.flags & AMPH_FLAG_SEPARATE_MERGE) != 0);
  }
  const void* wo[1] = {w.wo};
  P = project(ctx, XB_ATT, wo, 1, c.d_model, c.d_model, rows);
  { ProfScope p(ctx, AMPH_PROF_NORM);
  launch_resid_scale(x, P, 0, 1, w.ffn_norm, ctx->dtype, ctx->ws + l.xn, ctx->at<float>(l.ss_b), rows, c.d_model, st,
                     ctx->last_proj_one_wave);
  }
  bool fused_gu = false;
  if (ctx->tc && !(c.flags & AMPH_FLAG_SEPARATE_SWIGLU)) {         // gate / up projection with SwiGLU in its epilogue
    ProfScope p(ctx, AMPH_PROF_PROJECTION);
    fused_gu = tc_gemm_launch_swiglu(ctx->tc, XB_XN, w.w_gate, w.w_up, c.d_ffn, c.d_model, rows, ctx->ws + l.act,
                                     row_scale_of(ctx, l.ss_b), st);
    if (fused_gu && p.rec) ctx->prof_bytes += 2LL * c.d_ffn * c.d_model * (int64_t)ctx->esz;
    if (fused_gu) ctx->last_proj_one_wave = false;
  }
  if (!fused_gu) {
    const void* gu[2] = {w.w_gate, w.w_up};
    P = project(ctx, XB_XN, gu, 2, c.d_ffn, c.d_model, rows);
    ProfScope p(ctx, AMPH_PROF_SWIGLU);
    launch_swiglu(P, ctx->ws + l.act, ctx->dtype, rows, c.d_ffn, st, row_scale_of(ctx, l.ss_b), ctx->last_proj_one_wave);
  }
  const void* wd[1] = {w.w_down};
  P = project(ctx, XB_ACT, wd, 1, c.d_model, c.d_ffn, rows);
  ProfScope p(ctx, AMPH_PROF_NORM);
  if (hid != nullptr) {
    launch_resid_norm(x, P, 0, 1, next_gain, ctx->dtype, ctx->ws + l.xn, hid, c.rms_eps, rows, c.d_model, st);
    return false;
  }
  launch_resid_scale(x, P, 0, 1, next_gain, ctx->dtype, ctx->ws + l.xn, ctx->at<float>(l.ss_a), rows, c.d_model, st,
                     ctx->last_proj_one_wave && next_gain != nullptr);
  return next_gain != nullptr;
}

// Target forward of the tokens in `tok` (one per row of the pass); leaves post-final-norm rows in hidden and xn.
void target_forward(amph_ctx* ctx, const Pass& ps) {
  const amph_config& c = ctx->cfg;
  const Layout& l = ctx->lay;
  cudaStream_t st = ctx->stream;
  const int rows = ps.rows();
  float* x = ctx->at<float>(l.x);
  pass_rope_tables(ctx, ps);
  { ProfScope p(ctx, AMPH_PROF_OTHER);
  launch_embed(ctx->tok_emb, ctx->dtype, ctx->at<int>(l.tok), c.vocab, rows, c.d_model, x, st);
  }
  PartialView none = {nullptr, 0, 0, 0};
  { ProfScope p(ctx, AMPH_PROF_NORM);
  launch_resid_norm(x, none, 0, 0, ctx->layers[0].attn_norm, ctx->dtype, ctx->ws + l.xn, nullptr, c.rms_eps, rows,
                    c.d_model, st);
  }
  bool deferred = false;
  for (int i = 0; i < c.n_layers; ++i) {
    const bool last = i + 1 == c.n_layers;
    deferred = layer_forward(ctx, ctx->layers[i], [&](int b) { return ctx->kv_target[b][i]; }, x, ps,
                             last ? ctx->final_norm : ctx->layers[i + 1].attn_norm,
                             last ? ctx->at<float>(l.hidden) : nullptr, deferred);
  }
}

void target_head(amph_ctx* ctx, int rows) {
  const amph_config& c = ctx->cfg;
  const Layout& l = ctx->lay;
  const void* w[1] = {ctx->lm_head};
  PartialView P = project(ctx, XB_XN, w, 1, c.vocab, c.d_model, rows);
  { ProfScope p(ctx, AMPH_PROF_SELECT);
  launch_argmax_rows(P, c.vocab, rows, ctx->at<int>(l.amax), ctx->at<float>(l.logits), ctx->at<float>(l.amax_cand), ctx->stream);
  }
}

// Eq. 1: both adaptation stages over the rows of the pass.  feat: fp32 rows [rows][d]; next_tok[g]: the ids of the
// tokens that follow group g's rows (rpg entries).
void run_sals(amph_ctx* ctx, const float* feat, const int* const* next_tok, const Pass& ps) {
  const amph_config& c = ctx->cfg;
  const Layout& l = ctx->lay;
  cudaStream_t st = ctx->stream;
  const int rows = ps.rows();
  const bool with_tok = !(c.flags & AMPH_FLAG_NO_SAMPLED_TOKEN);             // Section 4.5, "w/o Sampled-Token"
  const size_t cat_pitch = (with_tok ? 2 : 1) * (size_t)c.d_model * ctx->esz;
  pass_rope_tables(ctx, ps);
  const float* in_feat = feat;
  for (int s = 0; s < c.n_sal; ++s) {
    float* hbuf = ctx->at<float>(s == 0 ? l.h1 : l.h2);
    for (int g = 0; g < ps.G; ++g) {
      ProfScope p(ctx, AMPH_PROF_OTHER);
      launch_concat(in_feat + (size_t)g * ps.rpg * c.d_model, with_tok ? ctx->tok_emb : nullptr, next_tok[g], c.vocab,
                    ctx->ws + l.cat + cat_pitch * g * ps.rpg, ctx->dtype, ps.rpg, c.d_model, st);
    }
    const void* w[1] = {ctx->fc[s]};
    PartialView P = project(ctx, XB_CAT, w, 1, c.d_model, (with_tok ? 2 : 1) * c.d_model, rows);
    { ProfScope p(ctx, AMPH_PROF_NORM);
    launch_resid_norm(hbuf, P, 0, 2, ctx->sal[s].attn_norm, ctx->dtype, ctx->ws + l.xn, nullptr, c.rms_eps, rows,
                      c.d_model, st);
    }
    layer_forward(ctx, ctx->sal[s], [&](int b) { return ctx->kv_sal[b][s]; }, hbuf, ps, nullptr, nullptr, false);
    in_feat = hbuf;
  }
}

amph_status copy_out(amph_ctx* ctx, void* dst, const void* src, size_t bytes) {
  if (!dst) return AMPH_OK;
  return cuda_check(ctx, cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDefault, ctx->stream), "copy of a result");
}

amph_status finish(amph_ctx* ctx, const char* what) { return cuda_check(ctx, cudaGetLastError(), what); }

amph_status refresh_ctx_hi(amph_ctx* ctx) {
  for (int b = 0; b < ctx->B; ++b) {
    if (!ctx->prefilled[b]) continue;
    DevState s;
    cudaError_t e = cudaMemcpyAsync(&s, ctx->state(b), sizeof s, cudaMemcpyDeviceToHost, ctx->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
    if (e != cudaSuccess) return cuda_check(ctx, e, "state read-back");
    ctx->ctx_hi[b] = s.C;
    if (s.err) return fail(ctx, s.err, "a device-side wait gave up (code %d)", s.err);
  }
  return AMPH_OK;
}

// out_ids / out_vals: [B][K][AMPH_TOPK_STRIDE]
amph_status do_draft(amph_ctx* ctx, int32_t* out_ids, float* out_vals) {
  const amph_config& c = ctx->cfg;
  const Layout& l = ctx->lay;
  cudaStream_t st = ctx->stream;
  const int B = ctx->B, K = c.K;
  const size_t d = c.d_model;
  Pass ps;
  ps.G = B;
  ps.rpg = ctx->rows_small;
  const int* next_tok[kMaxSeq];
  for (int b = 0; b < B; ++b) {
    ps.meta[b] = ctx->meta_s(b);
    ps.rope[b] = ctx->grp<float2>(l.rope_s, l.rope_s_, b);
    ps.seq[b] = b;
    ps.keys[b] = ctx->ctx_hi[b];
    next_tok[b] = ctx->state(b)->pend_tok;
    ProfScope p(ctx, AMPH_PROF_OTHER);
    launch_meta_pending(ctx->meta_s(b), ctx->state(b), st);
  }
  float* pend_h = ctx->at<float>(l.pend_h);            // [B][16][d] = the rows of this pass
  run_sals(ctx, pend_h, next_tok, ps);
  // without adaptation layers (the "w/o Staged-Adaptation" ablation) every head reads the target's hidden state itself
  const float* s1 = c.n_sal == 0 ? pend_h : ctx->at<float>(l.h1);
  const float* s2 = c.n_sal == 0 ? pend_h : ctx->at<float>(c.n_sal == 2 ? l.h2 : l.h1);
  for (int b = 0; b < B; ++b) {                        // rows 2 b, 2 b + 1 of the head MLPs' input: the last row of each stage
    ProfScope p(ctx, AMPH_PROF_OTHER);
    launch_gather_last(s1 + (size_t)b * ps.rpg * d, s2 + (size_t)b * ps.rpg * d, ctx->state(b), ctx->grp<float>(l.last, l.last_s, b),
                       ctx->ws + l.last_act + ctx->esz * 2 * b * d, ctx->dtype, c.d_model, st);
  }
  PartialView P = project(ctx, XB_LAST, ctx->mlp_w, K, c.d_model, c.d_model, 2 * B);                 // Eq. 2
  float* hp = ctx->at<float>(l.hp);
  float* ao = ctx->at<float>(l.attn_o);
  for (int b = 0; b < B; ++b) {                                                                       // Eq. 3-4
    ProfScope p(ctx, AMPH_PROF_OTHER);
    launch_mlp_heads(rows_from(P, 2 * b), ctx->grp<float>(l.last, l.last_s, b), ctx->mlp_b, ctx->pe, hp + (size_t)b * kMaxK * d,
                     ao + (size_t)b * K * d, ctx->ws + l.ao_act + ctx->esz * b * K * d, ctx->dtype, K, c.n_sal, c.d_model, st);
  }
  for (int a = 0; a < c.aeb_layers; ++a) {                                                            // Eq. 5
    P = project(ctx, XB_AO, ctx->aeb_w[a], 3, c.d_model, c.d_model, B * K);
    for (int b = 0; b < B; ++b) {                       // the K rows of a sequence attend to each other only
      ProfScope p(ctx, AMPH_PROF_ATTENTION);
      launch_aeb_attention(rows_from(P, b * K), ctx->ws + l.aeb_act + ctx->esz * b * K * d, ctx->dtype, K, c.n_heads, c.head_dim, st);
    }
    const void* wo[1] = {ctx->aeb_w[a][3]};
    P = project(ctx, XB_AEB, wo, 1, c.d_model, c.d_model, B * K);
    { ProfScope p(ctx, AMPH_PROF_NORM);
    launch_resid_norm(ao, P, 0, 1, nullptr, ctx->dtype, ctx->ws + l.ao_act, nullptr, c.rms_eps, B * K, c.d_model, st);
    }
  }
  if (c.lm_rank > 0) {                                                                                // Appendix A.2.4
    P = project(ctx, XB_AO, ctx->draft_lm_a, K, c.lm_rank, c.d_model, B * K);
    for (int b = 0; b < B; ++b) {
      ProfScope p(ctx, AMPH_PROF_OTHER);
      launch_gather_diag(rows_from(P, b * K), ctx->ws + l.lr_act + ctx->esz * b * K * (size_t)c.lm_rank, ctx->dtype, K, c.lm_rank, st);
    }
    P = project(ctx, XB_LR, ctx->draft_lm, K, c.vocab, c.lm_rank, B * K);
  } else {
    P = project(ctx, XB_AO, ctx->draft_lm, K, c.vocab, c.d_model, B * K);                             // Eq. 6
  }
  for (int b = 0; b < B; ++b) {
    { ProfScope p(ctx, AMPH_PROF_SELECT);
    launch_topk_heads(rows_from(P, b * K), c.vocab, K, c.topk, ctx->grp<int>(l.topk_ids, l.topk_ids_s, b),
                      ctx->grp<float>(l.topk_vals, l.topk_vals_s, b), ctx->grp<float>(l.d_logits, l.d_logits_s, b),
                      ctx->grp<float>(l.topk_cand, l.topk_cand_s, b), st);
    }
    { ProfScope p(ctx, AMPH_PROF_OTHER);
    launch_tree_build(ctx->at<TreeDev>(l.tree), ctx->state(b), ctx->grp<int>(l.topk_ids, l.topk_ids_s, b), nullptr,
                      ctx->at<int>(l.tok) + b * ctx->Mver, ctx->meta_v(b), st);
    }
  }
  amph_status rc = AMPH_OK;
  for (int b = 0; b < B && rc == AMPH_OK; ++b) {
    if (out_ids) rc = copy_out(ctx, out_ids + (size_t)b * K * kTopkStride, ctx->grp<int>(l.topk_ids, l.topk_ids_s, b), sizeof(int) * K * kTopkStride);
    if (rc == AMPH_OK && out_vals)
      rc = copy_out(ctx, out_vals + (size_t)b * K * kTopkStride, ctx->grp<float>(l.topk_vals, l.topk_vals_s, b), sizeof(float) * K * kTopkStride);
  }
  return rc;
}

// T > 0: replaces the greedy choices of every sequence's tree rows by draws from softmax(logits / T) (Section 2).
void sample_tree_choices(amph_ctx* ctx) {
  const Layout& l = ctx->lay;
  const amph_config& c = ctx->cfg;
  const unsigned long long seed = ((unsigned long long)c.seed_hi << 32) | c.seed_lo;
  for (int b = 0; b < ctx->B; ++b) {
    ProfScope p(ctx, AMPH_PROF_SELECT);
    launch_sample_rows(ctx->at<float>(l.logits), c.vocab, b * ctx->Mver, ctx->tree_host.n_nodes, ctx->at<TreeDev>(l.tree),
                       ctx->at<int>(l.tok) + b * ctx->Mver, ctx->state(b), b, 0, c.temperature, seed, ctx->at<int>(l.amax),
                       ctx->at<float>(l.uniforms) + b * ctx->Mver, ctx->stream);
  }
}

// tree_tokens / out_argmax: [B][n_nodes]
amph_status do_verify(amph_ctx* ctx, const int32_t* tree_tokens, int32_t* out_argmax) {
  const Layout& l = ctx->lay;
  cudaStream_t st = ctx->stream;
  const int N = ctx->tree_host.n_nodes, B = ctx->B;
  Pass ps;
  ps.G = B;
  ps.rpg = ctx->Mver;
  for (int b = 0; b < B; ++b) {
    ps.meta[b] = ctx->meta_v(b);
    ps.rope[b] = ctx->grp<float2>(l.rope_v, l.rope_s_, b);
    ps.seq[b] = b;
    ps.keys[b] = ctx->ctx_hi[b] + N;
    if (tree_tokens) {
      int* ov = ctx->at<int>(l.override_tok) + b * ctx->Mver;
      amph_status rc = cuda_check(ctx, cudaMemcpyAsync(ov, tree_tokens + (size_t)b * N, sizeof(int) * N, cudaMemcpyDefault, st), "copy of tree tokens");
      if (rc != AMPH_OK) return rc;
      ProfScope p(ctx, AMPH_PROF_OTHER);
      launch_tree_build(ctx->at<TreeDev>(l.tree), ctx->state(b), nullptr, ov, ctx->at<int>(l.tok) + b * ctx->Mver, ctx->meta_v(b), st);
    }
  }
  target_forward(ctx, ps);
  target_head(ctx, ps.rows());
  if (ctx->cfg.temperature > 0.f) sample_tree_choices(ctx);
  amph_status rc = AMPH_OK;
  for (int b = 0; b < B && rc == AMPH_OK && out_argmax; ++b)
    rc = copy_out(ctx, out_argmax + (size_t)b * N, ctx->at<int>(l.amax) + b * ctx->Mver, sizeof(int) * N);
  return rc;
}

void join_side(amph_ctx* ctx) {
  if (!ctx->side || !ctx->side_dirty) return;
  cudaEventRecord(ctx->join_ev, ctx->side);
  cudaStreamWaitEvent(ctx->stream, ctx->join_ev, 0);
  ctx->side_dirty = false;
  ctx->fork_used = 0;
}

// out_tokens, out_path: [B][K+1]; out_n, out_next_root: [B]
amph_status do_accept(amph_ctx* ctx, int32_t* out_tokens, int32_t* out_n, int32_t* out_path, int32_t* out_next_root) {
  const amph_config& c = ctx->cfg;
  const Layout& l = ctx->lay;
  cudaStream_t st = ctx->stream;
  join_side(ctx);
  amph_status rc = AMPH_OK;
  for (int b = 0; b < ctx->B && rc == AMPH_OK; ++b) {
    DevState* ds = ctx->state(b);
    { ProfScope p(ctx, AMPH_PROF_ACCEPT);
    launch_accept(ctx->at<TreeDev>(l.tree), ds, ctx->at<int>(l.tok) + b * ctx->Mver, ctx->at<int>(l.amax) + b * ctx->Mver, st);
    }
    { ProfScope p(ctx, AMPH_PROF_ACCEPT);
    launch_compact(ds, ctx->grp<KvView>(l.kv_tab, l.kv_tab_s, b), c.n_layers, ctx->dtype, c.n_heads, c.head_dim, c.max_ctx,
                   ctx->at<float>(l.hidden) + (size_t)b * ctx->Mver * c.d_model,
                   ctx->at<float>(l.pend_h) + (size_t)b * kSmallRows * c.d_model, c.d_model, st);
    }
    if (out_tokens) rc = copy_out(ctx, out_tokens + b * (c.K + 1), ds->out_tok, sizeof(int) * (c.K + 1));
    if (rc == AMPH_OK && out_n) rc = copy_out(ctx, out_n + b, &ds->L, sizeof(int));
    if (rc == AMPH_OK && out_path) rc = copy_out(ctx, out_path + b * (c.K + 1), ds->path, sizeof(int) * (c.K + 1));
    if (rc == AMPH_OK && out_next_root) rc = copy_out(ctx, out_next_root + b, &ds->next_root, sizeof(int));
  }
  return rc;
}

int attn_splits_for(const amph_ctx* ctx, int ctx_hi, int rows) {
  if (ctx->attn_tc) {         // split count and ring depth both shape the captured launch
    const int sp = attn_tc_splits(ctx->attn_tc, ctx_hi, ctx->cfg.n_heads, rows, ctx->lay.attn_splits);
    return sp * 8 + attn_tc_stages(ctx_hi, sp, ctx->cfg.head_dim);
  }
  int s = (ctx_hi + 127) / 128;
  if (s > ctx->lay.attn_splits) s = ctx->lay.attn_splits;
  return s < 1 ? 1 : s;
}

amph_status check_capacity(amph_ctx* ctx) {
  const int N = ctx->tree_host.n_nodes;
  if (ctx->max_ctx_hi() + N > ctx->cfg.max_ctx) {
    amph_status rc = refresh_ctx_hi(ctx);
    if (rc != AMPH_OK) return rc;
    if (ctx->max_ctx_hi() + N > ctx->cfg.max_ctx)
      return fail(ctx, AMPH_ERR_CAPACITY, "ctx_len %d + %d tree nodes exceeds max_ctx %d", ctx->max_ctx_hi(), N, ctx->cfg.max_ctx);
  }
  return AMPH_OK;
}

// The captured schedule depends on the host's bounds only through the attention launches of every sequence.
long long graph_key_of(const amph_ctx* ctx) {
  long long key = 0;
  for (int b = 0; b < ctx->B; ++b)
    key = key * 4099 + attn_splits_for(ctx, ctx->ctx_hi[b], ctx->rows_small) * 128 +
          attn_splits_for(ctx, ctx->ctx_hi[b] + ctx->tree_host.n_nodes, ctx->Mver);
  return key;
}

}  // namespace

// =============================================================================================
// C ABI
// =============================================================================================
extern "C" {

amph_status amph_workspace_bytes(const amph_config* cfg, const amph_tree* tree, size_t* kv_bytes, size_t* ws_bytes) {
  amph_status rc = validate(cfg, tree, nullptr);
  if (rc != AMPH_OK) return rc;
  if (!kv_bytes || !ws_bytes) return fail(nullptr, AMPH_ERR_INVALID_ARG, "output pointers must not be NULL");
  Layout l;
  int Mcap;
  make_layout(*cfg, tree->n_nodes, &l, &Mcap, kv_bytes);
  *ws_bytes = l.total;
  return AMPH_OK;
}

amph_status amph_init(const amph_config* cfg, const amph_tree* tree, void* kv_dev, size_t kv_bytes, void* ws_dev,
                      size_t ws_bytes, void* stream, amph_ctx** out) {
  if (!out) return fail(nullptr, AMPH_ERR_INVALID_ARG, "out must not be NULL");
  *out = nullptr;
  TreeDev td;
  amph_status rc = validate(cfg, tree, &td);
  if (rc != AMPH_OK) return rc;
  if (!kv_dev || !ws_dev) return fail(nullptr, AMPH_ERR_INVALID_ARG, "kv_dev and ws_dev must not be NULL");
  if (((uintptr_t)kv_dev | (uintptr_t)ws_dev) & 255) return fail(nullptr, AMPH_ERR_WORKSPACE, "regions must be 256-byte aligned");
  Layout l;
  int Mcap, Mver, Rcap, small_cap;
  size_t need_kv;
  make_layout(*cfg, tree->n_nodes, &l, &Mcap, &need_kv, &Mver, &Rcap, &small_cap);
  if (kv_bytes < need_kv) return fail(nullptr, AMPH_ERR_WORKSPACE, "kv region: %zu bytes given, %zu needed", kv_bytes, need_kv);
  if (ws_bytes < l.total) return fail(nullptr, AMPH_ERR_WORKSPACE, "workspace: %zu bytes given, %zu needed", ws_bytes, l.total);
  int dev_count = 0;
  if (cudaGetDeviceCount(&dev_count) != cudaSuccess || dev_count < 1) {
    cudaGetLastError();
    return fail(nullptr, AMPH_ERR_CUDA, "no CUDA device: this library has no CPU path");
  }
  amph_ctx* ctx = new amph_ctx();
  ctx->cfg = *cfg;
  ctx->tree_host = td;
  ctx->stream = (cudaStream_t)stream;
  ctx->dtype = cfg->weight_dtype;
  ctx->esz = cfg->weight_dtype == AMPH_DTYPE_F32 ? 4 : 2;
  ctx->B = cfg->max_batch;
  ctx->Mcap = Mcap;
  ctx->Rcap = Rcap;
  ctx->Mver = Mver;
  ctx->rows_small = kSmallRows;
  ctx->small_cap = small_cap;
  ctx->lay = l;
  ctx->ws = (char*)ws_dev;
  ctx->kv = (char*)kv_dev;
  ctx->resolved = false;
  ctx->phase = PH_CREATED;
  ctx->tc = nullptr;
  { int dv = 0; cudaGetDevice(&dv); cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, dv); }
  if (ctx->stream != nullptr && cfg->weight_dtype == AMPH_DTYPE_BF16 && !(cfg->flags & (AMPH_FLAG_NO_SIDE_PREFETCH | AMPH_FLAG_NO_TENSOR_CORE))) {
    if (cudaStreamCreateWithFlags(&ctx->side, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->join_ev, cudaEventDisableTiming) != cudaSuccess) {
      cudaGetLastError();
      ctx->side = nullptr;                 // no helper stream: the step runs without the prefetch
    }
  }
  const size_t half_layer = (size_t)cfg->n_heads * cfg->max_ctx * cfg->head_dim * ctx->esz;
  char* p = ctx->kv;
  for (int b = 0; b < ctx->B; ++b) {                   // sequence by sequence: target layers, then the adaptation layers
    ctx->kv_target[b].resize(cfg->n_layers);
    for (int i = 0; i < cfg->n_layers; ++i) { ctx->kv_target[b][i].k = p; ctx->kv_target[b][i].v = p + half_layer; p += 2 * half_layer; }
    for (int s = 0; s < cfg->n_sal; ++s) { ctx->kv_sal[b][s].k = p; ctx->kv_sal[b][s].v = p + half_layer; p += 2 * half_layer; }
  }
  cudaStream_t st = ctx->stream;
  cudaError_t e = cudaMemsetAsync(ctx->ws, 0, l.total, st);
  // The attention kernels fetch whole key tiles; slots past the live range are masked (probability 0), which only
  // cancels finite values, so the caches must never hold the NaN patterns of uninitialised memory.
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->kv, 0, need_kv, st);
  std::vector<double> inv(cfg->head_dim / 2);
  for (int i = 0; i < cfg->head_dim / 2; ++i) inv[i] = pow((double)cfg->rope_theta, -2.0 * i / cfg->head_dim);
  if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->ws + l.tree, &ctx->tree_host, sizeof(TreeDev), cudaMemcpyHostToDevice, st);
  for (int b = 0; b < ctx->B && e == cudaSuccess; ++b)
    e = cudaMemcpyAsync(ctx->ws + l.kv_tab + l.kv_tab_s * b, ctx->kv_target[b].data(), sizeof(KvView) * cfg->n_layers, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->ws + l.inv_freq, inv.data(), sizeof(double) * inv.size(), cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) {
    rc = cuda_check(nullptr, e, "workspace set-up");
    delete ctx;
    return rc;
  }
  *out = ctx;
  return AMPH_OK;
}

amph_status amph_load_weights(amph_ctx* ctx, const amph_tensor* tensors, int32_t n) {
  if (!ctx) return fail(nullptr, AMPH_ERR_INVALID_ARG, "ctx must not be NULL");
  if (!tensors || n < 0) return fail(ctx, AMPH_ERR_INVALID_ARG, "tensors must not be NULL");
  for (int i = 0; i < n; ++i) {
    const amph_tensor& t = tensors[i];
    if (!t.name || !t.dev_ptr) return fail(ctx, AMPH_ERR_INVALID_ARG, "tensor %d: NULL name or pointer", i);
    if (t.dtype != ctx->cfg.weight_dtype) return fail(ctx, AMPH_ERR_SHAPE, "tensor '%s': dtype %d != weight_dtype", t.name, t.dtype);
    if (t.ndim != 1 && t.ndim != 2) return fail(ctx, AMPH_ERR_SHAPE, "tensor '%s': ndim must be 1 or 2", t.name);
    if ((uintptr_t)t.dev_ptr & 15) return fail(ctx, AMPH_ERR_INVALID_ARG, "tensor '%s' is not 16-byte aligned", t.name);
    TensorRec r;
    r.ptr = t.dev_ptr;
    r.ndim = t.ndim;
    r.shape[0] = t.shape[0];
    r.shape[1] = t.ndim == 2 ? t.shape[1] : 0;
    ctx->tensors[t.name] = r;
  }
  ctx->resolved = false;
  if (ctx->graph_exec) {                       // the captured schedule holds the old pointers
    cudaGraphExecDestroy(ctx->graph_exec);
    ctx->graph_exec = nullptr;
    ctx->graph_key = -1;
  }
  return AMPH_OK;
}

amph_status amph_prefill_seq(amph_ctx* ctx, int32_t seq, const int32_t* prompt_ids, int32_t n, int32_t* out_root) {
  if (!ctx) return fail(nullptr, AMPH_ERR_INVALID_ARG, "ctx must not be NULL");
  if (seq < 0 || seq >= ctx->B) return fail(ctx, AMPH_ERR_INVALID_ARG, "sequence %d is outside 0..%d", seq, ctx->B - 1);
  if (!prompt_ids || n < 1) return fail(ctx, AMPH_ERR_INVALID_ARG, "prompt must hold at least one token");
  if (ctx->phase == PH_DRAFTED || ctx->phase == PH_VERIFIED) return fail(ctx, AMPH_ERR_STATE, "amph_prefill while a draft is in flight");
  const amph_config& c = ctx->cfg;
  for (int i = 0; i < n; ++i)
    if (prompt_ids[i] < 0 || prompt_ids[i] >= c.vocab) return fail(ctx, AMPH_ERR_INVALID_ARG, "prompt_ids[%d] = %d is outside the vocabulary", i, prompt_ids[i]);
  if (n + ctx->tree_host.n_nodes > c.max_ctx) return fail(ctx, AMPH_ERR_CAPACITY, "prompt of %d tokens + tree exceeds max_ctx %d", n, c.max_ctx);
  amph_status rc = resolve(ctx);
  if (rc != AMPH_OK) return rc;
  if (!ctx->tc && c.weight_dtype == AMPH_DTYPE_BF16 && !(c.flags & AMPH_FLAG_NO_TENSOR_CORE)) {
    void* xb[XB_COUNT];
    for (int i = 0; i < XB_COUNT; ++i) xb[i] = xbuf_ptr(ctx, i);
    const int sc = ctx->small_cap;
    const int xrows[XB_COUNT] = {ctx->Rcap, ctx->Rcap, ctx->Rcap, ctx->Rcap, sc, sc, sc, sc};
    const int xcols[XB_COUNT] = {c.d_model, c.d_model, c.d_ffn, ((c.flags & AMPH_FLAG_NO_SAMPLED_TOKEN) ? 1 : 2) * c.d_model,
                                 c.d_model, c.d_model, c.d_model,
                                 c.lm_rank > 0 ? c.lm_rank : 8};
    ctx->tc = tc_gemm_create(xb, xrows, xcols, XB_COUNT, &ctx->state(0)->err);
  }
  if (!ctx->attn_tc && c.kv_dtype == AMPH_DTYPE_BF16 && !(c.flags & AMPH_FLAG_MMA_SYNC_ATTENTION))
    ctx->attn_tc = attn_tc_create();
  const Layout& l = ctx->lay;
  cudaStream_t st = ctx->stream;
  const int M = kPrefillRows;
  // A pass carries up to kPrefillGroups chunks of 128 prompt tokens as row groups that share every weight tile: the
  // rows of chunk g see the committed slots plus the chunks before them, whose keys and values the same pass has
  // written by the time attention runs, and a causal mask inside the chunk.
  const int Gmax = (c.flags & AMPH_FLAG_CHUNKED_PREFILL) ? 1 : kPrefillGroups;
  cudaMemsetAsync(ctx->state(seq), 0, sizeof(DevState), st);
  ctx->prefilled[seq] = false;
  for (int start = 0; start < n; start += Gmax * M) {
    const int cnt = n - start < Gmax * M ? n - start : Gmax * M;
    const bool last = start + cnt == n;
    const int G = (cnt + M - 1) / M;
    const int rpg = G == 1 ? round_up(cnt, 16) : M;          // rows the kernels carry per group
    rc = cuda_check(ctx, cudaMemcpyAsync(ctx->at<int>(l.tok), prompt_ids + start, sizeof(int) * cnt, cudaMemcpyHostToDevice, st), "prompt upload");
    if (rc != AMPH_OK) return rc;
    Pass ps;
    ps.G = G;
    ps.rpg = rpg;
    for (int g = 0; g < G; ++g) {
      const int nr = cnt - g * M < M ? cnt - g * M : M;
      launch_meta_chain(ctx->meta_v(g), start + g * M, nr, st);
      ps.meta[g] = ctx->meta_v(g);
      ps.rope[g] = ctx->grp<float2>(l.rope_v, l.rope_s_, g);
      ps.seq[g] = seq;
      ps.keys[g] = start + g * M + nr;
    }
    target_forward(ctx, ps);
    if (last) target_head(ctx, ps.rows());
    const int nrs = last ? cnt - 1 : cnt;         // the last prompt row stays pending for the first draft
    if (nrs > 0 && c.n_sal > 0) {
      rc = cuda_check(ctx, cudaMemcpyAsync(ctx->at<int>(l.next_tok), prompt_ids + start + 1, sizeof(int) * nrs, cudaMemcpyHostToDevice, st), "prompt upload");
      if (rc != AMPH_OK) return rc;
      Pass pss;
      pss.G = (nrs + M - 1) / M;
      pss.rpg = rpg;
      const int* next_tok[kMaxSeq];
      for (int g = 0; g < pss.G; ++g) {
        const int nr = nrs - g * M < M ? nrs - g * M : M;
        launch_meta_chain(ctx->meta_s(g), start + g * M, nr, st);
        pss.meta[g] = ctx->meta_s(g);
        pss.rope[g] = ctx->grp<float2>(l.rope_s, l.rope_s_, g);
        pss.seq[g] = seq;
        pss.keys[g] = start + g * M + nr;
        next_tok[g] = ctx->at<int>(l.next_tok) + g * rpg;
      }
      run_sals(ctx, ctx->at<float>(l.hidden), next_tok, pss);
    }
    if (last && c.temperature > 0.f)        // the token after the prompt is drawn, not the arg-max (stream 1 of the generator, step 0)
      launch_sample_rows(ctx->at<float>(l.logits), c.vocab, cnt - 1, 1, nullptr, nullptr, ctx->state(seq), seq, 1, c.temperature,
                         ((unsigned long long)c.seed_hi << 32) | c.seed_lo, ctx->at<int>(l.amax), nullptr, st);
    if (last)
      launch_prefill_tail(ctx->state(seq), ctx->at<int>(l.amax), cnt - 1, ctx->at<float>(l.hidden),
                          ctx->at<float>(l.pend_h) + (size_t)seq * kSmallRows * c.d_model, c.d_model, n, st);
  }
  join_side(ctx);
  rc = finish(ctx, "prefill");
  if (rc != AMPH_OK) return rc;
  ctx->prefilled[seq] = true;
  rc = refresh_ctx_hi(ctx);
  if (rc != AMPH_OK) return rc;
  if (out_root) {
    DevState s;
    cudaMemcpy(&s, ctx->state(seq), sizeof s, cudaMemcpyDeviceToHost);
    *out_root = s.root;
  }
  bool all = true;
  for (int b = 0; b < ctx->B; ++b) all = all && ctx->prefilled[b];
  ctx->phase = all ? PH_READY : PH_CREATED;
  return AMPH_OK;
}

amph_status amph_prefill(amph_ctx* ctx, const int32_t* prompt_ids, int32_t n, int32_t* out_root) {
  return amph_prefill_seq(ctx, 0, prompt_ids, n, out_root);
}

amph_status amph_draft(amph_ctx* ctx, int32_t* out_topk_ids, float* out_topk_vals) {
  if (!ctx) return fail(nullptr, AMPH_ERR_INVALID_ARG, "ctx must not be NULL");
  if (ctx->phase != PH_READY) return fail(ctx, AMPH_ERR_STATE, "amph_draft needs a prefilled sequence and no draft in flight");
  amph_status rc = check_capacity(ctx);
  if (rc != AMPH_OK) return rc;
  rc = do_draft(ctx, out_topk_ids, out_topk_vals);
  if (rc == AMPH_OK) rc = finish(ctx, "draft");
  if (rc == AMPH_OK) ctx->phase = PH_DRAFTED;
  return rc;
}

amph_status amph_verify_tree(amph_ctx* ctx, const int32_t* tree_tokens, int32_t* out_argmax) {
  if (!ctx) return fail(nullptr, AMPH_ERR_INVALID_ARG, "ctx must not be NULL");
  if (ctx->phase != PH_DRAFTED) return fail(ctx, AMPH_ERR_STATE, "amph_verify_tree must follow amph_draft");
  amph_status rc = do_verify(ctx, tree_tokens, out_argmax);
  if (rc == AMPH_OK) rc = finish(ctx, "verify");
  if (rc == AMPH_OK) ctx->phase = PH_VERIFIED;
  return rc;
}

amph_status amph_accept(amph_ctx* ctx, int32_t* out_tokens, int32_t* out_n, int32_t* out_path, int32_t* out_next_root) {
  if (!ctx) return fail(nullptr, AMPH_ERR_INVALID_ARG, "ctx must not be NULL");
  if (ctx->phase != PH_VERIFIED) return fail(ctx, AMPH_ERR_STATE, "amph_accept must follow amph_verify_tree");
  amph_status rc = do_accept(ctx, out_tokens, out_n, out_path, out_next_root);
  if (rc == AMPH_OK) rc = finish(ctx, "accept");
  if (rc == AMPH_OK) {
    ctx->phase = PH_READY;
    for (int b = 0; b < ctx->B; ++b) ctx->ctx_hi[b] += ctx->cfg.K + 1;
  }
  return rc;
}

amph_status amph_step(amph_ctx* ctx, int32_t* out_tokens, int32_t* out_n) {
  if (!ctx) return fail(nullptr, AMPH_ERR_INVALID_ARG, "ctx must not be NULL");
  if (ctx->phase != PH_READY) return fail(ctx, AMPH_ERR_STATE, "amph_step needs a prefilled sequence and no draft in flight");
  amph_status rc = check_capacity(ctx);
  if (rc != AMPH_OK) return rc;
  const amph_config& c = ctx->cfg;
  const bool use_graph = !ctx->graph_off && !ctx->prof_on && !(c.flags & AMPH_FLAG_NO_GRAPH) && ctx->stream != nullptr;
  if (use_graph) {
    // The kernels read every length from device state; only the attention grids depend on the host's
    // bound of the context length, so the captured schedule is reused until that grid size changes.
    const long long key = graph_key_of(ctx);
    if (!ctx->graph_exec || key != ctx->graph_key) {
      if (ctx->graph_exec) { cudaGraphExecDestroy(ctx->graph_exec); ctx->graph_exec = nullptr; }
      cudaGraph_t graph = nullptr;
      if (cudaStreamBeginCapture(ctx->stream, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
        rc = do_draft(ctx, nullptr, nullptr);
        if (rc == AMPH_OK) rc = do_verify(ctx, nullptr, nullptr);
        if (rc == AMPH_OK) rc = do_accept(ctx, nullptr, nullptr, nullptr, nullptr);
        const cudaError_t e = cudaStreamEndCapture(ctx->stream, &graph);
        if (rc == AMPH_OK && e == cudaSuccess && graph &&
            cudaGraphInstantiate(&ctx->graph_exec, graph, 0) == cudaSuccess) {
          ctx->graph_key = key;
        } else {
          ctx->graph_exec = nullptr;
          ctx->graph_off = true;
        }
        if (graph) cudaGraphDestroy(graph);
      } else {
        ctx->graph_off = true;
      }
      cudaGetLastError();
    }
  }
  if (use_graph && ctx->graph_exec) {
    rc = cuda_check(ctx, cudaGraphLaunch(ctx->graph_exec, ctx->stream), "graph launch");
  } else {
    rc = do_draft(ctx, nullptr, nullptr);
    if (rc == AMPH_OK) rc = do_verify(ctx, nullptr, nullptr);
    if (rc == AMPH_OK) rc = do_accept(ctx, nullptr, nullptr, nullptr, nullptr);
  }
  for (int b = 0; b < ctx->B && rc == AMPH_OK; ++b) {
    DevState* ds = ctx->state(b);
    if (out_tokens) rc = copy_out(ctx, out_tokens + b * (c.K + 1), ds->out_tok, sizeof(int) * (c.K + 1));
    if (rc == AMPH_OK && out_n) rc = copy_out(ctx, out_n + b, &ds->L, sizeof(int));
  }
  if (rc == AMPH_OK) rc = finish(ctx, "step");
  if (rc == AMPH_OK)
    for (int b = 0; b < ctx->B; ++b) ctx->ctx_hi[b] += c.K + 1;
  return rc;
}

amph_status amph_get_tensor(amph_ctx* ctx, const char* name, void* dst, size_t bytes) {
  if (!ctx) return fail(nullptr, AMPH_ERR_INVALID_ARG, "ctx must not be NULL");
  if (!name || !dst) return fail(ctx, AMPH_ERR_INVALID_ARG, "name and dst must not be NULL");
  const amph_config& c = ctx->cfg;
  const Layout& l = ctx->lay;
  // optional suffixes: "#b" selects sequence b (default 0), "@row0" the first cache slot of a cache export
  std::string nm(name);
  int row0 = 0, seq = 0;
  size_t at = nm.find('@');
  if (at != std::string::npos) { row0 = atoi(nm.c_str() + at + 1); nm = nm.substr(0, at); }
  at = nm.find('#');
  if (at != std::string::npos) { seq = atoi(nm.c_str() + at + 1); nm = nm.substr(0, at); }
  if (seq < 0 || seq >= ctx->B) return fail(ctx, AMPH_ERR_INVALID_ARG, "'%s': sequence outside 0..%d", name, ctx->B - 1);
  const size_t d = c.d_model, V = c.vocab, N = ctx->tree_host.n_nodes, K = c.K, R = ctx->Rcap, Mv = ctx->Mver;
  // row buffers: sequence b's rows of a verification pass start at row b * Mver (after a prefill: the rows of its last pass)
  struct { const char* n; size_t off, size; } plain[] = {
      {"hidden", l.hidden + 4 * seq * Mv * d, 4 * (R - seq * Mv) * d},
      {"logits", l.logits + 4 * seq * Mv * V, 4 * (R - seq * Mv) * V},
      {"d_logits", l.d_logits + l.d_logits_s * seq, 4 * K * V},
      {"hp", l.hp + 4 * seq * kMaxK * d, 4 * K * d},
      {"attn_o", l.attn_o + 4 * seq * K * d, 4 * K * d},
      {"sal_h", l.last + l.last_s * seq, 4 * 2 * d},
      {"tree_tokens", l.tok + 4 * seq * Mv, 4 * N},
      {"argmax", l.amax + 4 * seq * Mv, 4 * N},
      {"uniforms", l.uniforms + 4 * seq * Mv, 4 * N},
  };
  for (auto& p : plain) {
    if (nm == p.n) {
      if (bytes > p.size) return fail(ctx, AMPH_ERR_INVALID_ARG, "'%s' holds %zu bytes, %zu requested", name, p.size, bytes);
      return copy_out(ctx, dst, ctx->ws + p.off, bytes);
    }
  }
  // cache exports: "kv.k.{i}", "kv.v.{i}", "sal{s}.k", "sal{s}.v"
  KvView kv = {nullptr, nullptr};
  int which = -1, idx = -1;
  char kvc = 0;
  if (sscanf(nm.c_str(), "kv.%c.%d", &kvc, &idx) == 2 && idx >= 0 && idx < c.n_layers) kv = ctx->kv_target[seq][idx];
  else if (sscanf(nm.c_str(), "sal%d.%c", &idx, &kvc) == 2 && idx >= 1 && idx <= c.n_sal) kv = ctx->kv_sal[seq][idx - 1];
  if (kvc == 'k') which = 0;
  if (kvc == 'v') which = 1;
  if (!kv.k || which < 0) return fail(ctx, AMPH_ERR_INVALID_ARG, "unknown tensor '%s'", name);
  const size_t rows = bytes / (4 * d);
  if (rows * 4 * d != bytes || row0 < 0 || row0 + (int)rows > c.max_ctx)
    return fail(ctx, AMPH_ERR_INVALID_ARG, "'%s': bytes must be a whole number of rows inside the cache", name);
  if (rows * d > l.partial_floats) return fail(ctx, AMPH_ERR_INVALID_ARG, "'%s': at most %zu rows per call", name, l.partial_floats / d);
  float* stage = ctx->at<float>(l.partial);
  launch_kv_export(kv, which, ctx->dtype, row0, (int)rows, c.n_heads, c.head_dim, c.max_ctx, stage, ctx->stream);
  amph_status rc = finish(ctx, "cache export");
  if (rc != AMPH_OK) return rc;
  return copy_out(ctx, dst, stage, bytes);
}

amph_status amph_set_tensor(amph_ctx* ctx, const char* name, const void* src, size_t bytes) {
  if (!ctx) return fail(nullptr, AMPH_ERR_INVALID_ARG, "ctx must not be NULL");
  if (!name || !src) return fail(ctx, AMPH_ERR_INVALID_ARG, "name and src must not be NULL");
  std::string nm(name);
  int seq = 0;
  const size_t at = nm.find('#');
  if (at != std::string::npos) { seq = atoi(nm.c_str() + at + 1); nm = nm.substr(0, at); }
  if (seq < 0 || seq >= ctx->B) return fail(ctx, AMPH_ERR_INVALID_ARG, "'%s': sequence outside 0..%d", name, ctx->B - 1);
  if (nm == "root") {                            // right after prefill: replaces the greedy root token
    if (ctx->phase != PH_READY || bytes != sizeof(int)) return fail(ctx, AMPH_ERR_STATE, "'root' takes one int32 right after amph_prefill");
    DevState* ds = ctx->state(seq);
    amph_status rc = cuda_check(ctx, cudaMemcpyAsync(&ds->root, src, sizeof(int), cudaMemcpyDefault, ctx->stream), "set_tensor");
    if (rc == AMPH_OK) rc = cuda_check(ctx, cudaMemcpyAsync(&ds->pend_tok[0], src, sizeof(int), cudaMemcpyDefault, ctx->stream), "set_tensor");
    return rc;
  }
  if (ctx->phase != PH_VERIFIED) return fail(ctx, AMPH_ERR_STATE, "amph_set_tensor must follow amph_verify_tree");
  if (nm == "logits") {                          // T > 0: replace the verified rows' logits and draw the choices again
    const amph_config& c = ctx->cfg;
    const size_t N = ctx->tree_host.n_nodes;
    if (!(c.temperature > 0.f)) return fail(ctx, AMPH_ERR_STATE, "'logits' can be set with temperature > 0 only");
    if (bytes != sizeof(float) * N * c.vocab) return fail(ctx, AMPH_ERR_INVALID_ARG, "'logits' takes exactly n_nodes * vocab floats");
    amph_status rc = cuda_check(ctx, cudaMemcpyAsync(ctx->at<float>(ctx->lay.logits) + (size_t)seq * ctx->Mver * c.vocab, src, bytes,
                                                     cudaMemcpyDefault, ctx->stream), "set_tensor");
    if (rc != AMPH_OK) return rc;
    sample_tree_choices(ctx);
    return finish(ctx, "sampling");
  }
  size_t off;
  if (nm == "tree_tokens") off = ctx->lay.tok;
  else if (nm == "argmax") off = ctx->lay.amax;
  else return fail(ctx, AMPH_ERR_INVALID_ARG, "'%s' cannot be set", name);
  if (bytes != sizeof(int) * (size_t)ctx->tree_host.n_nodes)
    return fail(ctx, AMPH_ERR_INVALID_ARG, "'%s' takes exactly n_nodes int32 values", name);
  return cuda_check(ctx, cudaMemcpyAsync(ctx->ws + off + sizeof(int) * seq * ctx->Mver, src, bytes, cudaMemcpyDefault, ctx->stream), "set_tensor");
}

amph_status amph_get_state_seq(amph_ctx* ctx, int32_t seq, int32_t* ctx_len, int32_t* root, int32_t* n_pending) {
  if (!ctx) return fail(nullptr, AMPH_ERR_INVALID_ARG, "ctx must not be NULL");
  if (seq < 0 || seq >= ctx->B) return fail(ctx, AMPH_ERR_INVALID_ARG, "sequence %d is outside 0..%d", seq, ctx->B - 1);
  DevState s;
  cudaError_t e = cudaMemcpyAsync(&s, ctx->state(seq), sizeof s, cudaMemcpyDeviceToHost, ctx->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
  if (e != cudaSuccess) return cuda_check(ctx, e, "state read-back");
  if (ctx->prefilled[seq]) ctx->ctx_hi[seq] = s.C;
  if (ctx_len) *ctx_len = s.C;
  if (root) *root = s.root;
  if (n_pending) *n_pending = s.n_pending;
  int err = s.err;
  if (seq != 0 && !err) {                        // device-side waits report through sequence 0's state word
    DevState s0;
    if (cudaMemcpy(&s0, ctx->state(0), sizeof s0, cudaMemcpyDeviceToHost) == cudaSuccess) err = s0.err;
  }
  if (err) return fail(ctx, err, "a device-side wait gave up (code %d)", err);
  return AMPH_OK;
}

amph_status amph_get_state(amph_ctx* ctx, int32_t* ctx_len, int32_t* root, int32_t* n_pending) {
  return amph_get_state_seq(ctx, 0, ctx_len, root, n_pending);
}

amph_status amph_profile_begin(amph_ctx* ctx) {
  if (!ctx) return fail(nullptr, AMPH_ERR_INVALID_ARG, "ctx must not be NULL");
  if (ctx->prof_ev.empty()) {
    ctx->prof_ev.resize(2 * 16384);
    for (auto& e : ctx->prof_ev)
      if (cudaEventCreate(&e) != cudaSuccess) {
        ctx->prof_ev.clear();
        return cuda_check(ctx, cudaGetLastError(), "event creation");
      }
  }
  ctx->prof_cat.assign(ctx->prof_ev.size() / 2, 0);
  ctx->prof_used = 0;
  ctx->prof_bytes = 0;
  ctx->prof_on = true;
  return AMPH_OK;
}

amph_status amph_profile_end(amph_ctx* ctx, double* proj_ms, int64_t* proj_launches, int64_t* proj_weight_bytes) {
  if (!ctx) return fail(nullptr, AMPH_ERR_INVALID_ARG, "ctx must not be NULL");
  if (!ctx->prof_on) return fail(ctx, AMPH_ERR_STATE, "amph_profile_end without amph_profile_begin");
  ctx->prof_on = false;
  amph_status rc = cuda_check(ctx, cudaStreamSynchronize(ctx->stream), "profile synchronise");
  if (rc != AMPH_OK) return rc;
  for (int c = 0; c < AMPH_PROF_CATEGORIES; ++c) { ctx->prof_cat_ms[c] = 0.0; ctx->prof_cat_n[c] = 0; }
  for (size_t i = 0; i + 1 < ctx->prof_used; i += 2) {
    float t = 0.f;
    const int cat = ctx->prof_cat[i / 2];
    if (cudaEventElapsedTime(&t, ctx->prof_ev[i], ctx->prof_ev[i + 1]) == cudaSuccess) {
      ctx->prof_cat_ms[cat] += t;
      ctx->prof_cat_n[cat] += 1;
    }
  }
  if (proj_ms) *proj_ms = ctx->prof_cat_ms[AMPH_PROF_PROJECTION];
  if (proj_launches) *proj_launches = ctx->prof_cat_n[AMPH_PROF_PROJECTION];
  if (proj_weight_bytes) *proj_weight_bytes = ctx->prof_bytes;
  return AMPH_OK;
}

static amph_status project_standalone(const void* x_dev, int32_t x_rows_cap, const void* const* w, int32_t n_seg, int32_t out,
                                      int32_t in, int32_t rows, int32_t dtype, int32_t use_tensor_core, float* y_dev, void* ws_dev,
                                      size_t ws_bytes, void* stream, unsigned long long limit_ns, unsigned extra_tx) {
  if (!x_dev || !w || !y_dev || !ws_dev) return fail(nullptr, AMPH_ERR_INVALID_ARG, "NULL pointer");
  if (n_seg < 1 || n_seg > kMaxK || out < 1 || in < 8 || rows < 1 || rows > 4 * kMaxRows || x_rows_cap < rows)
    return fail(nullptr, AMPH_ERR_SHAPE, "bad projection shape");
  if (dtype != AMPH_DTYPE_F32 && dtype != AMPH_DTYPE_BF16) return fail(nullptr, AMPH_ERR_SHAPE, "unknown dtype");
  if (in % (dtype == AMPH_DTYPE_F32 ? 4 : 8)) return fail(nullptr, AMPH_ERR_SHAPE, "in must be a multiple of 16 bytes");
  const size_t ld = (size_t)n_seg * out;
  const size_t need = 256 + (size_t)16 * 128 * ld * 4;
  if (ws_bytes < need || ((uintptr_t)ws_dev & 255)) return fail(nullptr, AMPH_ERR_WORKSPACE, "scratch: %zu bytes needed, 256-byte aligned", need);
  cudaStream_t st = (cudaStream_t)stream;
  int* err = (int*)ws_dev;
  float* P = (float*)((char*)ws_dev + 256);
  const size_t p_floats = (ws_bytes - 256) / 4;
  cudaMemsetAsync(err, 0, sizeof(int), st);
  PartialView pv;
  pv.p = P;
  pv.ld = (int)ld;
  if (use_tensor_core) {
    if (dtype != AMPH_DTYPE_BF16) return fail(nullptr, AMPH_ERR_SHAPE, "the tensor-core kernel takes bf16 only");
    void* xb[1] = {const_cast<void*>(x_dev)};
    const int xr[1] = {x_rows_cap}, xc[1] = {in};
    TcGemm* g = tc_gemm_create(xb, xr, xc, 1, err);
    if (!g) return fail(nullptr, AMPH_ERR_CUDA, "tensor-map encoder unavailable or not an sm_100 device");
    if (limit_ns) tc_gemm_set_selftest(g, limit_ns, extra_tx);
    int splits = 0;
    size_t stride = 0;
    const bool ok = tc_gemm_launch(g, 0, w, n_seg, out, in, rows, P, p_floats, &splits, &stride, st);
    tc_gemm_destroy(g);
    if (!ok) return fail(nullptr, AMPH_ERR_SHAPE, "shape not covered by the tensor-core kernel");
    pv.splits = splits;
    pv.split_stride = stride;
  } else {
    GemmSeg segs[kMaxK];
    for (int s = 0; s < n_seg; ++s) segs[s].w = w[s];
    launch_gemm_generic(x_dev, in, segs, n_seg, out, in, P, (int)ld, rows, dtype, st);
    pv.splits = 1;
    pv.split_stride = 0;
  }
  launch_reduce_partials(pv, y_dev, rows, (int)ld, st);
  return cuda_check(nullptr, cudaGetLastError(), "projection");
}

amph_status amph_project(const void* x_dev, int32_t x_rows_cap, const void* const* w, int32_t n_seg, int32_t out,
                         int32_t in, int32_t rows, int32_t dtype, int32_t use_tensor_core, float* y_dev, void* ws_dev,
                         size_t ws_bytes, void* stream) {
  return project_standalone(x_dev, x_rows_cap, w, n_seg, out, in, rows, dtype, use_tensor_core, y_dev, ws_dev, ws_bytes, stream,
                            0ull, 0u);
}

amph_status amph_selftest_wait_timeout(const void* x_dev, int32_t x_rows_cap, const void* const* w, int32_t n_seg,
                                       int32_t out, int32_t in, int32_t rows, float* y_dev, void* ws_dev, size_t ws_bytes,
                                       void* stream, int32_t limit_us) {
  if (limit_us < 1 || limit_us > 1000000) return fail(nullptr, AMPH_ERR_INVALID_ARG, "limit_us must be in 1..1000000");
  return project_standalone(x_dev, x_rows_cap, w, n_seg, out, in, rows, AMPH_DTYPE_BF16, 1, y_dev, ws_dev, ws_bytes, stream,
                            (unsigned long long)limit_us * 1000ull, 1024u);
}

amph_status amph_set_state(amph_ctx* ctx, int32_t ctx_len, int32_t root, int32_t n_pending, const float* pend_hidden,
                           const int32_t* pend_next) {
  if (!ctx) return fail(nullptr, AMPH_ERR_INVALID_ARG, "ctx must not be NULL");
  if (ctx->phase != PH_READY) return fail(ctx, AMPH_ERR_STATE, "amph_set_state needs a prefilled sequence and no draft in flight");
  const amph_config& c = ctx->cfg;
  if (!pend_hidden || !pend_next) return fail(ctx, AMPH_ERR_INVALID_ARG, "pend_hidden and pend_next must not be NULL");
  if (n_pending < 1 || n_pending > c.K + 1 || n_pending > ctx_len)
    return fail(ctx, AMPH_ERR_INVALID_ARG, "n_pending must be in 1..K+1 and at most ctx_len");
  if (root < 0 || root >= c.vocab) return fail(ctx, AMPH_ERR_INVALID_ARG, "root %d is outside the vocabulary", root);
  for (int j = 0; j < n_pending; ++j)
    if (pend_next[j] < 0 || pend_next[j] >= c.vocab) return fail(ctx, AMPH_ERR_INVALID_ARG, "pend_next[%d] is outside the vocabulary", j);
  if (ctx_len + ctx->tree_host.n_nodes > c.max_ctx)
    return fail(ctx, AMPH_ERR_CAPACITY, "ctx_len %d + %d tree nodes exceeds max_ctx %d", ctx_len, ctx->tree_host.n_nodes, c.max_ctx);
  DevState s;
  memset(&s, 0, sizeof s);
  s.C = ctx_len;
  s.root = root;
  s.n_pending = n_pending;
  for (int j = 0; j < n_pending; ++j) s.pend_tok[j] = pend_next[j];
  s.C_old = ctx_len;
  s.next_root = root;
  for (int j = 0; j < 16; ++j) { s.path[j] = -1; s.out_tok[j] = -1; }
  amph_status rc = cuda_check(ctx, cudaMemcpyAsync(ctx->state(0), &s, sizeof s, cudaMemcpyHostToDevice, ctx->stream), "set_state");
  if (rc == AMPH_OK) rc = cuda_check(ctx, cudaStreamSynchronize(ctx->stream), "set_state");       // s lives on this stack frame
  if (rc == AMPH_OK)
    rc = cuda_check(ctx, cudaMemcpyAsync(ctx->at<float>(ctx->lay.pend_h), pend_hidden, sizeof(float) * (size_t)n_pending * c.d_model,
                                         cudaMemcpyDefault, ctx->stream), "set_state");
  if (rc == AMPH_OK) ctx->ctx_hi[0] = ctx_len;
  return rc;
}

amph_status amph_profile_breakdown(amph_ctx* ctx, double* ms, int64_t* launches) {
  if (!ctx) return fail(nullptr, AMPH_ERR_INVALID_ARG, "ctx must not be NULL");
  for (int c = 0; c < AMPH_PROF_CATEGORIES; ++c) {
    if (ms) ms[c] = ctx->prof_cat_ms[c];
    if (launches) launches[c] = ctx->prof_cat_n[c];
  }
  return AMPH_OK;
}

amph_status amph_reset(amph_ctx* ctx) {
  if (!ctx) return fail(nullptr, AMPH_ERR_INVALID_ARG, "ctx must not be NULL");
  cudaError_t e = cudaMemsetAsync(ctx->ws + ctx->lay.state, 0, ctx->lay.state_s * kMaxSeq, ctx->stream);
  ctx->phase = PH_CREATED;
  for (int b = 0; b < kMaxSeq; ++b) { ctx->ctx_hi[b] = 0; ctx->prefilled[b] = false; }
  return cuda_check(ctx, e, "reset");
}

void amph_destroy(amph_ctx* ctx) {
  if (!ctx) return;
  if (ctx->tc) tc_gemm_destroy(ctx->tc);
  if (ctx->attn_tc) attn_tc_destroy(ctx->attn_tc);
  if (ctx->graph_exec) cudaGraphExecDestroy(ctx->graph_exec);
  for (auto& e : ctx->fork_ev) cudaEventDestroy(e);
  if (ctx->join_ev) cudaEventDestroy(ctx->join_ev);
  if (ctx->side) cudaStreamDestroy(ctx->side);
  for (auto& e : ctx->prof_ev) cudaEventDestroy(e);
  delete ctx;
}

const char* amph_last_error(const amph_ctx* ctx) { return ctx ? ctx->err.c_str() : g_last_error.c_str(); }

}  // extern "C"
