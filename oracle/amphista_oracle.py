"""CPU oracle for one Amphista speculative-decoding step (arXiv 2406.13170).

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, obviously-correct restatement
of what the decoding step computes, written from the paper, in plain PyTorch CPU
ops (float64 by default, float32 on request for the large shapes).  It shares no
code with the CUDA library and is imported only by the tests, the smoke check and
the benchmark's CPU-baseline leg; the product path never calls it.

Conventions
  * every linear map is y = W x with W stored [out_features, in_features];
  * a "row" is one token position; KV caches are Python lists indexed by slot;
  * the target's hidden state h_t handed to the draft module is the vector its
    lm_head consumes (after the final RMSNorm);
  * state.C committed tokens sit in cache slots 0..C-1; `root` is the token the
    target chose for position C (not yet in the cache);
  * `pending` holds, for every committed position the adaptation layers have not
    seen yet, (h_j, id of the token at position j+1, j).

Parity status of the parts
  * tree mask / positions / slots, acceptance, compaction, target forward: pinned
    by tests (per-path causal brute force, losslessness against greedy
    autoregressive decoding, Fig. 5's node / candidate counts, exhaustive
    acceptance patterns, chain-tree == causal forward, single-key attention,
    RoPE relative-position property, torch's own attention routine).
  * input of the adaptation layers (Eq. 1): concatenation order [hidden ; embedding],
    which token's embedding, and causality over the pending rows are pinned.
  * draft-module numerics (inside of the adaptation layers, the head MLP form, the
    residual in the Auto-embedding Block): the paper prints no values and ships
    no weights, so beyond the structural pins (permutation equivariance of the
    block, head -> stage split, shapes) these are "parity unpinned".
  * tree topology: "parity unpinned" against the paper's data-fitted tree, which
    is not printed; pinned structurally only.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import torch


# ----------------------------------------------------------------------------
# primitives
# ----------------------------------------------------------------------------
def rmsnorm(x: torch.Tensor, g: torch.Tensor, eps: float) -> torch.Tensor:
    """g * x / sqrt(mean(x^2) + eps) over the last axis (Llama-style, as in Vicuna)."""
    ms = (x * x).mean(dim=-1, keepdim=True)
    return g * (x / torch.sqrt(ms + eps))


def rope(x: torch.Tensor, pos: int, n_heads: int, head_dim: int, theta: float) -> torch.Tensor:
    """Rotary embedding of one row x[n_heads*head_dim] at integer position `pos`.

    Within each head, pair (i, i + head_dim/2) is rotated by pos * theta^(-2i/head_dim).
    """
    half = head_dim // 2
    xh = x.view(n_heads, head_dim)
    i = torch.arange(half, dtype=torch.float64)
    ang = pos * torch.pow(torch.tensor(theta, dtype=torch.float64), -2.0 * i / head_dim)
    c, s = torch.cos(ang).to(x.dtype), torch.sin(ang).to(x.dtype)
    a, b = xh[:, :half], xh[:, half:]
    return torch.cat([a * c - b * s, b * c + a * s], dim=1).reshape(-1)


def linear(x: torch.Tensor, w: torch.Tensor) -> torch.Tensor:
    """y = W x for every row of x; W is [out_features, in_features] (the projection every
    fully connected layer, attention projection and vocabulary head of Eq. 1-6 applies)."""
    return x @ w.T


def silu(x: torch.Tensor) -> torch.Tensor:
    return x / (1.0 + torch.exp(-x))


def attend(q: torch.Tensor, keys: torch.Tensor, vals: torch.Tensor, n_heads: int,
           head_dim: int) -> torch.Tensor:
    """Softmax attention of ONE query row over the given key / value rows, per head.

    q [H*dh]; keys, vals [S, H*dh].  Scores are q.k / sqrt(dh); softmax subtracts the max.
    """
    S = keys.shape[0]
    qh = q.view(n_heads, head_dim)
    kh = keys.view(S, n_heads, head_dim)
    vh = vals.view(S, n_heads, head_dim)
    out = torch.empty_like(qh)
    for h in range(n_heads):
        s = (kh[:, h, :] @ qh[h]) / math.sqrt(head_dim)
        p = torch.exp(s - s.max())
        p = p / p.sum()
        out[h] = p @ vh[:, h, :]
    return out.reshape(-1)


def argmax_lowest(x: torch.Tensor) -> int:
    """Index of the maximum; among equal maxima the lowest index."""
    m = x.max()
    return int(torch.nonzero(x == m)[0, 0])


def topk_desc(x: torch.Tensor, k: int) -> Tuple[List[int], List[float]]:
    """k largest entries, value descending, ties by ascending index."""
    order = sorted(range(x.numel()), key=lambda i: (-float(x[i]), i)) if x.numel() <= 4096 else None
    if order is None:
        vals, idx = torch.sort(x, descending=True, stable=True)   # stable: equal values keep index order
        order = idx[:k].tolist()
    order = order[:k]
    return [int(i) for i in order], [float(x[i]) for i in order]


# ----------------------------------------------------------------------------
# tree tables (Appendix A.1, Fig. 5)
# ----------------------------------------------------------------------------
@dataclass
class TreeTables:
    parent: List[int]
    depth: List[int]
    rank: List[int]
    ancestors: List[List[int]]      # ancestors[n]: node ids on the root -> n path, root and n included
    leaves: List[int]

    @property
    def n_nodes(self) -> int:
        return len(self.parent)


def tree_tables(parent: Sequence[int], depth: Sequence[int], rank: Sequence[int]) -> TreeTables:
    """Ancestor lists and leaves of a draft tree whose root is node 0 (Appendix A.1).

    Each node may attend only to the nodes on its own root path (Section 2, Tree Attention).
    """
    n = len(parent)
    anc: List[List[int]] = []
    for v in range(n):
        chain = []
        u = v
        while u != -1:
            chain.append(u)
            u = parent[u]
        anc.append(chain[::-1])
        assert len(anc[v]) == depth[v] + 1
    has_child = [False] * n
    for v in range(1, n):
        has_child[parent[v]] = True
    leaves = [v for v in range(n) if not has_child[v]]
    return TreeTables(list(parent), list(depth), list(rank), anc, leaves)


def tree_mask(t: TreeTables) -> torch.Tensor:
    """[N, N] 0/1 matrix: row n has ones exactly at n's ancestors (itself and the root included)."""
    m = torch.zeros(t.n_nodes, t.n_nodes, dtype=torch.int64)
    for v in range(t.n_nodes):
        for a in t.ancestors[v]:
            m[v, a] = 1
    return m


# ----------------------------------------------------------------------------
# model
# ----------------------------------------------------------------------------
@dataclass
class LayerCache:
    k: List[Optional[torch.Tensor]] = field(default_factory=list)   # k[slot] = post-RoPE key row
    v: List[Optional[torch.Tensor]] = field(default_factory=list)

    def put(self, slot: int, k: torch.Tensor, v: torch.Tensor) -> None:
        while len(self.k) <= slot:
            self.k.append(None)
            self.v.append(None)
        self.k[slot], self.v[slot] = k, v

    def rows(self, slots: Sequence[int]) -> Tuple[torch.Tensor, torch.Tensor]:
        return torch.stack([self.k[s] for s in slots]), torch.stack([self.v[s] for s in slots])

    def clone(self) -> "LayerCache":
        return LayerCache(list(self.k), list(self.v))


@dataclass
class State:
    C: int
    root: int
    kv: List[LayerCache]                 # target, one per layer
    sal_kv: List[LayerCache]             # one per adaptation layer
    pending: List[Tuple[torch.Tensor, int, int]]   # (h_j, token id at j+1, j)
    last_logits: Optional[torch.Tensor] = None     # target logits of the last prompt position (set by prefill)


class Oracle:
    """storage=None: every activation stays in `dtype` (the plain definition).
    storage=torch.bfloat16: the precision reading for bf16 models, in which every tensor that is stored
    for a later contraction is kept in bf16: the input rows of every projection, the rotated queries and
    the key / value cache rows.  Accumulation, residual stream, softmax and norms stay in `dtype`."""

    def __init__(self, shape, weights: Dict[str, torch.Tensor], dtype=torch.float64, storage=None):
        self.s = shape
        self.dtype = dtype
        self.storage = storage
        self.w = weights            # kept in storage dtype; widened on use

    def st(self, t: torch.Tensor) -> torch.Tensor:
        """Round-trip through the activation storage type (identity when storage is None)."""
        return t if self.storage is None else t.to(self.storage).to(t.dtype)

    def W(self, name: str) -> torch.Tensor:
        return self.w[name].to(self.dtype)

    # ---- one decoder layer over a set of rows ---------------------------------------------
    def decoder_rows(self, prefix: str, X: torch.Tensor, pos: Sequence[int], slots: Sequence[int],
                     visible: Sequence[Sequence[int]], cache: LayerCache) -> torch.Tensor:
        """Llama-style decoder layer applied to the rows of X [R, d].

        Row r is at position pos[r]; its key / value go to cache[slots[r]]; it attends to the
        slots in visible[r] (which include slots[r] and may include slots written by other rows
        of this call).  x <- x + Wo Attn(RMSNorm(x)); x <- x + W_down(silu(W_gate xn) * W_up xn).
        """
        s = self.s
        R = X.shape[0]
        Xn = self.st(rmsnorm(X, self.W(prefix + "attn_norm"), s.rms_eps))
        Q = Xn @ self.W(prefix + "wq").T
        Kx = Xn @ self.W(prefix + "wk").T
        V = Xn @ self.W(prefix + "wv").T
        for r in range(R):
            cache.put(slots[r], self.st(rope(Kx[r], pos[r], s.n_heads, s.head_dim, s.rope_theta)), self.st(V[r]))
        A = torch.empty_like(X)
        for r in range(R):
            assert slots[r] in visible[r]
            keys, vals = cache.rows(visible[r])
            q = self.st(rope(Q[r], pos[r], s.n_heads, s.head_dim, s.rope_theta))
            A[r] = attend(q, keys, vals, s.n_heads, s.head_dim)
        X = X + self.st(A) @ self.W(prefix + "wo").T
        Xn = self.st(rmsnorm(X, self.W(prefix + "ffn_norm"), s.rms_eps))
        act = silu(Xn @ self.W(prefix + "w_gate").T) * (Xn @ self.W(prefix + "w_up").T)
        return X + self.st(act) @ self.W(prefix + "w_down").T

    def embed(self, tok: int) -> torch.Tensor:
        return self.w["tok_emb"][int(tok)].to(self.dtype)

    def target_rows(self, toks: Sequence[int], pos: Sequence[int], slots: Sequence[int],
                    visible: Sequence[Sequence[int]], kv: List[LayerCache]
                    ) -> Tuple[torch.Tensor, torch.Tensor]:
        """Target forward of several rows, each with its own position, slot and visible set.
        Returns (post-final-norm hidden [R, d], logits [R, V])."""
        s = self.s
        X = torch.stack([self.embed(t) for t in toks])
        for l in range(s.n_layers):
            X = self.decoder_rows(f"layers.{l}.", X, pos, slots, visible, kv[l])
        hid = rmsnorm(X, self.W("final_norm"), s.rms_eps)
        return hid, self.st(hid) @ self.W("lm_head").T

    # ---- O1: prefill -------------------------------------------------------------------
    def prefill(self, prompt: Sequence[int]) -> State:
        """Causal forward of the prompt; root = greedy token after the prompt.

        The adaptation layers have seen nothing yet: every prompt position is pending.
        """
        n = len(prompt)
        kv = [LayerCache() for _ in range(self.s.n_layers)]
        vis = [list(range(j + 1)) for j in range(n)]
        hid, logits = self.target_rows(prompt, list(range(n)), list(range(n)), vis, kv)
        root = argmax_lowest(logits[n - 1])
        pending = [(hid[j], int(prompt[j + 1]) if j + 1 < n else root, j) for j in range(n)]
        return State(n, root, kv, [LayerCache() for _ in range(self.s.n_sal)], pending, logits[n - 1])

    def greedy_ar(self, prompt: Sequence[int], n_new: int) -> List[int]:
        """Plain greedy autoregressive decoding of the target: the definition the speculative
        output must reproduce token for token (lossless; Sections 1, 2 and A.3)."""
        st = self.prefill(prompt)
        out = [st.root]
        C = st.C
        while len(out) < n_new:
            _, logits = self.target_rows([out[-1]], [C], [C], [list(range(C + 1))], st.kv)
            C += 1
            out.append(argmax_lowest(logits[0]))
        return out

    # ---- O2: draft module (Section 3, Eq. 1-6) -------------------------------------------
    def draft(self, st: State, taps: Optional[dict] = None):
        """Runs the adaptation layers over the pending rows, then heads, block and LM heads.

        Returns (topk_ids[K][c_k], topk_vals[K][c_k], d_logits [K, V]).  Consumes st.pending.
        """
        s = self.s
        K = s.K
        assert st.pending, "draft needs at least one pending row"
        stage_out: List[torch.Tensor] = []          # h^1_t, h^2_t of the LAST pending row
        feats = [h for (h, _, _) in st.pending]
        for stage in range(1, s.n_sal + 1):
            fc = self.W(f"draft.fc{stage}")
            if getattr(s, "use_sampled_token", True):
                X = torch.stack([fc @ self.st(torch.cat([f, self.embed(nxt)]))   # Eq. 1: fc([h ; e_{t+1}])
                                 for (h, nxt, pos), f in zip(st.pending, feats)])
            else:            # Section 4.5, "w/o Sampled-Token": the stage sees the hidden state alone, fc is d -> d
                X = torch.stack([fc @ self.st(f) for f in feats])
            poss = [pos for (_, _, pos) in st.pending]
            vis = [list(range(p + 1)) for p in poss]                  # causal: kv_{1:t-1} and itself
            outs = list(self.decoder_rows(f"draft.sal{stage}.", X, poss, poss, vis,
                                          st.sal_kv[stage - 1]))
            feats = outs
            stage_out.append(outs[-1])
        if s.n_sal == 0:                                              # Section 4.5, "w/o Staged-Adaptation":
            stage_out = [feats[-1]]                                   # the heads read the target's h_t itself
        st.pending = []
        rows = []
        for k in range(1, K + 1):                                     # Eq. 2: head -> stage split
            src = stage_out[0] if (k <= K // 2 or s.n_sal <= 1) else stage_out[1]
            rows.append(src + silu(self.W(f"draft.mlp.{k-1}.w") @ self.st(src) + self.W(f"draft.mlp.{k-1}.b")))
        Hp = torch.stack(rows) + self.W("draft.pe")                   # Eq. 3, Eq. 4
        attn_o = Hp
        for l in range(s.aeb_layers):                                 # Eq. 5
            attn_o = self.aeb(attn_o, l)
        if s.lm_rank > 0:      # Appendix A.2.4: the head's matrix replaced by two low-rank factors, logits = B (A x)
            d_logits = torch.stack([self.W(f"draft.lm_head.{k}.b") @ self.st(self.W(f"draft.lm_head.{k}.a") @ self.st(attn_o[k]))
                                    for k in range(K)])
        else:
            d_logits = torch.stack([self.W(f"draft.lm_head.{k}") @ self.st(attn_o[k]) for k in range(K)])  # Eq. 6
        ids, vals = [], []
        for k in range(K):
            i, v = topk_desc(d_logits[k], s.topk[k])
            ids.append(i)
            vals.append(v)
        if taps is not None:
            taps.update(h1=stage_out[0], h2=stage_out[-1], Hp=Hp, attn_o=attn_o)
        return ids, vals, d_logits

    def aeb(self, Hp: torch.Tensor, l: int = 0) -> torch.Tensor:
        """Auto-embedding Block: unmasked multi-head self-attention across the K head rows,
        with a residual connection (Eq. 5; bi-directional: no mask, no positional rotation)."""
        s = self.s
        K = Hp.shape[0]
        Hs = self.st(Hp)
        q = Hs @ self.W(f"draft.aeb.{l}.wq").T
        k = Hs @ self.W(f"draft.aeb.{l}.wk").T
        v = Hs @ self.W(f"draft.aeb.{l}.wv").T
        mixed = torch.stack([attend(q[i], k, v, s.n_heads, s.head_dim) for i in range(K)])
        return Hp + self.st(mixed) @ self.W(f"draft.aeb.{l}.wo").T

    # ---- O3: tree tokens (Appendix A.1) -------------------------------------------------
    @staticmethod
    def tree_tokens(root: int, topk_ids: Sequence[Sequence[int]], t: TreeTables) -> List[int]:
        """Node 0 is the root token; a depth-k node carries head k's rank[n]-th candidate."""
        return [root] + [int(topk_ids[t.depth[n] - 1][t.rank[n]]) for n in range(1, t.n_nodes)]

    # ---- O4: tree verification (Section 2, Appendix A.1, Fig. 5) ---------------------------
    def verify(self, st: State, toks: Sequence[int], t: TreeTables):
        """One target forward over all tree tokens.  Node n sits at position C + depth[n],
        its key / value at slot C + n, and it sees the C committed slots plus its ancestors."""
        C = st.C
        N = t.n_nodes
        pos = [C + t.depth[n] for n in range(N)]
        slots = [C + n for n in range(N)]
        vis = [list(range(C)) + [C + a for a in t.ancestors[n]] for n in range(N)]
        hid, logits = self.target_rows(toks, pos, slots, vis, st.kv)
        return hid, logits, [argmax_lowest(logits[n]) for n in range(N)]

    def verify_paths_bruteforce(self, st: State, toks: Sequence[int], t: TreeTables) -> torch.Tensor:
        """Every root-to-leaf path run on its own with ordinary causal attention on a copy of
        the cache.  Returns logits [N, V] (a node shared by several paths is checked equal)."""
        C = st.C
        out: Dict[int, torch.Tensor] = {}
        for leaf in t.leaves:
            path = t.ancestors[leaf]
            kv = [c.clone() for c in st.kv]
            m = len(path)
            _, logits = self.target_rows([toks[n] for n in path], [C + i for i in range(m)],
                                         [C + i for i in range(m)],
                                         [list(range(C + i + 1)) for i in range(m)], kv)
            for i, n in enumerate(path):
                if n in out:
                    assert torch.allclose(out[n], logits[i], atol=1e-9 if self.dtype == torch.float64 else 1e-4)
                out[n] = logits[i]
        return torch.stack([out[n] for n in range(t.n_nodes)])

    # ---- O5: greedy acceptance -----------------------------------------------------------
    @staticmethod
    def accept(toks: Sequence[int], amax: Sequence[int], t: TreeTables):
        """Longest root path whose every drafted token equals the target's greedy choice at its
        parent.  Returns (L, path node ids, emitted tokens, next_root)."""
        N = t.n_nodes
        match = [True] + [int(toks[n]) == int(amax[t.parent[n]]) for n in range(1, N)]
        ok = [all(match[a] for a in t.ancestors[n]) for n in range(N)]
        best = 0
        for n in range(N):
            if ok[n] and t.depth[n] > t.depth[best]:
                best = n                                  # deepest; lowest index among equals
        path = t.ancestors[best]
        return len(path), list(path), [int(toks[n]) for n in path], int(amax[best])

    # ---- O6: compaction and carry ---------------------------------------------------------
    def commit(self, st: State, toks: Sequence[int], hid: torch.Tensor, path: Sequence[int],
               next_root: int, t: TreeTables) -> List[Tuple[int, int]]:
        """Moves the accepted nodes' key / value rows to consecutive slots C..C+L-1, drops the
        rest, and queues the accepted rows for the adaptation layers.  Returns the (dst, src)
        slot moves performed (identical for every layer)."""
        C, L = st.C, len(path)
        moves = [(C + j, C + path[j]) for j in range(L) if path[j] != j]
        for cache in st.kv:
            for j in range(L):
                cache.put(C + j, cache.k[C + path[j]], cache.v[C + path[j]])
            del cache.k[C + L:], cache.v[C + L:]
        st.pending = [(hid[path[j]], int(toks[path[j + 1]]) if j + 1 < L else int(next_root), C + j)
                      for j in range(L)]
        st.C = C + L
        st.root = int(next_root)
        return moves

    # ---- whole step ------------------------------------------------------------------------
    def step(self, st: State, t: TreeTables, override_tokens: Optional[Sequence[int]] = None,
             taps: Optional[dict] = None) -> List[int]:
        """draft -> tree -> verify -> accept -> compact.  Returns the tokens emitted this step.

        `override_tokens` (length N, entry -1 = keep the drafted token) lets a caller plant
        tokens in the tree, as a trained draft module would produce."""
        ids, vals, d_logits = self.draft(st, taps)
        toks = self.tree_tokens(st.root, ids, t)
        if override_tokens is not None:
            toks = [tk if int(o) < 0 else int(o) for tk, o in zip(toks, override_tokens)]
            toks[0] = st.root
        hid, logits, amax = self.verify(st, toks, t)
        L, path, emitted, next_root = self.accept(toks, amax, t)
        if taps is not None:
            taps.update(topk_ids=ids, topk_vals=vals, d_logits=d_logits, toks=toks, hid=hid,
                        logits=logits, amax=amax, L=L, path=path, next_root=next_root, C_before=st.C)
        moves = self.commit(st, toks, hid, path, next_root, t)
        if taps is not None:
            taps["moves"] = moves
        return emitted
