"""CPU oracle for several sequences decoded side by side (arXiv 2406.13170, Section 4.4).

TEST INFRASTRUCTURE ONLY (imported by the tests alone; the product path never calls it).

Section 4.4 evaluates Amphista at batch sizes above one: sentences of different lengths are padded to a common
length and the position of every sentence's last valid token is tracked.  This module restates the decoding step
in exactly that form: every tensor carries a leading batch axis, rows and cache slots beyond a sentence's own
length are padding, a boolean visibility tensor keeps padding out of every softmax, and the quantities a step
reads from "the last token" (the greedy root after the prompt, the row that feeds the drafting heads) are taken
at each sentence's own last valid index.  The arithmetic per valid row is that of the single-sequence oracle
(amphista_oracle.Oracle); the formulation differs on purpose (dense padded tensors and masks here, per-row Python
lists there), and tests pin the two against each other: a batched step must reproduce, sentence by sentence,
what each sentence gives when it is decoded alone.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence, Tuple

import torch

from oracle.amphista_oracle import Oracle, TreeTables, argmax_lowest, rmsnorm, silu, topk_desc


@dataclass
class BatchState:
    C: List[int]                           # committed tokens per sentence (cache slots 0..C-1 are valid)
    root: List[int]                        # token chosen for position C of each sentence
    K: List[torch.Tensor]                  # per target layer [B, S, d] (padded; S grows on demand)
    V: List[torch.Tensor]
    sal_K: List[torch.Tensor]              # per adaptation layer [B, S, d]
    sal_V: List[torch.Tensor]
    pending: List[List[Tuple[torch.Tensor, int, int]]]   # per sentence (h_j, token id at j+1, j)
    last_logits: List[torch.Tensor]


def _grow(t: torch.Tensor, S: int) -> torch.Tensor:
    """Pads the slot axis of a [B, S0, d] cache with zero rows up to S slots."""
    if t.shape[1] >= S:
        return t
    pad = torch.zeros(t.shape[0], S - t.shape[1], t.shape[2], dtype=t.dtype)
    return torch.cat([t, pad], dim=1)


class BatchOracle:
    def __init__(self, shape, weights: Dict[str, torch.Tensor], dtype=torch.float64, storage=None):
        self.s = shape
        self.dtype = dtype
        self.storage = storage
        self.w = weights

    def st(self, t: torch.Tensor) -> torch.Tensor:
        return t if self.storage is None else t.to(self.storage).to(t.dtype)

    def W(self, name: str) -> torch.Tensor:
        return self.w[name].to(self.dtype)

    # ---- rotary embedding of a padded block of rows -----------------------------------------
    def rope_rows(self, X: torch.Tensor, pos: torch.Tensor) -> torch.Tensor:
        """X [B, R, H*dh], pos [B, R] integer positions: pair (i, i + dh/2) of every head rotated by pos * theta^(-2i/dh)."""
        s = self.s
        B, R, _ = X.shape
        half = s.head_dim // 2
        i = torch.arange(half, dtype=torch.float64)
        inv = torch.pow(torch.tensor(s.rope_theta, dtype=torch.float64), -2.0 * i / s.head_dim)
        ang = pos.to(torch.float64).unsqueeze(-1) * inv                       # [B, R, half]
        c, sn = torch.cos(ang).to(X.dtype).unsqueeze(2), torch.sin(ang).to(X.dtype).unsqueeze(2)
        xh = X.view(B, R, s.n_heads, s.head_dim)
        a, b = xh[..., :half], xh[..., half:]
        return torch.cat([a * c - b * sn, b * c + a * sn], dim=-1).reshape(B, R, -1)

    # ---- one decoder layer over a padded block of rows ----------------------------------------
    def decoder_block(self, prefix: str, X: torch.Tensor, pos: torch.Tensor, slot: torch.Tensor, vis: torch.Tensor,
                      valid: torch.Tensor, Kc: torch.Tensor, Vc: torch.Tensor):
        """X [B, R, d]; row (b, r) sits at position pos[b, r], writes its key / value to slot[b, r] of sentence b's
        cache and may see the slots s with vis[b, r, s]; rows with valid[b, r] == False are padding (they write
        nothing and their output is meaningless).  Returns (X_out, Kc, Vc)."""
        s = self.s
        B, R, d = X.shape
        H, dh = s.n_heads, s.head_dim
        Xn = self.st(rmsnorm(X, self.W(prefix + "attn_norm"), s.rms_eps))
        Q = self.st(self.rope_rows(Xn @ self.W(prefix + "wq").T, pos))
        Kn = self.st(self.rope_rows(Xn @ self.W(prefix + "wk").T, pos))
        Vn = self.st(Xn @ self.W(prefix + "wv").T)
        S = max(int(vis.shape[2]), int(slot[valid].max()) + 1 if bool(valid.any()) else 0)
        Kc, Vc = _grow(Kc, S), _grow(Vc, S)
        for b in range(B):
            for r in range(R):
                if bool(valid[b, r]):
                    Kc[b, int(slot[b, r])] = Kn[b, r]
                    Vc[b, int(slot[b, r])] = Vn[b, r]
        vis = torch.cat([vis, torch.zeros(B, R, S - vis.shape[2], dtype=torch.bool)], dim=2) if vis.shape[2] < S else vis
        vis = vis.clone()
        vis[~valid] = False
        vis[..., 0] |= ~valid                                      # a padding row looks at one slot so that its softmax is defined
        qh = Q.view(B, R, H, dh).permute(0, 2, 1, 3)              # [B, H, R, dh]
        kh = Kc[:, :S].reshape(B, S, H, dh).permute(0, 2, 3, 1)   # [B, H, dh, S]
        vh = Vc[:, :S].reshape(B, S, H, dh).permute(0, 2, 1, 3)   # [B, H, S, dh]
        sc = (qh @ kh) / math.sqrt(dh)                            # [B, H, R, S]
        sc = sc.masked_fill(~vis.unsqueeze(1), float("-inf"))     # padding and foreign tree branches never enter the softmax
        p = torch.exp(sc - sc.max(dim=-1, keepdim=True).values)
        p = p / p.sum(dim=-1, keepdim=True)
        A = (p @ vh).permute(0, 2, 1, 3).reshape(B, R, d)
        X = X + self.st(A) @ self.W(prefix + "wo").T
        Xn = self.st(rmsnorm(X, self.W(prefix + "ffn_norm"), s.rms_eps))
        act = silu(Xn @ self.W(prefix + "w_gate").T) * (Xn @ self.W(prefix + "w_up").T)
        return X + self.st(act) @ self.W(prefix + "w_down").T, Kc, Vc

    def target_block(self, toks: torch.Tensor, pos, slot, vis, valid, bs_K, bs_V):
        s = self.s
        X = self.w["tok_emb"][toks.clamp(min=0)].to(self.dtype)
        for l in range(s.n_layers):
            X, bs_K[l], bs_V[l] = self.decoder_block(f"layers.{l}.", X, pos, slot, vis, valid, bs_K[l], bs_V[l])
        hid = rmsnorm(X, self.W("final_norm"), s.rms_eps)
        return hid, self.st(hid) @ self.W("lm_head").T

    # ---- prefill: prompts padded on the right to the longest one -------------------------------
    def prefill(self, prompts: Sequence[Sequence[int]]) -> BatchState:
        s = self.s
        B = len(prompts)
        n = [len(p) for p in prompts]
        R = max(n)
        toks = torch.zeros(B, R, dtype=torch.long)
        valid = torch.zeros(B, R, dtype=torch.bool)
        for b, p in enumerate(prompts):
            toks[b, :n[b]] = torch.tensor(list(p), dtype=torch.long)
            valid[b, :n[b]] = True
        pos = torch.arange(R).unsqueeze(0).repeat(B, 1)
        vis = (torch.arange(R).view(1, 1, R) <= torch.arange(R).view(1, R, 1)).repeat(B, 1, 1)   # causal; padding comes after
        K = [torch.zeros(B, R, s.d_model, dtype=self.dtype) for _ in range(s.n_layers)]
        V = [torch.zeros(B, R, s.d_model, dtype=self.dtype) for _ in range(s.n_layers)]
        hid, logits = self.target_block(toks, pos, pos, vis, valid, K, V)
        root, pending, last = [], [], []
        for b in range(B):
            j_last = n[b] - 1                                          # the sentence's last valid token
            root.append(argmax_lowest(logits[b, j_last]))
            last.append(logits[b, j_last])
            pending.append([(hid[b, j], int(prompts[b][j + 1]) if j + 1 < n[b] else root[b], j) for j in range(n[b])])
        z = lambda: [torch.zeros(B, 1, s.d_model, dtype=self.dtype) for _ in range(s.n_sal)]
        return BatchState(list(n), root, K, V, z(), z(), pending, last)

    # ---- draft module over the padded pending rows -----------------------------------------------
    def draft(self, bs: BatchState, taps: Optional[List[dict]] = None):
        s = self.s
        B, K, d = len(bs.C), s.K, s.d_model
        P = [len(p) for p in bs.pending]
        assert min(P) >= 1
        R = max(P)
        valid = torch.zeros(B, R, dtype=torch.bool)
        pos = torch.zeros(B, R, dtype=torch.long)
        feats = torch.zeros(B, R, d, dtype=self.dtype)
        nxt = torch.zeros(B, R, dtype=torch.long)
        for b in range(B):
            for r, (h, tok, p) in enumerate(bs.pending[b]):
                valid[b, r], pos[b, r], nxt[b, r] = True, p, tok
                feats[b, r] = h
        S = int(pos.max()) + 1
        vis = (torch.arange(S).view(1, 1, S) <= pos.unsqueeze(-1)) & valid.unsqueeze(-1)       # causal over the stage's own cache
        emb = self.w["tok_emb"][nxt].to(self.dtype)
        stage_last: List[torch.Tensor] = []
        for stage in range(1, s.n_sal + 1):
            fc = self.W(f"draft.fc{stage}")
            if getattr(s, "use_sampled_token", True):
                X = self.st(torch.cat([feats, emb], dim=-1)) @ fc.T                          # Eq. 1
            else:
                X = self.st(feats) @ fc.T
            X, bs.sal_K[stage - 1], bs.sal_V[stage - 1] = self.decoder_block(
                f"draft.sal{stage}.", X, pos, pos, vis, valid, bs.sal_K[stage - 1], bs.sal_V[stage - 1])
            feats = X
            stage_last.append(torch.stack([X[b, P[b] - 1] for b in range(B)]))                # each sentence's last valid row
        if s.n_sal == 0:
            stage_last = [torch.stack([feats[b, P[b] - 1] for b in range(B)])]
        bs.pending = [[] for _ in range(B)]
        rows = []
        for k in range(1, K + 1):                                                             # Eq. 2
            src = stage_last[0] if (k <= K // 2 or s.n_sal <= 1) else stage_last[1]
            rows.append(src + silu(self.st(src) @ self.W(f"draft.mlp.{k-1}.w").T + self.W(f"draft.mlp.{k-1}.b")))
        Hp = torch.stack(rows, dim=1) + self.W("draft.pe")                                    # [B, K, d], Eq. 3-4
        attn_o = Hp
        H, dh = s.n_heads, s.head_dim
        for l in range(s.aeb_layers):                                                         # Eq. 5, per sentence, no mask
            Hs = self.st(attn_o)
            q = (Hs @ self.W(f"draft.aeb.{l}.wq").T).view(B, K, H, dh).permute(0, 2, 1, 3)
            k_ = (Hs @ self.W(f"draft.aeb.{l}.wk").T).view(B, K, H, dh).permute(0, 2, 3, 1)
            v = (Hs @ self.W(f"draft.aeb.{l}.wv").T).view(B, K, H, dh).permute(0, 2, 1, 3)
            sc = (q @ k_) / math.sqrt(dh)
            p = torch.exp(sc - sc.max(dim=-1, keepdim=True).values)
            p = p / p.sum(dim=-1, keepdim=True)
            mixed = (p @ v).permute(0, 2, 1, 3).reshape(B, K, d)
            attn_o = attn_o + self.st(mixed) @ self.W(f"draft.aeb.{l}.wo").T
        if s.lm_rank > 0:
            d_logits = torch.stack([self.st(self.st(attn_o[:, k]) @ self.W(f"draft.lm_head.{k}.a").T) @ self.W(f"draft.lm_head.{k}.b").T
                                    for k in range(K)], dim=1)
        else:
            d_logits = torch.stack([self.st(attn_o[:, k]) @ self.W(f"draft.lm_head.{k}").T for k in range(K)], dim=1)   # Eq. 6
        ids = [[topk_desc(d_logits[b, k], s.topk[k])[0] for k in range(K)] for b in range(B)]
        if taps is not None:
            for b in range(B):
                taps[b].update(h1=stage_last[0][b], h2=stage_last[-1][b], Hp=Hp[b], attn_o=attn_o[b], d_logits=d_logits[b],
                               topk_ids=ids[b])
        return ids, d_logits

    # ---- tree verification over all sentences ------------------------------------------------------
    def verify(self, bs: BatchState, toks: Sequence[Sequence[int]], t: TreeTables):
        B, N = len(bs.C), t.n_nodes
        S = max(bs.C) + N
        tk = torch.tensor([list(x) for x in toks], dtype=torch.long)
        C = torch.tensor(bs.C).view(B, 1)
        depth = torch.tensor(t.depth).view(1, N)
        pos = C + depth
        slot = C + torch.arange(N).view(1, N)
        vis = torch.zeros(B, N, S, dtype=torch.bool)
        for b in range(B):
            vis[b, :, :bs.C[b]] = True                              # the sentence's own committed tokens; nothing of the padding
            for n in range(N):
                for a in t.ancestors[n]:
                    vis[b, n, bs.C[b] + a] = True
        valid = torch.ones(B, N, dtype=torch.bool)
        hid, logits = self.target_block(tk, pos, slot, vis, valid, bs.K, bs.V)
        amax = [[argmax_lowest(logits[b, n]) for n in range(N)] for b in range(B)]
        return hid, logits, amax

    # ---- acceptance, compaction and carry, sentence by sentence --------------------------------------
    def commit(self, bs: BatchState, b: int, toks, hid_b, path, next_root):
        C, L = bs.C[b], len(path)
        for Kc, Vc in zip(bs.K, bs.V):
            for j in range(L):
                Kc[b, C + j] = Kc[b, C + path[j]].clone()
                Vc[b, C + j] = Vc[b, C + path[j]].clone()
            Kc[b, C + L:] = 0                                        # what follows the last valid token is padding again
            Vc[b, C + L:] = 0
        bs.pending[b] = [(hid_b[path[j]], int(toks[path[j + 1]]) if j + 1 < L else int(next_root), C + j) for j in range(L)]
        bs.C[b] = C + L
        bs.root[b] = int(next_root)

    def step(self, bs: BatchState, t: TreeTables, overrides: Optional[Sequence[Optional[Sequence[int]]]] = None,
             taps: Optional[List[dict]] = None) -> List[List[int]]:
        """draft -> tree -> verify -> accept -> compact for every sentence; returns the tokens each emitted."""
        B = len(bs.C)
        ids, _ = self.draft(bs, taps)
        toks = []
        for b in range(B):
            tb = Oracle.tree_tokens(bs.root[b], ids[b], t)
            if overrides is not None and overrides[b] is not None:
                tb = [x if int(o) < 0 else int(o) for x, o in zip(tb, overrides[b])]
                tb[0] = bs.root[b]
            toks.append(tb)
        hid, logits, amax = self.verify(bs, toks, t)
        out = []
        for b in range(B):
            L, path, emitted, nxt = Oracle.accept(toks[b], amax[b], t)
            if taps is not None:
                taps[b].update(toks=toks[b], hid=hid[b], logits=logits[b], amax=amax[b], L=L, path=path, next_root=nxt,
                               C_before=bs.C[b])
            self.commit(bs, b, toks[b], hid[b], path, nxt)
            out.append(emitted)
        return out
