"""Step-by-step comparison of the CUDA library with the CPU oracle on the same seeded inputs.

Protocol (per step): both sides draft from their own state; the drafted top-k lists are
compared; the oracle's tree tokens (drafted, or with a planted path) are handed to
amph_verify_tree so both sides verify the same tokens; logits / hidden rows are compared
within tolerance; integer outputs (argmax, accepted path, emitted tokens, next root,
compacted cache rows) must be identical wherever the oracle's own decision has a margin
larger than the floating-point tolerance.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import torch

import inputs
from oracle import amphista_oracle as ao


@dataclass
class Report:
    steps: int = 0
    max_logit_err: float = 0.0
    max_hidden_err: float = 0.0
    max_dlogit_err: float = 0.0
    max_draft_err: float = 0.0
    max_kv_err: float = 0.0
    own_tree_steps: int = 0        # steps verified on the tree the GPU built from its own candidates
    topk_tie_swaps: int = 0
    argmax_near_ties: int = 0
    gated_steps: int = 0
    accepted: List[int] = field(default_factory=list)


def rel_err(g: torch.Tensor, o: torch.Tensor) -> float:
    """max |g - o| / max(1, max |o|)"""
    o = o.to(torch.float64)
    return float((g.to(torch.float64).cpu() - o).abs().max() / max(1.0, float(o.abs().max())))


def plant(t: ao.TreeTables, future: List[int], leaf: int) -> List[int]:
    ov = [-1] * t.n_nodes
    for i, n in enumerate(t.ancestors[leaf]):
        if i > 0 and i - 1 < len(future):
            ov[n] = future[i - 1]
    return ov


def compare_topk(shape, g_ids, g_vals, o_dlogits, tie_tol, rep: Report):
    for k in range(shape.K):
        c = shape.topk[k]
        row = o_dlogits[k].to(torch.float64)
        o_ids, _ = ao.topk_desc(row, c)
        gi = [int(v) for v in g_ids[k, :c].tolist()]
        assert len(set(gi)) == c, f"head {k}: duplicate candidates {gi}"
        kth = float(row[o_ids[-1]])
        for pos, (a, b) in enumerate(zip(gi, o_ids)):
            if a != b:
                # only allowed when the oracle's own values are within the tie tolerance
                assert abs(float(row[a]) - float(row[b])) <= tie_tol, \
                    f"head {k} rank {pos}: gpu id {a} ({float(row[a]):.6f}) vs oracle id {b} ({float(row[b]):.6f})"
                rep.topk_tie_swaps += 1
        for a in set(gi) - set(o_ids):
            assert float(row[a]) >= kth - tie_tol
        gv = g_vals[k, :c].to(torch.float64).cpu()
        ov = torch.tensor([float(row[i]) for i in gi], dtype=torch.float64)
        assert float((gv - ov).abs().max()) <= max(tie_tol, 1e-6) * 40 + 1e-9


def run_parity(model, orc: ao.Oracle, shape, topo, prompt: List[int], steps: int, tol: float,
               tie_tol: float, planted: bool, kv_check_layers=(0, -1), tol_draft: Optional[float] = None) -> Report:
    """model: paper_2406_13170_b200.Amphista.  Returns the error report; raises on a mismatch.
    tol bounds the target's tensors, tol_draft (default: tol) those of the draft module."""
    if tol_draft is None:
        tol_draft = tol
    dev = model.device
    t = ao.tree_tables(topo.parent, topo.depth, topo.rank)
    N, K, d, V = t.n_nodes, shape.K, shape.d_model, shape.vocab
    rep = Report()
    st = orc.prefill(prompt)
    root = model.prefill(prompt)
    # logits of the last prompt position: row (n-1) mod 512 of the last prefill pass (a pass carries 4 x AMPH_MAX_NODES
    # prompt tokens; AMPH_MAX_NODES with AMPH_FLAG_CHUNKED_PREFILL = 128)
    last_row = (len(prompt) - 1) % (128 if (model.cfg.flags & 128) else 512)
    g_last = model.get_tensor("logits", (last_row + 1, V))[last_row]
    e = rel_err(g_last, st.last_logits)
    rep.max_logit_err = max(rep.max_logit_err, e)
    assert e <= tol, f"prefill logits off by {e}"
    if root != st.root:
        # only a near-tie of the oracle's own top two logits may flip the greedy choice
        top2 = torch.topk(st.last_logits.to(torch.float64), 2).values
        e_abs = float((g_last.to(torch.float64).cpu() - st.last_logits.to(torch.float64)).abs().max())
        assert float(top2[0] - top2[1]) <= 2.0 * e_abs, f"prefill root {root} vs oracle {st.root}"
        rep.argmax_near_ties += 1
        model.set_tensor("root", torch.tensor([st.root], dtype=torch.int32, device=dev))
    future = orc.greedy_ar(prompt, steps * (K + 1) + K + 2) if planted else None
    emitted_total: List[int] = []
    g_ids = torch.zeros(K, 16, dtype=torch.int32, device=dev)
    g_vals = torch.zeros(K, 16, dtype=torch.float32, device=dev)
    g_amax = torch.zeros(N, dtype=torch.int32, device=dev)
    g_tok = torch.zeros(K + 1, dtype=torch.int32, device=dev)
    g_path = torch.zeros(K + 1, dtype=torch.int32, device=dev)
    g_n = torch.zeros(1, dtype=torch.int32, device=dev)
    g_next = torch.zeros(1, dtype=torch.int32, device=dev)
    for i in range(steps):
        C0 = st.C
        assert model.get_state()[0] == C0
        ov = None
        if planted:
            leaf = t.leaves[i % len(t.leaves)]
            ov = plant(t, future[len(emitted_total) + 1: len(emitted_total) + 1 + t.depth[leaf]], leaf)
        taps = {}
        emitted = orc.step(st, t, ov, taps)
        # ---- draft
        model.draft(g_ids, g_vals)
        torch.cuda.synchronize(dev)
        g_dl = model.get_tensor("d_logits", (K, V))
        scale = max(1.0, float(taps["d_logits"].abs().max()))
        rep.max_dlogit_err = max(rep.max_dlogit_err, rel_err(g_dl, taps["d_logits"]))
        assert rel_err(g_dl, taps["d_logits"]) <= tol_draft, f"step {i}: draft logits off by {rel_err(g_dl, taps['d_logits'])}"
        e_hp = rel_err(model.get_tensor("hp", (K, d)), taps["Hp"])
        e_ao = rel_err(model.get_tensor("attn_o", (K, d)), taps["attn_o"])
        sal_h = model.get_tensor("sal_h", (2, d))
        e_h1, e_h2 = rel_err(sal_h[0], taps["h1"]), rel_err(sal_h[1], taps["h2"])
        rep.max_draft_err = max(rep.max_draft_err, e_hp, e_ao, e_h1, e_h2)
        assert max(e_hp, e_ao, e_h1, e_h2) <= tol_draft, f"step {i}: draft hidden states off by {(e_h1, e_h2, e_hp, e_ao)}"
        # two candidates can only trade places if their oracle values are closer than twice the
        # measured error of the draft logits (itself bounded by tol above), or than the stated tie width
        e_abs = float((g_dl.to(torch.float64).cpu() - taps["d_logits"].to(torch.float64)).abs().max())
        compare_topk(shape, g_ids, g_vals, taps["d_logits"], max(tie_tol * scale, 2.0 * e_abs), rep)
        # ---- tree construction (Appendix A.1): node 0 carries the root, a depth-k node head k's candidate of its
        # rank.  The tokens the library gathered must be that function of the library's OWN candidate lists.
        root_i = int(taps["toks"][0])
        g_tt = model.get_tensor("tree_tokens", (N,), torch.int32).tolist()
        assert g_tt == ao.Oracle.tree_tokens(root_i, g_ids.tolist(), t), f"step {i}: tree tokens are not the gathered candidates"
        # ---- verify.  When the library drafted the oracle's candidates (no near-tie swap) it verifies its own tree:
        # NULL keeps every drafted token, a planted path arrives as overrides with -1 = "keep the drafted token".
        # Otherwise both sides verify the oracle's tokens so that the rows stay comparable.
        if g_tt == ao.Oracle.tree_tokens(root_i, taps["topk_ids"], t):
            rep.own_tree_steps += 1
            model.verify_tree(None if ov is None else torch.tensor(ov, dtype=torch.int32, device=dev), g_amax)
        else:
            model.verify_tree(torch.tensor(taps["toks"], dtype=torch.int32, device=dev), g_amax)
        torch.cuda.synchronize(dev)
        assert model.get_tensor("tree_tokens", (N,), torch.int32).tolist() == taps["toks"]
        g_logits = model.get_tensor("logits", (N, V))
        g_hidden = model.get_tensor("hidden", (N, d))
        le, he = rel_err(g_logits, taps["logits"]), rel_err(g_hidden, taps["hid"])
        rep.max_logit_err, rep.max_hidden_err = max(rep.max_logit_err, le), max(rep.max_hidden_err, he)
        assert le <= tol, f"step {i}: logits off by {le}"
        assert he <= tol, f"step {i}: hidden off by {he}"
        lscale = max(1.0, float(taps["logits"].abs().max()))
        top2 = torch.topk(taps["logits"].to(torch.float64), 2, dim=1).values
        gaps = (top2[:, 0] - top2[:, 1])
        # a greedy choice can only flip if the oracle's top-2 gap is below twice the measured logit error
        e_log = float((g_logits.to(torch.float64).cpu() - taps["logits"].to(torch.float64)).abs().max())
        safe = gaps > max(2.0 * e_log, 1e-6 * lscale)
        ga = g_amax.tolist()
        for n in range(N):
            if bool(safe[n]):
                assert ga[n] == taps["amax"][n], f"step {i} node {n}: argmax {ga[n]} vs {taps['amax'][n]}"
            else:
                rep.argmax_near_ties += 1
        # ---- accept.  The acceptance kernel itself is integer logic: fed the oracle's argmax it must
        # reproduce the oracle bit for bit, whatever the floating-point margins were.
        all_safe = bool(safe.all())
        if not all_safe:
            rep.gated_steps += 1
            model.set_tensor("argmax", torch.tensor(taps["amax"], dtype=torch.int32, device=dev))
        model.accept(g_tok, g_n, g_path, g_next)
        torch.cuda.synchronize(dev)
        L = int(g_n[0])
        assert L == taps["L"], f"step {i}: accepted {L} vs oracle {taps['L']}"
        assert g_path[:L].tolist() == taps["path"]
        assert g_tok[:L].tolist() == emitted
        assert int(g_next[0]) == taps["next_root"]
        C1, groot, npend = model.get_state()
        assert (C1, groot, npend) == (st.C, st.root, L)
        # ---- compacted cache rows of this step
        for l in sorted(set(x % shape.n_layers for x in kv_check_layers)):
            for which, cache in (("k", st.kv[l].k), ("v", st.kv[l].v)):
                rows = model.get_tensor(f"kv.{which}.{l}@{C0}", (L, d))
                ref = torch.stack(cache[C0:C0 + L])
                e = rel_err(rows, ref)
                rep.max_kv_err = max(rep.max_kv_err, e)
                assert e <= tol, f"step {i}: layer {l} {which} cache rows off by {e}"
        emitted_total += emitted
        rep.accepted.append(L)
        rep.steps += 1
    # adaptation-layer caches cover every position committed before the last step
    for s in range(shape.n_sal):
        n_rows = len(st.sal_kv[s].k)
        for which, cache in (("k", st.sal_kv[s].k), ("v", st.sal_kv[s].v)):
            rows = model.get_tensor(f"sal{s+1}.{which}", (n_rows, d))
            e = rel_err(rows, torch.stack(cache))
            rep.max_kv_err = max(rep.max_kv_err, e)
            assert e <= tol_draft, f"stage {s+1} {which} cache off by {e}"
    return rep


def run_parity_batch(model, borc, shape, topo, prompts: List[List[int]], steps: int, tol: float, tie_tol: float,
                     futures: Optional[List[List[int]]] = None) -> List[Report]:
    """The same protocol for max_batch sequences decoded side by side (Section 4.4): `borc` is the batched oracle
    (oracle.amphista_batch_oracle.BatchOracle), prompts one list per sequence (lengths may differ).  With `futures`
    (each sequence's true greedy continuation) a path of a different depth is planted per sequence and step, so that
    the sequences accept different numbers of tokens and their lengths drift apart.  One Report per sequence."""
    dev = model.device
    t = ao.tree_tables(topo.parent, topo.depth, topo.rank)
    N, K, d, V, B = t.n_nodes, shape.K, shape.d_model, shape.vocab, len(prompts)
    reps = [Report() for _ in range(B)]
    bs = borc.prefill(prompts)
    for b in range(B):
        root = model.prefill(prompts[b], seq=b)
        if root != bs.root[b]:
            top2 = torch.topk(bs.last_logits[b].to(torch.float64), 2).values
            assert float(top2[0] - top2[1]) <= 2.0 * tol * max(1.0, float(bs.last_logits[b].abs().max())), \
                f"sequence {b}: prefill root {root} vs oracle {bs.root[b]}"
            reps[b].argmax_near_ties += 1
            model.set_tensor(f"root#{b}", torch.tensor([bs.root[b]], dtype=torch.int32, device=dev))
    done = [0] * B
    g_ids = torch.zeros(B, K, 16, dtype=torch.int32, device=dev)
    g_vals = torch.zeros(B, K, 16, dtype=torch.float32, device=dev)
    g_amax = torch.zeros(B, N, dtype=torch.int32, device=dev)
    g_tok = torch.zeros(B, K + 1, dtype=torch.int32, device=dev)
    g_path = torch.zeros(B, K + 1, dtype=torch.int32, device=dev)
    g_n = torch.zeros(B, dtype=torch.int32, device=dev)
    g_next = torch.zeros(B, dtype=torch.int32, device=dev)
    for i in range(steps):
        C0 = list(bs.C)
        for b in range(B):
            assert model.get_state(b)[0] == C0[b]
        ovs = None
        if futures is not None:
            ovs = []
            for b in range(B):
                leaf = t.leaves[(i + 2 * b) % len(t.leaves)]
                ovs.append(plant(t, futures[b][done[b] + 1: done[b] + 1 + t.depth[leaf]], leaf) if (i + b) % 3 else None)
        taps = [dict() for _ in range(B)]
        emitted = borc.step(bs, t, ovs, taps)
        model.draft(g_ids, g_vals)
        torch.cuda.synchronize(dev)
        for b in range(B):
            tp, rep = taps[b], reps[b]
            g_dl = model.get_tensor(f"d_logits#{b}", (K, V))
            e_dl = rel_err(g_dl, tp["d_logits"])
            e_hp = rel_err(model.get_tensor(f"hp#{b}", (K, d)), tp["Hp"])
            e_ao = rel_err(model.get_tensor(f"attn_o#{b}", (K, d)), tp["attn_o"])
            sal_h = model.get_tensor(f"sal_h#{b}", (2, d))
            e_h = max(rel_err(sal_h[0], tp["h1"]), rel_err(sal_h[1], tp["h2"]))
            rep.max_dlogit_err = max(rep.max_dlogit_err, e_dl)
            rep.max_draft_err = max(rep.max_draft_err, e_hp, e_ao, e_h)
            assert max(e_dl, e_hp, e_ao, e_h) <= tol, f"step {i} sequence {b}: draft tensors off by {(e_dl, e_hp, e_ao, e_h)}"
            scale = max(1.0, float(tp["d_logits"].abs().max()))
            e_abs = float((g_dl.to(torch.float64).cpu() - tp["d_logits"].to(torch.float64)).abs().max())
            compare_topk(shape, g_ids[b], g_vals[b], tp["d_logits"], max(tie_tol * scale, 2.0 * e_abs), rep)
            g_tt = model.get_tensor(f"tree_tokens#{b}", (N,), torch.int32).tolist()
            assert g_tt == ao.Oracle.tree_tokens(int(tp["toks"][0]), g_ids[b].tolist(), t), f"step {i} sequence {b}: tree tokens"
        model.verify_tree(torch.tensor([tp["toks"] for tp in taps], dtype=torch.int32, device=dev), g_amax)
        torch.cuda.synchronize(dev)
        for b in range(B):
            tp, rep = taps[b], reps[b]
            g_logits = model.get_tensor(f"logits#{b}", (N, V))
            g_hidden = model.get_tensor(f"hidden#{b}", (N, d))
            le, he = rel_err(g_logits, tp["logits"]), rel_err(g_hidden, tp["hid"])
            rep.max_logit_err, rep.max_hidden_err = max(rep.max_logit_err, le), max(rep.max_hidden_err, he)
            assert max(le, he) <= tol, f"step {i} sequence {b}: logits / hidden off by {(le, he)}"
            lscale = max(1.0, float(tp["logits"].abs().max()))
            top2 = torch.topk(tp["logits"].to(torch.float64), 2, dim=1).values
            e_log = float((g_logits.to(torch.float64).cpu() - tp["logits"].to(torch.float64)).abs().max())
            safe = (top2[:, 0] - top2[:, 1]) > max(2.0 * e_log, 1e-6 * lscale)
            ga = g_amax[b].tolist()
            for n in range(N):
                if bool(safe[n]):
                    assert ga[n] == tp["amax"][n], f"step {i} sequence {b} node {n}: argmax {ga[n]} vs {tp['amax'][n]}"
                else:
                    rep.argmax_near_ties += 1
            if not bool(safe.all()):
                rep.gated_steps += 1
                model.set_tensor(f"argmax#{b}", torch.tensor(tp["amax"], dtype=torch.int32, device=dev))
        model.accept(g_tok, g_n, g_path, g_next)
        torch.cuda.synchronize(dev)
        for b in range(B):
            tp, rep = taps[b], reps[b]
            L = int(g_n[b])
            assert L == tp["L"], f"step {i} sequence {b}: accepted {L} vs oracle {tp['L']}"
            assert g_path[b, :L].tolist() == tp["path"] and g_tok[b, :L].tolist() == emitted[b]
            assert int(g_next[b]) == tp["next_root"]
            assert model.get_state(b) == (bs.C[b], bs.root[b], L)
            for which, cache in (("k", bs.K[0]), ("v", bs.V[0])):       # compacted rows of the first layer, this sequence's cache
                rows = model.get_tensor(f"kv.{which}.0#{b}@{C0[b]}", (L, d))
                e = rel_err(rows, cache[b, C0[b]:C0[b] + L])
                rep.max_kv_err = max(rep.max_kv_err, e)
                assert e <= tol, f"step {i} sequence {b}: {which} cache rows off by {e}"
            done[b] += L
            rep.accepted.append(L)
            rep.steps += 1
    for b in range(B):                                                  # adaptation-layer caches, per sequence
        for s in range(shape.n_sal):
            n_rows = bs.C[b] - len(bs.pending[b])
            rows = model.get_tensor(f"sal{s+1}.k#{b}", (n_rows, d))
            e = rel_err(rows, bs.sal_K[s][b, :n_rows])
            reps[b].max_kv_err = max(reps[b].max_kv_err, e)
            assert e <= tol, f"sequence {b}: stage {s+1} cache off by {e}"
    return reps
