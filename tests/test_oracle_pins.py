"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each one is meant to fail under a
plausible mistake in the oracle (a wrong mask bit, position, slot, sign, transposed
operand, dropped residual, off-by-one in the accepted path, ...).
"""
import itertools
import math
import os

import pytest
import torch

import inputs
from inputs.configs import ModelShape
from oracle import amphista_oracle as ao

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
MICRO = ModelShape("micro", 2, 64, 2, 32, 96, 50, "fp32", topk=(3, 2, 2, 1), n_nodes=12,
                   prompt_len=9, steps=6)
TINY = inputs.get_shape("tiny")


def _golden(name):
    out = {}
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            k, *v = line.split()
            out[k] = [int(x) for x in v]
    return out


def _oracle(shape, std=0.02, seed=0):
    w = inputs.make_weights(shape, seed=seed, std=std)
    return ao.Oracle(shape, w, dtype=torch.float64)


def _tables(topo):
    return ao.tree_tables(topo.parent, topo.depth, topo.rank)


# --------------------------------------------------------------------------------------
# Fig. 5 worked example and the paper's shape facts
# --------------------------------------------------------------------------------------
def test_fig5_counts():
    g = _golden("fig5_tree.txt")
    topo = inputs.full_tree(g["top"])
    t = _tables(topo)
    assert t.n_nodes == g["nodes"][0]
    assert len(t.leaves) == g["candidates"][0]
    m = ao.tree_mask(t)
    for n in range(t.n_nodes):
        assert int(m[n].sum()) == t.depth[n] + 1          # ancestors only, self and root included
        assert m[n, 0] == 1 and m[n, n] == 1
    # the 6 candidates are all rank pairs (head-1 rank, head-2 rank)
    cands = sorted((t.rank[t.ancestors[l][1]], t.rank[t.ancestors[l][2]]) for l in t.leaves)
    assert cands == [(a, b) for a in range(2) for b in range(3)]
    # a drafted token at depth k comes from head k's list at the node's rank
    ids = [[11, 12], [21, 22, 23]]
    toks = ao.Oracle.tree_tokens(7, ids, t)
    assert toks[0] == 7
    assert sorted(tuple(toks[n] for n in t.ancestors[l]) for l in t.leaves) == \
        sorted((7, a, b) for a in ids[0] for b in ids[1])


def test_paper_shape_facts():
    g = _golden("paper_shapes.txt")
    s7 = inputs.get_shape("7b")
    assert s7.K == g["K"][0] and s7.n_nodes == g["tree_nodes"][0]
    specs = {n: shp for n, shp, _ in inputs.weight_specs(s7)}
    assert math.prod(specs["draft.lm_head.0"]) == g["lm_head_params_7b"][0]
    assert specs["draft.pe"] == (s7.K, s7.d_model)
    assert specs["draft.mlp.0.w"] == (s7.d_model, s7.d_model)
    topo = inputs.make_tree(s7.n_nodes, s7.topk)
    assert topo.n_nodes == g["tree_nodes"][0] and topo.max_depth == g["tree_depth"][0]


def test_head_stage_split():
    """Eq. 2: heads 1..floor(K/2) depend on stage 1 only, the others on stage 2."""
    g = _golden("paper_shapes.txt")
    orc = _oracle(MICRO, std=0.2)
    prompt = inputs.make_prompt(MICRO).tolist()
    st = orc.prefill(prompt)
    taps = {}
    orc.draft(st, taps)
    base = taps["Hp"] - orc.W("draft.pe")
    # recompute from the taps with an independent formula and perturb one stage at a time
    for k in range(1, MICRO.K + 1):
        src = taps["h1"] if k in g["stage1_heads_K4"] else taps["h2"]
        w, b = orc.W(f"draft.mlp.{k-1}.w"), orc.W(f"draft.mlp.{k-1}.b")
        ref = src + torch.nn.functional.silu(w @ src + b)
        assert torch.allclose(base[k - 1], ref, atol=1e-12)
    assert not torch.allclose(taps["h1"], taps["h2"])


# --------------------------------------------------------------------------------------
# primitives against library routines and closed forms
# --------------------------------------------------------------------------------------
def test_primitives_against_library():
    torch.manual_seed(0)
    x = torch.randn(5, 48, dtype=torch.float64)
    g = torch.randn(48, dtype=torch.float64)
    assert torch.allclose(ao.rmsnorm(x, g, 1e-6), torch.nn.functional.rms_norm(x, (48,), g, 1e-6), atol=1e-12)
    assert torch.allclose(ao.rmsnorm(3.7 * x, g, 0.0), ao.rmsnorm(x, g, 0.0), atol=1e-12)   # scale invariance
    assert torch.allclose(ao.silu(x), torch.nn.functional.silu(x), atol=1e-12)
    H, dh, S = 3, 16, 7
    q = torch.randn(H * dh, dtype=torch.float64)
    k = torch.randn(S, H * dh, dtype=torch.float64)
    v = torch.randn(S, H * dh, dtype=torch.float64)
    ref = torch.nn.functional.scaled_dot_product_attention(
        q.view(1, H, 1, dh), k.view(1, S, H, dh).transpose(1, 2), v.view(1, S, H, dh).transpose(1, 2))
    assert torch.allclose(ao.attend(q, k, v, H, dh), ref.reshape(-1), atol=1e-12)
    assert ao.argmax_lowest(torch.tensor([1.0, 5.0, 5.0, 2.0])) == 1
    ids, vals = ao.topk_desc(torch.tensor([1.0, 5.0, 5.0, 2.0, 7.0]), 3)
    assert ids == [4, 1, 2] and vals == [7.0, 5.0, 5.0]
    big = torch.randn(5000, dtype=torch.float64)
    big[100] = big[4000] = 9.0
    ids, _ = ao.topk_desc(big, 3)
    assert ids[:2] == [100, 4000]


def test_rope_is_complex_rotation_and_relative():
    torch.manual_seed(1)
    H, dh, theta = 2, 16, 10000.0
    x = torch.randn(H * dh, dtype=torch.float64)
    for pos in (0, 1, 17, 513):
        y = ao.rope(x, pos, H, dh, theta).view(H, dh)
        xh = x.view(H, dh)
        z = torch.complex(xh[:, : dh // 2], xh[:, dh // 2:])
        w = torch.tensor([theta ** (-2.0 * i / dh) for i in range(dh // 2)], dtype=torch.float64)
        r = z * torch.polar(torch.ones_like(w), pos * w)
        assert torch.allclose(y[:, : dh // 2], r.real, atol=1e-12)
        assert torch.allclose(y[:, dh // 2:], r.imag, atol=1e-12)
    assert torch.equal(ao.rope(x, 0, H, dh, theta), x)
    q, k = torch.randn(H * dh, dtype=torch.float64), torch.randn(H * dh, dtype=torch.float64)
    d0 = ao.rope(q, 9, H, dh, theta) @ ao.rope(k, 4, H, dh, theta)
    d1 = ao.rope(q, 109, H, dh, theta) @ ao.rope(k, 104, H, dh, theta)
    assert abs(float(d0 - d1)) < 1e-10                      # depends on the offset only


def test_single_key_attention_ignores_query():
    """With an empty cache and one row, attention returns Wo Wv RMSNorm(x): no dependence on
    Wq, Wk, RoPE or the position (softmax over one key is 1)."""
    orc = _oracle(MICRO, std=0.2)
    x = inputs.normal_tensor((1, MICRO.d_model), 1.0, 5, "x", dtype=torch.float64)
    outs = []
    for pos in (0, 7):
        cache = ao.LayerCache()
        outs.append(orc.decoder_rows("layers.0.", x, [pos], [0], [[0]], cache))
    assert torch.allclose(outs[0], outs[1], atol=1e-12)
    xn = ao.rmsnorm(x[0], orc.W("layers.0.attn_norm"), MICRO.rms_eps)
    x1 = x[0] + orc.W("layers.0.wo") @ (orc.W("layers.0.wv") @ xn)
    xn2 = ao.rmsnorm(x1, orc.W("layers.0.ffn_norm"), MICRO.rms_eps)
    ffn = orc.W("layers.0.w_down") @ (torch.nn.functional.silu(orc.W("layers.0.w_gate") @ xn2)
                                      * (orc.W("layers.0.w_up") @ xn2))
    assert torch.allclose(outs[0][0], x1 + ffn, atol=1e-12)


def test_target_forward_matches_hf_llama():
    """The target is a Vicuna (= Llama architecture) model: the oracle's causal forward must
    equal the transformers library's LlamaForCausalLM on the same weights."""
    tr = pytest.importorskip("transformers")
    s = MICRO
    orc = _oracle(s, std=0.2)
    cfg = tr.LlamaConfig(vocab_size=s.vocab, hidden_size=s.d_model, intermediate_size=s.d_ffn,
                         num_hidden_layers=s.n_layers, num_attention_heads=s.n_heads,
                         num_key_value_heads=s.n_heads, head_dim=s.head_dim, rms_norm_eps=s.rms_eps,
                         rope_theta=s.rope_theta, max_position_embeddings=256, attention_bias=False,
                         mlp_bias=False, tie_word_embeddings=False, hidden_act="silu")
    try:
        model = tr.LlamaForCausalLM(cfg).to(torch.float64).eval()
    except Exception as e:          # pragma: no cover - library drift
        pytest.skip(f"transformers could not build the model: {e}")
    sd = {"model.embed_tokens.weight": orc.W("tok_emb"), "model.norm.weight": orc.W("final_norm"),
          "lm_head.weight": orc.W("lm_head")}
    m = {"attn_norm": "input_layernorm", "wq": "self_attn.q_proj", "wk": "self_attn.k_proj",
         "wv": "self_attn.v_proj", "wo": "self_attn.o_proj", "ffn_norm": "post_attention_layernorm",
         "w_gate": "mlp.gate_proj", "w_up": "mlp.up_proj", "w_down": "mlp.down_proj"}
    for l in range(s.n_layers):
        for a, b in m.items():
            sd[f"model.layers.{l}.{b}.weight"] = orc.W(f"layers.{l}.{a}")
    missing = model.load_state_dict(sd, strict=False)
    assert not [k for k in missing.missing_keys if "rotary" not in k and "inv_freq" not in k]
    prompt = inputs.make_prompt(s).tolist()
    with torch.no_grad():
        ref = model(torch.tensor([prompt])).logits[0].to(torch.float64)
    n = len(prompt)
    kv = [ao.LayerCache() for _ in range(s.n_layers)]
    _, logits = orc.target_rows(prompt, list(range(n)), list(range(n)),
                                [list(range(j + 1)) for j in range(n)], kv)
    assert float((logits - ref).abs().max()) < 1e-6 * max(1.0, float(ref.abs().max()))


# --------------------------------------------------------------------------------------
# tree verification == per-path causal decoding; chain == prefill
# --------------------------------------------------------------------------------------
@pytest.mark.parametrize("topo", [inputs.full_tree([2, 3]), inputs.make_tree(16, [4, 2, 2, 1]),
                                  inputs.full_tree([2, 1, 2, 1])], ids=["fig5", "tiny16", "depth4"])
def test_tree_mask_equals_per_path_causal(topo):
    orc = _oracle(MICRO, std=0.2)
    t = _tables(topo)
    st = orc.prefill(inputs.make_prompt(MICRO).tolist())
    toks = [st.root] + inputs.uniform_ids(t.n_nodes - 1, MICRO.vocab, 3, "treetoks").tolist()
    brute = orc.verify_paths_bruteforce(st, toks, t)
    _, logits, _ = orc.verify(st, toks, t)
    assert float((logits - brute).abs().max()) < 1e-10


def test_chain_tree_equals_causal_forward_and_incremental_prefill():
    orc = _oracle(MICRO, std=0.2)
    prompt = inputs.make_prompt(MICRO, n=12).tolist()
    n0 = 7
    st = orc.prefill(prompt[:n0])
    t = _tables(inputs.chain_tree(len(prompt) - n0))
    _, logits_chain, _ = orc.verify(st, prompt[n0:], t)
    full = orc.prefill(prompt)
    kv = [ao.LayerCache() for _ in range(MICRO.n_layers)]
    n = len(prompt)
    _, logits_full = orc.target_rows(prompt, list(range(n)), list(range(n)),
                                     [list(range(j + 1)) for j in range(n)], kv)
    assert float((logits_chain - logits_full[n0:]).abs().max()) < 1e-10
    # token-by-token prefill fills the same cache
    kv1 = [ao.LayerCache() for _ in range(MICRO.n_layers)]
    for j in range(n):
        orc.target_rows([prompt[j]], [j], [j], [list(range(j + 1))], kv1)
    for l in range(MICRO.n_layers):
        for j in range(n):
            assert torch.allclose(kv1[l].k[j], full.kv[l].k[j], atol=1e-10)
            assert torch.allclose(kv1[l].v[j], full.kv[l].v[j], atol=1e-10)


# --------------------------------------------------------------------------------------
# Auto-embedding Block: bi-directional => permutation equivariant
# --------------------------------------------------------------------------------------
def test_aeb_permutation_equivariance_and_bidirectionality():
    orc = _oracle(MICRO, std=0.2)
    Hp = inputs.normal_tensor((MICRO.K, MICRO.d_model), 1.0, 9, "Hp", dtype=torch.float64)
    base = orc.aeb(Hp)
    for perm in itertools.permutations(range(MICRO.K)):
        p = list(perm)
        assert torch.allclose(orc.aeb(Hp[p]), base[p], atol=1e-10)
    # every row depends on every other row (earlier heads see later ones and vice versa)
    for j in range(MICRO.K):
        Hq = Hp.clone()
        Hq[j] += 1.0
        diff = (orc.aeb(Hq) - base).abs().amax(dim=1)
        assert bool((diff > 1e-8).all())


# --------------------------------------------------------------------------------------
# acceptance and compaction: exhaustive on small trees
# --------------------------------------------------------------------------------------
def _naive_accept(toks, amax, t):
    best_path = [0]
    for n in range(t.n_nodes):          # every node ends a candidate prefix
        path = t.ancestors[n]
        good = True
        for i in range(1, len(path)):
            if toks[path[i]] != amax[path[i - 1]]:
                good = False
                break
        if good and len(path) > len(best_path):
            best_path = path
    return best_path


@pytest.mark.parametrize("topo", [inputs.full_tree([2, 3]), inputs.make_tree(12, [3, 2, 2, 1]),
                                  inputs.full_tree([2, 1, 2, 1])])
def test_accept_exhaustive(topo):
    t = _tables(topo)
    N = t.n_nodes
    # distinct tokens per node; amax[p] chosen to hit one child, or none
    toks = [100 + n for n in range(N)]
    children = [[c for c in range(1, N) if t.parent[c] == p] for p in range(N)]
    choices = [[-1] + children[p] for p in range(N)]
    count = 0
    for pick in itertools.product(*choices):
        amax = [toks[c] if c >= 0 else 999 for c in pick]
        L, path, emitted, nxt = ao.Oracle.accept(toks, amax, t)
        ref = _naive_accept(toks, amax, t)
        assert path == ref and L == len(ref)
        assert emitted == [toks[n] for n in ref] and nxt == amax[ref[-1]]
        # the emitted tokens continue greedily: token j+1 is the target's choice after token j
        for j in range(L - 1):
            assert emitted[j + 1] == amax[path[j]]
        count += 1
        if count > 20000:
            break


def test_commit_moves_tagged_rows():
    t = _tables(inputs.make_tree(12, [3, 2, 2, 1]))
    orc = _oracle(MICRO)
    C = 5
    for leaf in range(t.n_nodes):
        path = t.ancestors[leaf]
        kv = [ao.LayerCache() for _ in range(2)]
        for cache in kv:
            for s in range(C + t.n_nodes):
                cache.put(s, torch.tensor([float(s)]), torch.tensor([float(-s)]))
        st = ao.State(C, 1, kv, [], [])
        hid = torch.arange(t.n_nodes, dtype=torch.float64).view(-1, 1)
        toks = [50 + n for n in range(t.n_nodes)]
        moves = orc.commit(st, toks, hid, path, 77, t)
        assert st.C == C + len(path) and st.root == 77
        for cache in st.kv:
            assert len(cache.k) == st.C
            for j, n in enumerate(path):
                assert float(cache.k[C + j]) == C + n and float(cache.v[C + j]) == -(C + n)
            for s in range(C):
                assert float(cache.k[s]) == s
        assert moves == [(C + j, C + n) for j, n in enumerate(path) if n != j]
        assert [p for (_, _, p) in st.pending] == [C + j for j in range(len(path))]
        assert [int(h) for (h, _, _) in st.pending] == path
        assert [nx for (_, nx, _) in st.pending] == [toks[n] for n in path[1:]] + [77]


# --------------------------------------------------------------------------------------
# losslessness: speculative output == greedy autoregressive output
# --------------------------------------------------------------------------------------
def _plant(t, st_root, future, leaf):
    """Override tokens so that the path to `leaf` carries the true continuation."""
    ov = [-1] * t.n_nodes
    for i, n in enumerate(t.ancestors[leaf]):
        if i > 0:
            ov[n] = future[i - 1]
    return ov


@pytest.mark.parametrize("shape,planted", [(MICRO, False), (MICRO, True), (TINY, True)],
                         ids=["micro-natural", "micro-planted", "tiny-planted"])
def test_lossless_vs_greedy_ar(shape, planted):
    orc = _oracle(shape, std=0.2 if shape is MICRO else 0.02)
    prompt = inputs.make_prompt(shape).tolist()
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    t = _tables(topo)
    steps = shape.steps
    ref = orc.greedy_ar(prompt, steps * (shape.K + 1) + 1)
    st = orc.prefill(prompt)
    out = []
    lens = []
    for i in range(steps):
        ov = None
        if planted:
            leaf = t.leaves[i % len(t.leaves)]
            future = ref[len(out) + 1: len(out) + 1 + t.depth[leaf]]
            ov = _plant(t, st.root, future, leaf)
        taps = {}
        emitted = orc.step(st, t, ov, taps)
        assert emitted[0] == ref[len(out)]
        out += emitted
        lens.append(len(emitted))
        assert st.C == len(prompt) + len(out)
        assert all(len(c.k) == st.C for c in st.kv)
        # the adaptation layers have seen every position committed before this step exactly once
        assert all(len(c.k) == taps["C_before"] for c in st.sal_kv)
        assert len(st.pending) == len(emitted)
    assert out == ref[: len(out)]
    assert st.root == ref[len(out)]
    if planted:
        assert max(lens) >= 3                                  # real multi-token acceptance happened
        # the committed cache equals the cache of a plain causal forward of the same tokens
        seq = prompt + out
        full = orc.prefill(seq)
        for l in range(shape.n_layers):
            for s in range(len(seq)):
                assert torch.allclose(st.kv[l].k[s], full.kv[l].k[s], atol=1e-9)
                assert torch.allclose(st.kv[l].v[s], full.kv[l].v[s], atol=1e-9)


def test_sal_cache_equals_one_shot():
    """Feeding the adaptation layers the accepted rows step by step gives the same stage
    caches as feeding all positions at once (each position enters exactly once, causally)."""
    shape = MICRO
    orc = _oracle(shape, std=0.2)
    prompt = inputs.make_prompt(shape).tolist()
    t = _tables(inputs.make_tree(shape.n_nodes, shape.topk))
    ref = orc.greedy_ar(prompt, 40)
    st = orc.prefill(prompt)
    out = []
    for i in range(4):
        leaf = t.leaves[(2 * i + 1) % len(t.leaves)]
        ov = _plant(t, st.root, ref[len(out) + 1: len(out) + 1 + t.depth[leaf]], leaf)
        out += orc.step(st, t, ov)
    orc.draft(st)                                              # flush the last pending rows
    seq = prompt + out
    st2 = orc.prefill(seq)
    orc.draft(st2)
    for a, b in zip(st.sal_kv, st2.sal_kv):
        assert len(a.k) == len(b.k) == len(seq)
        for s in range(len(seq)):
            assert torch.allclose(a.k[s], b.k[s], atol=1e-9) and torch.allclose(a.v[s], b.v[s], atol=1e-9)


def test_storage_rounding_mode_is_identity_without_rounding_and_small_with_bf16():
    """storage=float64 rounds nothing: bit-identical to the plain oracle.  bf16 storage perturbs the
    logits only at the bf16 level (it never changes the structure of the computation)."""
    shape = MICRO
    w = inputs.make_weights(shape, seed=0, std=0.2)
    prompt = inputs.make_prompt(shape).tolist()
    t = _tables(inputs.make_tree(shape.n_nodes, shape.topk))
    outs = []
    for storage in (None, torch.float64, torch.bfloat16):
        orc = ao.Oracle(shape, w, dtype=torch.float64, storage=storage)
        st = orc.prefill(prompt)
        taps = {}
        orc.step(st, t, None, taps)
        outs.append((st.last_logits, taps["logits"], taps["d_logits"]))
    for a, b in zip(outs[0], outs[1]):
        assert torch.equal(a, b)
    for a, c in zip(outs[0], outs[2]):
        err = float((a - c).abs().max()) / max(1.0, float(a.abs().max()))
        assert 0.0 < err < 3e-2


# --------------------------------------------------------------------------------------
# draft-module variants (Section 4.5 "One-Adaptation-Layer", Appendix A.2.3 "Amphista-alpha")
# --------------------------------------------------------------------------------------
def test_variant_one_adaptation_layer_feeds_every_head_from_stage_one():
    """With a single adaptation layer every head reads h1 (Section 4.5): the variant's stage-1 output
    equals the two-stage model's (same weights, same inputs), and each head row is the Eq. 2 form of it."""
    two = _oracle(MICRO, std=0.2)
    one_shape = MICRO.with_(n_sal=1)
    one = ao.Oracle(one_shape, inputs.make_weights(MICRO, seed=0, std=0.2), dtype=torch.float64)
    prompt = inputs.make_prompt(MICRO).tolist()
    t2, t1 = {}, {}
    two.draft(two.prefill(prompt), t2)
    st = one.prefill(prompt)
    one.draft(st, t1)
    assert len(st.sal_kv) == 1
    assert torch.allclose(t1["h1"], t2["h1"], atol=1e-12)
    base = t1["Hp"] - one.W("draft.pe")
    for k in range(MICRO.K):
        w, b = one.W(f"draft.mlp.{k}.w"), one.W(f"draft.mlp.{k}.b")
        assert torch.allclose(base[k], t1["h1"] + torch.nn.functional.silu(w @ t1["h1"] + b), atol=1e-12)
    # heads of the second half differ from the two-stage model (there they read h2), the first half does not
    b2 = t2["Hp"] - two.W("draft.pe")
    assert torch.allclose(base[: MICRO.K // 2], b2[: MICRO.K // 2], atol=1e-12)
    assert not torch.allclose(base[MICRO.K // 2:], b2[MICRO.K // 2:], atol=1e-6)


def test_variant_two_aeb_layers_is_composition_and_reduces_to_one():
    """Amphista-alpha stacks two self-attention layers (Appendix A.2.3): the block is the composition of the
    two layers, stays permutation equivariant, and with a zero output projection in the second layer the
    residual makes it equal to the one-layer block."""
    shape = MICRO.with_(aeb_layers=2)
    w = inputs.make_weights(shape, seed=0, std=0.2)
    orc = ao.Oracle(shape, w, dtype=torch.float64)
    prompt = inputs.make_prompt(shape).tolist()
    taps = {}
    orc.draft(orc.prefill(prompt), taps)
    assert torch.allclose(taps["attn_o"], orc.aeb(orc.aeb(taps["Hp"], 0), 1), atol=1e-12)
    assert not torch.allclose(taps["attn_o"], orc.aeb(taps["Hp"], 0), atol=1e-6)
    Hp = inputs.normal_tensor((shape.K, shape.d_model), 1.0, 9, "Hp", dtype=torch.float64)
    two = lambda X: orc.aeb(orc.aeb(X, 0), 1)
    p = [2, 0, 3, 1]
    assert torch.allclose(two(Hp[p]), two(Hp)[p], atol=1e-10)
    w0 = dict(w)
    w0["draft.aeb.1.wo"] = torch.zeros_like(w["draft.aeb.1.wo"])
    orc0 = ao.Oracle(shape, w0, dtype=torch.float64)
    t0 = {}
    orc0.draft(orc0.prefill(prompt), t0)
    assert torch.allclose(t0["attn_o"], orc0.aeb(t0["Hp"], 0), atol=1e-12)


@pytest.mark.parametrize("variant", [dict(n_sal=1), dict(aeb_layers=2)], ids=["one-sal", "two-aeb-layers"])
def test_variants_stay_lossless(variant):
    shape = MICRO.with_(**variant)
    orc = ao.Oracle(shape, inputs.make_weights(shape, seed=0, std=0.2), dtype=torch.float64)
    prompt = inputs.make_prompt(shape).tolist()
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    t = _tables(topo)
    ref = orc.greedy_ar(prompt, 4 * (shape.K + 1) + 1)
    st = orc.prefill(prompt)
    out = []
    for i in range(4):
        leaf = t.leaves[i % len(t.leaves)]
        emitted = orc.step(st, t, _plant(t, st.root, ref[len(out) + 1: len(out) + 1 + t.depth[leaf]], leaf), {})
        out += emitted
    assert out == ref[: len(out)] and st.root == ref[len(out)]


def test_variant_low_rank_lm_heads_equal_the_product_matrix():
    """Appendix A.2.4 replaces each head's [V, d] matrix by two low-rank factors: the draft logits must be
    those of a full head whose matrix is the product B.A, and the factors hold (V + d) r parameters each."""
    r = 8
    shape = MICRO.with_(lm_rank=r)
    w = inputs.make_weights(shape, seed=0, std=0.2)
    specs = {n: shp for n, shp, _ in inputs.weight_specs(shape)}
    assert specs["draft.lm_head.0.a"] == (r, MICRO.d_model) and specs["draft.lm_head.0.b"] == (MICRO.vocab, r)
    assert "draft.lm_head.0" not in specs
    full = {k: v for k, v in w.items() if ".lm_head." not in k or k == "lm_head"}
    for k in range(MICRO.K):
        full[f"draft.lm_head.{k}"] = (w[f"draft.lm_head.{k}.b"].double() @ w[f"draft.lm_head.{k}.a"].double())
    lo = ao.Oracle(shape, w, dtype=torch.float64)
    hi = ao.Oracle(MICRO, full, dtype=torch.float64)
    prompt = inputs.make_prompt(MICRO).tolist()
    ids_l, vals_l, dl_l = lo.draft(lo.prefill(prompt))
    ids_h, vals_h, dl_h = hi.draft(hi.prefill(prompt))
    assert torch.allclose(dl_l, dl_h, atol=1e-10)
    assert [list(map(int, i)) for i in ids_l] == [list(map(int, i)) for i in ids_h]
    assert torch.linalg.matrix_rank(full["draft.lm_head.0"]).item() == r


def test_variant_without_adaptation_layers_or_auto_embedding():
    """Section 4.5's ablations that remove a module.  Without adaptation layers every head's MLP reads the target's
    last hidden state (the row the target's own head consumed) and the sampled token plays no part; without the
    Auto-embedding Block the head rows go to their vocabulary projections unchanged."""
    prompt = inputs.make_prompt(MICRO).tolist()
    # -- no adaptation layers
    s0 = MICRO.with_(n_sal=0)
    o0 = ao.Oracle(s0, inputs.make_weights(s0, seed=0, std=0.2), dtype=torch.float64)
    assert not any(n.startswith("draft.sal") or n.startswith("draft.fc") for n, _, _ in inputs.weight_specs(s0))
    st = o0.prefill(prompt)
    h_t = st.pending[-1][0].clone()
    assert torch.allclose(o0.W("lm_head") @ h_t, st.last_logits, atol=1e-10)      # it is the row the target head consumed
    taps = {}
    o0.draft(st, taps)
    base = taps["Hp"] - o0.W("draft.pe")
    for k in range(MICRO.K):
        w, b = o0.W(f"draft.mlp.{k}.w"), o0.W(f"draft.mlp.{k}.b")
        assert torch.allclose(base[k], h_t + torch.nn.functional.silu(w @ h_t + b), atol=1e-12)
    st2 = o0.prefill(prompt)                       # the sampled token is unused: change it, nothing moves
    st2.pending = [(h, (nxt + 1) % MICRO.vocab, p) for (h, nxt, p) in st2.pending]
    t2 = {}
    o0.draft(st2, t2)
    assert torch.equal(t2["Hp"], taps["Hp"])
    # -- no Auto-embedding Block
    s1 = MICRO.with_(aeb_layers=0)
    o1 = ao.Oracle(s1, inputs.make_weights(s1, seed=0, std=0.2), dtype=torch.float64)
    assert not any(n.startswith("draft.aeb") for n, _, _ in inputs.weight_specs(s1))
    t1 = {}
    _, _, dl = o1.draft(o1.prefill(prompt), t1)
    assert torch.equal(t1["attn_o"], t1["Hp"])
    for k in range(MICRO.K):
        assert torch.allclose(dl[k], o1.W(f"draft.lm_head.{k}") @ t1["Hp"][k], atol=1e-12)
    # a head's logits then depend on its own row only (no exchange between the heads)
    two = ao.Oracle(MICRO, inputs.make_weights(MICRO, seed=0, std=0.2), dtype=torch.float64)
    Hp = inputs.normal_tensor((MICRO.K, MICRO.d_model), 1.0, 9, "Hp", dtype=torch.float64)
    Hq = Hp.clone(); Hq[0] += 1.0
    assert bool(((two.aeb(Hq) - two.aeb(Hp)).abs().amax(dim=1)[1:] > 1e-8).all())   # with the block, rows do interact


def test_variant_without_sampled_token():
    """Section 4.5, "w/o Sampled-Token": fc is d -> d on the hidden state alone, so nothing in the draft module depends
    on the token sampled from h_t; and it equals the full model whose fc has its embedding columns zeroed."""
    prompt = inputs.make_prompt(MICRO).tolist()
    d = MICRO.d_model
    s0 = MICRO.with_(use_sampled_token=False)
    specs = {n: shp for n, shp, _ in inputs.weight_specs(s0)}
    assert specs["draft.fc1"] == (d, d) and specs["draft.fc2"] == (d, d)
    w0 = inputs.make_weights(s0, seed=0, std=0.2)
    o0 = ao.Oracle(s0, w0, dtype=torch.float64)
    st = o0.prefill(prompt)
    t0 = {}
    _, _, dl0 = o0.draft(st, t0)
    st2 = o0.prefill(prompt)
    st2.pending = [(h, (nxt + 5) % MICRO.vocab, p) for (h, nxt, p) in st2.pending]
    _, _, dl2 = o0.draft(st2, {})
    assert torch.equal(dl0, dl2)
    wf = dict(w0)                                   # the full form with zero embedding columns computes the same thing
    for sname in ("draft.fc1", "draft.fc2"):
        wf[sname] = torch.cat([w0[sname], torch.zeros(d, d)], dim=1)
    of = ao.Oracle(MICRO, wf, dtype=torch.float64)
    _, _, dlf = of.draft(of.prefill(prompt), {})
    assert torch.allclose(dl0, dlf, atol=1e-12)


@pytest.mark.parametrize("variant", [dict(n_sal=0), dict(aeb_layers=0), dict(use_sampled_token=False)],
                         ids=["no-sal", "no-aeb", "no-sampled-token"])
def test_ablations_stay_lossless(variant):
    shape = MICRO.with_(**variant)
    orc = ao.Oracle(shape, inputs.make_weights(shape, seed=0, std=0.2), dtype=torch.float64)
    prompt = inputs.make_prompt(shape).tolist()
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    t = _tables(topo)
    ref = orc.greedy_ar(prompt, 4 * (shape.K + 1) + 1)
    st = orc.prefill(prompt)
    out = []
    for i in range(4):
        leaf = t.leaves[i % len(t.leaves)]
        out += orc.step(st, t, _plant(t, st.root, ref[len(out) + 1: len(out) + 1 + t.depth[leaf]], leaf), {})
    assert out == ref[: len(out)] and st.root == ref[len(out)]


# --------------------------------------------------------------------------------------
# Eq. 1: what the adaptation layers are fed
# --------------------------------------------------------------------------------------
def _draft_with(shape, w, pending_mod=None, prompt=None):
    """Prefill + draft on a copy of the state; returns (h1 of the last row, stage-1 cache, stage-2 cache)."""
    orc = ao.Oracle(shape, w, dtype=torch.float64)
    st = orc.prefill(prompt)
    if pending_mod is not None:
        st.pending = pending_mod(list(st.pending))
    taps = {}
    orc.draft(st, taps)
    return taps["h1"], st.sal_kv[0], st.sal_kv[-1]


def test_eq1_input_is_hidden_then_embedding():
    """Eq. 1 feeds fc the concatenation [h_t ; e_{t+1}] in that order.  With the embedding half of fc1's columns
    zeroed the stage output cannot depend on the sampled token (but does on h_t); with the hidden half zeroed it
    cannot depend on h_t (but does on the token).  A swapped concatenation, or an embedding that is ignored,
    fails one of the four assertions."""
    shape = MICRO
    d = shape.d_model
    prompt = inputs.make_prompt(shape).tolist()
    base = inputs.make_weights(shape, seed=0, std=0.2)
    other_tok = lambda p: p[:-1] + [(p[-1][0], (p[-1][1] + 7) % shape.vocab, p[-1][2])]
    other_hid = lambda p: p[:-1] + [(p[-1][0] * 1.5 + 0.25, p[-1][1], p[-1][2])]

    w = dict(base)
    w["draft.fc1"] = base["draft.fc1"].clone()
    w["draft.fc1"][:, d:] = 0                                   # no embedding columns
    h_ref, _, _ = _draft_with(shape, w, None, prompt)
    h_tok, _, _ = _draft_with(shape, w, other_tok, prompt)
    h_hid, _, _ = _draft_with(shape, w, other_hid, prompt)
    assert torch.equal(h_ref, h_tok)
    assert float((h_ref - h_hid).abs().max()) > 1e-3

    w = dict(base)
    w["draft.fc1"] = base["draft.fc1"].clone()
    w["draft.fc1"][:, :d] = 0                                   # no hidden-state columns
    h_ref, _, _ = _draft_with(shape, w, None, prompt)
    h_tok, _, _ = _draft_with(shape, w, other_tok, prompt)
    h_hid, _, _ = _draft_with(shape, w, other_hid, prompt)
    assert torch.equal(h_ref, h_hid)
    assert float((h_ref - h_tok).abs().max()) > 1e-3


def test_eq1_embedding_is_that_of_the_next_token():
    """e_{t+1} is the embedding row of the token that follows position t.  With the adaptation layer reduced to
    its residual path (zero output and down projections) and fc1 = [0 | I], h^1 of a row IS that embedding row."""
    shape = MICRO
    d = shape.d_model
    prompt = inputs.make_prompt(shape).tolist()
    w = inputs.make_weights(shape, seed=0, std=0.2)
    w["draft.fc1"] = torch.cat([torch.zeros(d, d), torch.eye(d)], dim=1)
    w["draft.sal1.wo"] = torch.zeros(d, d)
    w["draft.sal1.w_down"] = torch.zeros(d, shape.d_ffn)
    orc = ao.Oracle(shape, w, dtype=torch.float64)
    st = orc.prefill(prompt)
    root = st.root
    taps = {}
    orc.draft(st, taps)
    assert torch.allclose(taps["h1"], w["tok_emb"][root].to(torch.float64), atol=1e-12)
    # and with fc1 = [I | 0] it is the target's hidden state of the last prompt position
    w["draft.fc1"] = torch.cat([torch.eye(d), torch.zeros(d, d)], dim=1)
    orc = ao.Oracle(shape, w, dtype=torch.float64)
    st = orc.prefill(prompt)
    h_last = st.pending[-1][0].clone()
    taps = {}
    orc.draft(st, taps)
    assert torch.allclose(taps["h1"], h_last, atol=1e-12)


def test_eq1_adaptation_layers_are_causal_over_the_pending_rows():
    """kv_{1:t-1} in Eq. 1: a row of an adaptation layer sees earlier positions only.  Changing the next-token of
    pending row j changes the cache rows of positions >= j in both stages and leaves every earlier row bit-identical."""
    shape = MICRO
    prompt = inputs.make_prompt(shape).tolist()
    w = inputs.make_weights(shape, seed=0, std=0.2)
    j = 4

    def mod(p):
        p[j] = (p[j][0], (p[j][1] + 11) % shape.vocab, p[j][2])
        return p
    _, c1, c2 = _draft_with(shape, w, None, prompt)
    _, m1, m2 = _draft_with(shape, w, mod, prompt)
    for a, b, stage in ((c1, m1, 1), (c2, m2, 2)):
        for s in range(len(prompt)):
            same = torch.equal(a.k[s], b.k[s]) and torch.equal(a.v[s], b.v[s])
            if s < j:
                assert same, f"stage {stage}: position {s} < {j} changed"
            elif s == j or stage == 2:
                assert not same, f"stage {stage}: position {s} did not react"
