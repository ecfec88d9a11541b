"""GPU parity of decoding at a sampling temperature (Table 2) against the sampling oracle.

Both sides get the same uniforms (a counter-based generator implemented on each side from its published definition;
the test checks them equal bit for bit) and the same logits (the oracle draws from the logits the GPU produced, read
back as float32), so every decision must agree except where the uniform lies within the floating-point error of a
decision boundary; such nodes are counted, and there the GPU's choice must still be one of the two tokens that meet at
that boundary.  The logits themselves are compared with the oracle's own as in every other parity test.
"""
import pytest
import torch

import inputs
from oracle import amphista_oracle as ao
from oracle import amphista_sampling as sm
from tests.parity import plant, rel_err

pytestmark = pytest.mark.gpu

SEED = 0x1234_5678_9ABC_DEF0
MARGIN = 2e-6            # float32 running sums of up to 2048 weights against float64 ones


def _check_choices(g_choice, toks, logits64, t, T, u, stats):
    margins = []
    want = sm.choices_flat(toks, logits64, t, T, u, margins)
    for n in range(t.n_nodes):
        if margins[n] > MARGIN:
            assert g_choice[n] == want[n], f"node {n}: gpu drew {g_choice[n]}, oracle {want[n]} (margin {margins[n]:.3g})"
        else:
            stats["near_boundary"] += 1
            lo = sm.choice_flat(toks, logits64[n], sm.children_of(t, n), T, max(0.0, u[n] - 2 * MARGIN))
            hi = sm.choice_flat(toks, logits64[n], sm.children_of(t, n), T, min(1.0 - 2 ** -25, u[n] + 2 * MARGIN))
            kids = {int(toks[c]) for c in sm.children_of(t, n)}
            if lo in kids or hi in kids:
                assert g_choice[n] in (lo, hi, want[n])
            else:              # a residual draw: the other ids are walked in ascending order, narrow ones may lie in between
                assert lo <= g_choice[n] <= hi and g_choice[n] not in kids
    stats["nodes"] += t.n_nodes


@pytest.mark.parametrize("base,T,planted", [("tiny", 0.7, False), ("tiny", 0.02, True), ("small_bf16", 0.7, False),
                                            ("small_bf16", 0.02, True)],
                         ids=["fp32-T0.7", "fp32-T0.02-planted", "bf16-T0.7", "bf16-T0.02-planted"])
def test_sampled_steps_match_the_oracle(base, T, planted):
    from paper_2406_13170_b200 import Amphista
    shape = inputs.get_shape(base)
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    t = ao.tree_tables(topo.parent, topo.depth, topo.rank)
    N, K, V, d = t.n_nodes, shape.K, shape.vocab, shape.d_model
    bf = shape.dtype == "bf16"
    tol = 2e-2 if bf else 1e-5
    w_cpu = inputs.make_weights(shape, seed=0, init="fan_in")       # logits of a useful spread
    w_gpu = {k: v.to("cuda:0") for k, v in w_cpu.items()}
    model = Amphista(shape, topo, w_gpu, temperature=T, seed=SEED)
    orc = ao.Oracle(shape, w_cpu, dtype=torch.float64)
    prompt = inputs.make_prompt(shape).tolist()
    dev = model.device
    stats = {"near_boundary": 0, "nodes": 0}
    st = orc.prefill(prompt)
    g_root = model.prefill(prompt)
    last_row = (len(prompt) - 1) % 512
    g_last = model.get_tensor("logits", (last_row + 1, V))[last_row].cpu()
    assert rel_err(g_last, st.last_logits) <= tol
    # the token after the prompt: drawn from the GPU's own logits with stream 1 of the generator
    m = []
    want_root = sm.choice_flat([], g_last.to(torch.float64), [], T, sm.uniform(SEED, 0, 0, 0, stream=1), m)
    if m[0] > MARGIN:
        assert g_root == want_root
    sm.sample_root(st, T, SEED, 0, g_last.to(torch.float64))
    st.root = g_root
    st.pending[-1] = (st.pending[-1][0], g_root, st.pending[-1][2])
    g_amax = torch.zeros(N, dtype=torch.int32, device=dev)
    g_tok = torch.zeros(K + 1, dtype=torch.int32, device=dev)
    g_path = torch.zeros(K + 1, dtype=torch.int32, device=dev)
    g_n = torch.zeros(1, dtype=torch.int32, device=dev)
    g_next = torch.zeros(1, dtype=torch.int32, device=dev)
    accepted = []
    for step in range(6):
        ids, _, _ = orc.draft(st)
        toks = ao.Oracle.tree_tokens(st.root, ids, t)
        if planted:                 # the target's most likely continuation on one path: at a low temperature it is mostly accepted
            leaf = t.leaves[step % len(t.leaves)]
            cont = _greedy_continuation(orc, st, t.depth[leaf])
            ov = plant(t, cont, leaf)
            toks = [x if o < 0 else o for x, o in zip(toks, ov)]
            toks[0] = st.root
        hid, logits_o, _ = orc.verify(st, toks, t)
        model.draft()
        model.verify_tree(torch.tensor(toks, dtype=torch.int32, device=dev), g_amax)
        torch.cuda.synchronize(dev)
        g_logits = model.get_tensor("logits", (N, V)).cpu()
        assert rel_err(g_logits, logits_o) <= tol, f"step {step}: logits off by {rel_err(g_logits, logits_o)}"
        # same uniforms on both sides, bit for bit
        u = sm.node_uniforms(SEED, step, 0, N)
        g_u = model.get_tensor("uniforms", (N,)).cpu().tolist()
        assert g_u == u, f"step {step}: the generators disagree"
        g_choice = g_amax.tolist()
        _check_choices(g_choice, toks, g_logits.to(torch.float64), t, T, u, stats)
        # acceptance is integer logic on the choices; and the walk in rejection-sampling form agrees with it
        L, path, emitted, nxt = ao.Oracle.accept(toks, g_choice, t)
        mg = []
        sm.choices_flat(toks, g_logits.to(torch.float64), t, T, u, mg)
        if all(mg[n] > MARGIN for n in path):
            assert sm.accept_sampled(toks, g_logits.to(torch.float64), t, T, u) == (L, path, emitted, nxt)
        model.accept(g_tok, g_n, g_path, g_next)
        torch.cuda.synchronize(dev)
        assert int(g_n[0]) == L and g_path[:L].tolist() == path and g_tok[:L].tolist() == emitted and int(g_next[0]) == nxt
        orc.commit(st, toks, hid, path, nxt, t)
        assert model.get_state() == (st.C, st.root, L)
        accepted.append(L)
    print(stats, accepted)
    assert stats["near_boundary"] <= max(2, stats["nodes"] // 50)
    if planted:
        assert max(accepted) >= 3
    model.close()


def _greedy_continuation(orc, st, n):
    """The target's n most likely next tokens after the state's root (on copies of the caches)."""
    kv = [c.clone() for c in st.kv]
    out, tok, C = [], st.root, st.C
    for _ in range(n):
        _, logits = orc.target_rows([tok], [C], [C], [list(range(C + 1))], kv)
        tok = ao.argmax_lowest(logits[0])
        out.append(tok)
        C += 1
    return out


def test_replaced_logits_are_sampled_again_with_the_same_uniforms():
    """amph_set_tensor("logits"): the oracle's own logits go in, and the choices must be the oracle's draws from them."""
    from paper_2406_13170_b200 import Amphista
    shape = inputs.get_shape("tiny")
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    t = ao.tree_tables(topo.parent, topo.depth, topo.rank)
    N, V = t.n_nodes, shape.vocab
    w_cpu = inputs.make_weights(shape, seed=0, init="fan_in")
    model = Amphista(shape, topo, {k: v.to("cuda:0") for k, v in w_cpu.items()}, temperature=0.7, seed=7)
    model.prefill(inputs.make_prompt(shape).tolist())
    model.draft()
    model.verify_tree()
    toks = model.get_tensor("tree_tokens", (N,), torch.int32).tolist()
    torch.manual_seed(11)
    fake = (torch.randn(N, V) * 3.0).to(torch.float32)
    model.set_tensor("logits", fake.to("cuda:0"))
    g_choice = model.get_tensor("argmax", (N,), torch.int32).tolist()
    stats = {"near_boundary": 0, "nodes": 0}
    _check_choices(g_choice, toks, fake.to(torch.float64), t, 0.7, sm.node_uniforms(7, 0, 0, N), stats)
    assert stats["near_boundary"] <= 1
    model.close()


def test_free_running_sampled_steps_are_reproducible_and_seed_dependent():
    """amph_step at T = 0.7 (graph replay): the same seed gives the same tokens as the call-by-call path and as
    launches outside a graph; another seed gives other tokens."""
    from paper_2406_13170_b200 import Amphista
    shape = inputs.get_shape("tiny")
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    w = inputs.make_weights(shape, seed=0, init="fan_in")
    w_gpu = {k: v.to("cuda:0") for k, v in w.items()}
    prompt = inputs.make_prompt(shape).tolist()
    K = shape.K

    def run(seed, flags, stepwise):
        model = Amphista(shape, topo, w_gpu, temperature=0.7, seed=seed, flags=flags)
        out = [model.prefill(prompt)]
        tok = torch.zeros(K + 1, dtype=torch.int32, device="cuda:0")
        n = torch.zeros(1, dtype=torch.int32, device="cuda:0")
        for _ in range(6):
            if stepwise:
                model.draft(); model.verify_tree(); model.accept(tok, n)
            else:
                model.step(tok, n)
            torch.cuda.synchronize()
            out += tok[:int(n[0])].tolist()
        model.close()
        return out

    a = run(5, 0, False)
    assert a == run(5, 0, True) == run(5, 2, False)
    assert a != run(6, 0, False)


def test_low_temperature_is_greedy_on_the_gpu():
    from paper_2406_13170_b200 import Amphista
    shape = inputs.get_shape("tiny")
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    w = inputs.make_weights(shape, seed=0, init="fan_in")
    w_gpu = {k: v.to("cuda:0") for k, v in w.items()}
    prompt = inputs.make_prompt(shape).tolist()
    outs = []
    for T in (0.0, 1e-4):
        model = Amphista(shape, topo, w_gpu, temperature=T, seed=3)
        out = [model.prefill(prompt)]
        tok = torch.zeros(shape.K + 1, dtype=torch.int32, device="cuda:0")
        n = torch.zeros(1, dtype=torch.int32, device="cuda:0")
        for _ in range(6):
            model.step(tok, n)
            torch.cuda.synchronize()
            out += tok[:int(n[0])].tolist()
        outs.append(out)
        model.close()
    assert outs[0] == outs[1]


def test_sampling_in_a_batch_uses_one_generator_stream_per_sequence():
    """Two sequences with the SAME prompt at T = 0.7: sequence 0 draws what a single-sequence context with that seed
    draws (its uniforms are keyed by sequence index 0), sequence 1 has uniforms of its own and soon emits other tokens;
    the uniforms tap of each sequence equals the oracle's generator for that sequence index."""
    from paper_2406_13170_b200 import Amphista
    shape = inputs.get_shape("tiny")
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    w = inputs.make_weights(shape, seed=0, init="fan_in")
    w_gpu = {k: v.to("cuda:0") for k, v in w.items()}
    prompt = inputs.make_prompt(shape).tolist()
    K, N = shape.K, topo.n_nodes

    def run(batch):
        model = Amphista(shape, topo, w_gpu, temperature=0.7, seed=SEED, max_batch=batch)
        out = [[model.prefill(prompt, seq=b)] for b in range(batch)]
        tok = torch.zeros(batch, K + 1, dtype=torch.int32, device="cuda:0")
        n = torch.zeros(batch, dtype=torch.int32, device="cuda:0")
        for step in range(5):
            model.draft(); model.verify_tree()
            for b in range(batch):
                assert model.get_tensor(f"uniforms#{b}", (N,)).cpu().tolist() == sm.node_uniforms(SEED, step, b, N)
            model.accept(tok, n)
            torch.cuda.synchronize()
            for b in range(batch):
                out[b] += tok[b, :int(n[b])].tolist()
        model.close()
        return out

    single = run(1)[0]
    both = run(2)
    assert both[0] == single
    assert both[1] != both[0]


def test_sampling_at_the_full_vocabulary():
    """The benchmark's vocabulary (32000 ids, 64-node tree, 7B widths, two layers): every node's draw against the oracle on
    the GPU's own logits and uniforms.  A token's probability is about 3e-5 here, the same order as the float32 error of a
    32000-term running sum, so more nodes than usual sit near a boundary; there the draw must still be one of the tokens
    that meet at it."""
    from paper_2406_13170_b200 import Amphista
    shape = inputs.get_shape("7b").with_(n_layers=2, prompt_len=40)
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    t = ao.tree_tables(topo.parent, topo.depth, topo.rank)
    N, V = t.n_nodes, shape.vocab
    w_gpu = inputs.make_weights(shape, seed=0, device="cuda:0", init="fan_in")
    model = Amphista(shape, topo, w_gpu, temperature=0.7, seed=SEED)
    model.prefill(inputs.make_prompt(shape).tolist())
    stats = {"near_boundary": 0, "nodes": 0}
    for step in range(2):
        model.draft()
        model.verify_tree()
        toks = model.get_tensor("tree_tokens", (N,), torch.int32).tolist()
        logits = model.get_tensor("logits", (N, V)).cpu().to(torch.float64)
        u = sm.node_uniforms(SEED, step, 0, N)
        assert model.get_tensor("uniforms", (N,)).cpu().tolist() == u
        choice = model.get_tensor("argmax", (N,), torch.int32).tolist()
        _check_choices(choice, toks, logits, t, 0.7, u, stats)
        g_tok = torch.zeros(shape.K + 1, dtype=torch.int32, device="cuda:0")
        g_n = torch.zeros(1, dtype=torch.int32, device="cuda:0")
        model.accept(g_tok, g_n)
        torch.cuda.synchronize()
        L, path, emitted, nxt = ao.Oracle.accept(toks, choice, t)
        assert int(g_n[0]) == L and g_tok[:L].tolist() == emitted and model.get_state()[1] == nxt
    print(stats)
    assert stats["nodes"] == 2 * N and stats["near_boundary"] < stats["nodes"] // 2
    model.close()
