"""Error behaviour of the C ABI on a device: every misuse returns a status and leaves the context usable.
None of these cases runs a kernel on bad input; they are all caught on the host."""
import pytest
import torch

import inputs

pytestmark = pytest.mark.gpu


def _model(weights=None, **kw):
    from paper_2406_13170_b200 import Amphista
    shape = inputs.get_shape("tiny")
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    w = inputs.make_weights(shape, seed=0, device="cuda:0") if weights is None else weights
    return Amphista(shape, topo, w, **kw), shape, topo


def test_call_order_is_enforced_and_the_context_survives():
    from paper_2406_13170_b200.binding import AmphError
    m, shape, topo = _model()
    out_tok = torch.zeros(shape.K + 1, dtype=torch.int32, device="cuda:0")
    out_n = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    for call in (lambda: m.step(out_tok, out_n), m.draft, m.verify_tree, m.accept):     # nothing prefilled yet
        with pytest.raises(AmphError) as e:
            call()
        assert e.value.status == 3                                                     # AMPH_ERR_STATE
    m.prefill(inputs.make_prompt(shape).tolist())
    for call in (m.verify_tree, m.accept):                                             # no draft in flight
        with pytest.raises(AmphError) as e:
            call()
        assert e.value.status == 3
    m.draft()
    with pytest.raises(AmphError) as e:                                                # a draft is in flight
        m.step(out_tok, out_n)
    assert e.value.status == 3
    m.verify_tree()
    m.accept()
    m.step(out_tok, out_n)                                                             # and the sequence goes on
    torch.cuda.synchronize()
    assert 1 <= int(out_n[0]) <= shape.K + 1
    m.close()


def test_bad_prompts_are_rejected():
    from paper_2406_13170_b200.binding import AmphError
    m, shape, topo = _model()
    for bad in ([], [shape.vocab], [-1, 3]):
        with pytest.raises(AmphError) as e:
            m.prefill(bad)
        assert e.value.status == 1                                                     # AMPH_ERR_INVALID_ARG
    m.prefill([5, 7, 11])                                                              # still usable
    m.close()


def test_capacity_is_reported_before_the_cache_overflows():
    from paper_2406_13170_b200.binding import AmphError
    shape = inputs.get_shape("tiny")
    m, shape, topo = _model(max_ctx=shape.prompt_len + topo_nodes(shape) + 2 * (shape.K + 1))
    with pytest.raises(AmphError) as e:
        m.prefill(list(range(shape.prompt_len + 40)))                                  # prompt + tree does not fit
    assert e.value.status == 4                                                         # AMPH_ERR_CAPACITY
    m.prefill(inputs.make_prompt(shape).tolist())
    out_tok = torch.zeros(shape.K + 1, dtype=torch.int32, device="cuda:0")
    out_n = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    done = 0
    with pytest.raises(AmphError) as e:
        for _ in range(64):
            m.step(out_tok, out_n)
            done += 1
    assert e.value.status == 4 and done >= 2                                           # some steps fit, then a clean refusal
    C, _, _ = m.get_state()
    assert C + topo.n_nodes > m.cfg.max_ctx - (shape.K + 1) - 1                         # it stopped at the edge, not before
    m.close()


def topo_nodes(shape):
    return shape.n_nodes


def test_missing_weight_is_named():
    from paper_2406_13170_b200.binding import AmphError
    shape = inputs.get_shape("tiny")
    w = inputs.make_weights(shape, seed=0, device="cuda:0")
    del w["draft.pe"]
    m, shape, topo = _model(weights=w)
    with pytest.raises(AmphError) as e:
        m.prefill(inputs.make_prompt(shape).tolist())
    assert e.value.status == 6 and "draft.pe" in str(e.value)                          # AMPH_ERR_MISSING_WEIGHT
    m.close()


def test_a_bounded_device_wait_runs_out_and_the_device_stays_usable():
    """Every pipeline wait in the projection kernel has a time limit.  The self-test entry point makes one wait
    impossible to satisfy (its barrier expects more bytes than the copies deliver) with a 1 ms limit: the kernel must
    return, the status word must read AMPH_ERR_TIMEOUT, and an ordinary projection right after must be correct."""
    from paper_2406_13170_b200 import binding
    x = inputs.normal_tensor((64, 512), 1.0, 3, "x", dtype=torch.bfloat16).cuda()
    w = inputs.normal_tensor((256, 512), 0.05, 3, "w", dtype=torch.bfloat16).cuda()
    status, y = binding.selftest_wait_timeout(x, [w], rows=40, limit_us=1000)
    assert status == 8                                                                 # AMPH_ERR_TIMEOUT
    assert torch.equal(y, torch.zeros_like(y))                                         # abandoned tiles contribute zeros
    y2 = binding.project(x, [w], rows=40, use_tensor_core=True)                        # same device, same process
    ref = x[:40].double() @ w.double().T
    assert float((y2.double() - ref).abs().max()) < 1e-3 * float(ref.abs().max()) + 1e-4


def test_set_state_teacher_forces_the_draft():
    """amph_set_state replaces (ctx_len, root, pending rows).  Fed the oracle's own pending rows, the draft module's
    tensors match the oracle more closely than the target's hidden rows do (nothing of the target's error is
    inherited), and the state reads back as set."""
    from oracle import amphista_oracle as ao
    m, shape, topo = _model()
    prompt = inputs.make_prompt(shape).tolist()
    orc = ao.Oracle(shape, inputs.make_weights(shape, seed=0), dtype=torch.float64)
    st = orc.prefill(prompt)
    m.prefill(prompt)
    # keep only the last pending row on both sides, with a root of our choosing
    h, _, pos = st.pending[-1]
    forced_root = (st.root + 17) % shape.vocab
    st.pending = [(h, forced_root, pos)]
    st.root = forced_root
    for bad in (dict(ctx_len=len(prompt), root=shape.vocab, pend_hidden=h[None], pend_next=[forced_root]),
                dict(ctx_len=len(prompt), root=forced_root, pend_hidden=h[None], pend_next=[-1])):
        from paper_2406_13170_b200.binding import AmphError
        with pytest.raises(AmphError):
            m.set_state(**bad)
    m.set_state(len(prompt), forced_root, h[None].to(torch.float32), [forced_root])
    assert m.get_state() == (len(prompt), forced_root, 1)
    # the adaptation layers' caches cover positions 0..n-2 on the GPU already; give the oracle the same history
    taps = {}
    o_ids, o_vals, o_dl = None, None, None
    full = orc.prefill(prompt)
    full.pending = full.pending[:-1]
    orc.draft(full)                                        # oracle stage caches for positions 0..n-2
    st.sal_kv = full.sal_kv
    o_ids, o_vals, o_dl = orc.draft(st, taps)
    ids = torch.zeros(shape.K, 16, dtype=torch.int32, device="cuda:0")
    m.draft(ids)
    torch.cuda.synchronize()
    g_dl = m.get_tensor("d_logits", (shape.K, shape.vocab))
    assert float((g_dl.double().cpu() - o_dl).abs().max()) < 1e-5
    for k in range(shape.K):
        assert ids[k, :shape.topk[k]].tolist() == o_ids[k]
    assert m.get_tensor("tree_tokens", (topo.n_nodes,), torch.int32)[0].item() == forced_root
    m.close()
