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
