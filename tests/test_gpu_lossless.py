"""Losslessness on the GPU (Sections 1-2, Appendix A.3): amph_step running free, with nobody handing it tokens,
must emit exactly the tokens that plain greedy autoregressive decoding of the target emits.  The oracle's
greedy_ar is the plain definition; the library is the call the benchmark times (CUDA-graph replay) and the
same schedule launched kernel by kernel."""
import pytest
import torch

import inputs
from oracle import amphista_oracle as ao

pytestmark = pytest.mark.gpu

AMPH_FLAG_NO_GRAPH = 2


def _free_run(shape, topo, weights, prompt, steps, flags):
    from paper_2406_13170_b200 import Amphista
    m = Amphista(shape, topo, weights, flags=flags)
    out_tok = torch.zeros(shape.K + 1, dtype=torch.int32, device="cuda:0")
    out_n = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    toks, per_step = [], []
    m.prefill(prompt)
    for _ in range(steps):
        m.step(out_tok, out_n)
        m.synchronize()
        n = int(out_n[0])
        assert 1 <= n <= shape.K + 1
        per_step.append(out_tok[:n].tolist())
        toks += per_step[-1]
    C, root, n_pending = m.get_state()
    m.close()
    return toks, per_step, C, root


@pytest.mark.parametrize("flags", [0, AMPH_FLAG_NO_GRAPH], ids=["graph-replay", "kernel-by-kernel"])
def test_tiny_fp32_free_running_equals_greedy_autoregressive(flags):
    shape = inputs.get_shape("tiny")
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    w_cpu = inputs.make_weights(shape, seed=0)
    w_gpu = {k: v.to("cuda:0") for k, v in w_cpu.items()}
    prompt = inputs.make_prompt(shape).tolist()
    steps = 8
    toks, per_step, C, root = _free_run(shape, topo, w_gpu, prompt, steps, flags)
    orc = ao.Oracle(shape, w_cpu, dtype=torch.float64)
    ref = orc.greedy_ar(prompt, len(toks) + 1)
    assert toks == ref[:len(toks)], f"emitted {toks} vs greedy {ref[:len(toks)]}"
    assert root == ref[len(toks)]                      # the carried root is the next greedy token
    assert C == len(prompt) + len(toks)


@pytest.mark.parametrize("flags", [0, AMPH_FLAG_NO_GRAPH], ids=["graph-replay", "kernel-by-kernel"])
def test_small_bf16_free_running_against_greedy_autoregressive(flags):
    """bf16 storage: the stream must agree with the float64 oracle's greedy stream up to the first position where
    the oracle's own top-2 gap is smaller than the bf16 error of the logits (2e-2 of the logit scale); the test
    reports that position and fails on any earlier disagreement."""
    shape = inputs.get_shape("small_bf16")
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    w_cpu = inputs.make_weights(shape, seed=0)
    w_gpu = {k: v.to("cuda:0") for k, v in w_cpu.items()}
    prompt = inputs.make_prompt(shape).tolist()
    toks, per_step, C, root = _free_run(shape, topo, w_gpu, prompt, 8, flags)
    orc = ao.Oracle(shape, w_cpu, dtype=torch.float64)
    ref = orc.greedy_ar(prompt, len(toks) + 1)
    stream = toks + [root]
    first = next((i for i, (a, b) in enumerate(zip(stream, ref)) if a != b), None)
    print("first divergence at token", first, "of", len(stream))
    if first is not None:
        # logits of the oracle at the diverging position: run the agreed prefix through the plain forward
        st = orc.prefill(prompt + ref[:first]) if first > 0 else orc.prefill(prompt)
        lg = st.last_logits.to(torch.float64)
        top2 = torch.topk(lg, 2).values
        scale = max(1.0, float(lg.abs().max()))
        assert float(top2[0] - top2[1]) <= 2e-2 * scale, \
            f"token {first}: gpu {stream[first]} vs greedy {ref[first]} with an oracle gap of {float(top2[0] - top2[1])}"
        assert float(lg[stream[first]]) >= float(top2[0]) - 2e-2 * scale
