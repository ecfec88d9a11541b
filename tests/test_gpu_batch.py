"""GPU parity of several sequences decoded side by side (Section 4.4, Table 6) against the batched CPU oracle."""
import pytest
import torch

import inputs
from oracle import amphista_oracle as ao
from oracle import amphista_batch_oracle as bo
from tests.parity import run_parity_batch

pytestmark = pytest.mark.gpu


def _prompts(shape, lens):
    return [inputs.make_prompt(shape.with_(prompt_len=n), seed=1 + i).tolist() for i, n in enumerate(lens)]


@pytest.mark.parametrize("planted", [False, True], ids=["natural", "planted"])
@pytest.mark.parametrize("base,lens", [("tiny", (32, 19)), ("tiny", (32, 7, 45, 150)), ("small_bf16", (48, 33)),
                                       ("small_bf16", (48, 21, 70, 140)), ("tiny", (5, 9, 3, 17, 11, 8, 2, 30))],
                         ids=["fp32-b2", "fp32-b4-ragged", "bf16-b2", "bf16-b4-ragged", "fp32-b8"])
def test_batched_steps_match_the_batched_oracle(base, lens, planted):
    """Every sequence of the batch against the padded batched oracle: drafted candidates, tree tokens, logits and
    hidden rows of its own tree, greedy choices, accepted path / tokens / next root, its compacted cache rows and its
    adaptation-layer caches.  Prompts of different lengths (one longer than a 128-token prefill chunk) and planted
    continuations of different depths make the sequences' lengths drift apart."""
    from paper_2406_13170_b200 import Amphista
    shape = inputs.get_shape(base)
    B = len(lens)
    if shape.n_nodes * B > 512:
        pytest.skip("more rows than one pass carries")
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    w_cpu = inputs.make_weights(shape, seed=0)
    w_gpu = {k: v.to("cuda:0") for k, v in w_cpu.items()}
    bf = shape.dtype == "bf16"
    model = Amphista(shape, topo, w_gpu, max_batch=B, max_ctx=max(lens) + 6 * (shape.K + 1) + shape.n_nodes + 16)
    borc = bo.BatchOracle(shape, w_cpu, dtype=torch.float64)
    prompts = _prompts(shape, lens)
    futures = None
    if planted:
        single = ao.Oracle(shape, w_cpu, dtype=torch.float64)
        futures = [single.greedy_ar(p, 5 * (shape.K + 1) + shape.K + 2) for p in prompts]
    reps = run_parity_batch(model, borc, shape, topo, prompts, 4, 2e-2 if bf else 1e-5, 1e-3 if bf else 1e-5, futures)
    for r in reps:
        print(r)
        assert r.steps == 4
    if planted:
        assert max(max(r.accepted) for r in reps) >= 3
        assert len({tuple(r.accepted) for r in reps}) > 1           # the sequences did advance by different amounts
    model.close()


def test_batched_free_running_steps_are_lossless():
    """amph_step on a batch of four (graph replay, no host involvement between steps): every sequence's emitted
    tokens equal plain greedy decoding of the target for its own prompt (Sections 1-2), on the fp32 shape token for token."""
    from paper_2406_13170_b200 import Amphista
    shape = inputs.get_shape("tiny")
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    w_cpu = inputs.make_weights(shape, seed=0)
    w_gpu = {k: v.to("cuda:0") for k, v in w_cpu.items()}
    lens = (32, 11, 64, 27)
    prompts = _prompts(shape, lens)
    single = ao.Oracle(shape, w_cpu, dtype=torch.float64)
    want = [single.greedy_ar(p, 8 * (shape.K + 1) + 2) for p in prompts]
    B = len(lens)
    model = Amphista(shape, topo, w_gpu, max_batch=B)
    roots = [model.prefill(p, seq=b) for b, p in enumerate(prompts)]
    assert roots == [w[0] for w in want]
    out_tok = torch.zeros(B, shape.K + 1, dtype=torch.int32, device="cuda:0")
    out_n = torch.zeros(B, dtype=torch.int32, device="cuda:0")
    got = [[] for _ in range(B)]
    for _ in range(8):
        model.step(out_tok, out_n)
        torch.cuda.synchronize()
        for b in range(B):
            got[b] += out_tok[b, :int(out_n[b])].tolist()
    for b in range(B):
        assert len(got[b]) >= 8 and got[b] == want[b][:len(got[b])]
    model.close()


def test_batch_of_four_at_7b_widths():
    """Four ragged sequences with 64-node trees at the 7B widths (two layers, well-conditioned weights): 256 rows per
    verification pass, i.e. two 128-row blocks per weight tile in the projections and four row groups per attention and
    rotary launch at head_dim 128: the launch shapes of the sweep's batch-4 column, at the stated tolerance."""
    from paper_2406_13170_b200 import Amphista
    shape = inputs.get_shape("7b").with_(n_layers=2)
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    w_gpu = inputs.make_weights(shape, seed=0, device="cuda:0", init="fan_in")
    w_cpu = {k: v.cpu() for k, v in w_gpu.items()}
    lens = (70, 40, 130, 55)
    model = Amphista(shape, topo, w_gpu, max_batch=4, max_ctx=512)
    borc = bo.BatchOracle(shape, w_cpu, dtype=torch.float32)
    reps = run_parity_batch(model, borc, shape, topo, _prompts(shape, lens), 2, 2e-2, 1e-3, None)
    for r in reps:
        print(r)
        assert r.steps == 2
    model.close()
