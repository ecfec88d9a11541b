"""GPU parity: the CUDA library against the CPU oracle, through the C ABI."""
import pytest
import torch

import inputs
from inputs.configs import ModelShape
from oracle import amphista_oracle as ao
from tests.parity import run_parity

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-5      # fp32 kernels against the float64 oracle
TOL_BF16 = 2e-2     # bf16 weights / activations, fp32 accumulation, against the oracle
TIE_F32 = 1e-5
TIE_BF16 = 1e-3


def _setup(shape, topo, flags=0, max_ctx=None):
    from paper_2406_13170_b200 import Amphista
    w_cpu = inputs.make_weights(shape, seed=0)
    w_gpu = inputs.make_weights(shape, seed=0, device="cuda:0")
    for k in ("tok_emb", "layers.0.wq", "draft.lm_head.0.b" if shape.lm_rank else "draft.lm_head.0"):
        assert torch.equal(w_cpu[k], w_gpu[k].cpu()), "input generator must be device independent"
    model = Amphista(shape, topo, w_gpu, max_ctx=max_ctx, flags=flags)
    orc = ao.Oracle(shape, w_cpu, dtype=torch.float64)
    return model, orc


@pytest.mark.parametrize("planted", [False, True], ids=["natural", "planted"])
def test_tiny_fp32_eight_steps(planted):
    shape = inputs.get_shape("tiny")
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    model, orc = _setup(shape, topo)
    prompt = inputs.make_prompt(shape).tolist()
    rep = run_parity(model, orc, shape, topo, prompt, shape.steps, TOL_F32, TIE_F32, planted)
    print(rep)
    assert rep.steps == shape.steps
    if planted:
        assert max(rep.accepted) >= 3
    model.close()


def test_tiny_depth4_tree_and_ragged_prompt():
    shape = inputs.get_shape("tiny").with_(n_nodes=15, prompt_len=37, topk=(2, 2, 1, 1))
    topo = inputs.full_tree([2, 2, 1, 1])
    model, orc = _setup(shape, topo)
    prompt = inputs.make_prompt(shape).tolist()
    rep = run_parity(model, orc, shape, topo, prompt, 5, TOL_F32, TIE_F32, True)
    assert max(rep.accepted) == 5
    model.close()


@pytest.mark.parametrize("flags", [1, 0, 4, 8, 16, 32, 256], ids=["plain-kernels", "tensor-core", "separate-rope", "separate-merge",
                                                                 "separate-swiglu", "mma-sync-attention", "no-side-prefetch"])
@pytest.mark.parametrize("planted", [False, True], ids=["natural", "planted"])
def test_small_bf16_eight_steps(planted, flags):
    """bf16 storage, several 128-row weight tiles, a 32-node tree, a prompt that is not a
    multiple of the chunk size; every step compared against the float64 oracle."""
    shape = inputs.get_shape("small_bf16")
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    model, orc = _setup(shape, topo, flags=flags)
    prompt = inputs.make_prompt(shape).tolist()
    rep = run_parity(model, orc, shape, topo, prompt, shape.steps, TOL_BF16, TIE_BF16, planted,
                     kv_check_layers=(0, 1, 2))
    print(rep)
    if planted:
        assert max(rep.accepted) >= 3
    model.close()


def test_long_prompt_many_attention_splits_fp32():
    """A 300-token context: several KV splits per head, three prefill chunks (fp32: tight tolerance)."""
    shape = inputs.get_shape("tiny").with_(prompt_len=300)
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    model, orc = _setup(shape, topo)
    rep = run_parity(model, orc, shape, topo, inputs.make_prompt(shape).tolist(), 3, TOL_F32, TIE_F32, True)
    print(rep)
    model.close()


def test_long_prompt_many_attention_splits_bf16():
    shape = inputs.get_shape("small_bf16").with_(prompt_len=333)
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    model, orc = _setup(shape, topo)
    rep = run_parity(model, orc, shape, topo, inputs.make_prompt(shape).tolist(), 3, TOL_BF16, TIE_BF16, True,
                     kv_check_layers=(0, 1, 2))
    print(rep)
    model.close()


@pytest.mark.parametrize("variant", [dict(n_sal=1), dict(aeb_layers=2), dict(n_sal=1, aeb_layers=2), dict(lm_rank=64),
                                     dict(lm_rank=24), dict(n_sal=0), dict(aeb_layers=0), dict(n_sal=0, aeb_layers=0),
                                     dict(use_sampled_token=False)],
                         ids=["one-sal", "alpha-two-aeb-layers", "one-sal-two-aeb-layers", "low-rank-heads-64",
                              "low-rank-heads-24", "no-sal", "no-aeb", "no-sal-no-aeb", "no-sampled-token"])
@pytest.mark.parametrize("base", ["tiny", "small_bf16"])
def test_draft_module_variants(base, variant):
    """The draft-module variants the paper evaluates: a single adaptation layer (the "One-Adaptation-Layer"
    ablation of Section 4.5: every head then reads h1), the two-layer Auto-embedding Block ("Amphista-alpha",
    Appendix A.2.3) and vocabulary heads factored into two low-rank matrices (Appendix A.2.4; on bf16, rank 64
    takes the tensor-core projection and rank 24 the plain one); and the ablations of Section 4.5 that remove a
    module: no adaptation layers (the heads read the target's hidden state), no Auto-embedding Block, and no
    sampled token (fc is d -> d on the hidden state alone)."""
    shape = inputs.get_shape(base).with_(**variant)
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    model, orc = _setup(shape, topo)
    prompt = inputs.make_prompt(shape).tolist()
    bf = shape.dtype == "bf16"
    rep = run_parity(model, orc, shape, topo, prompt, 4, TOL_BF16 if bf else TOL_F32, TIE_BF16 if bf else TIE_F32, True)
    print(rep)
    assert rep.steps == 4 and max(rep.accepted) >= 3
    model.close()


@pytest.mark.parametrize("case", ["root-only-tree", "one-token-prompt", "max-nodes-128", "one-head", "eight-heads-top16"])
def test_degenerate_and_maximum_shapes(case):
    """The corners of the interface: a tree that is only its root (every step then emits exactly one token, i.e.
    plain autoregressive decoding through the speculative path), a prompt of one token, the largest tree the
    library takes (128 nodes: two 64-row blocks in attention, 128 activation rows in the projections), a single
    drafting head, and the maximum of eight heads keeping 16 candidates each."""
    base = inputs.get_shape("tiny")
    if case == "root-only-tree":
        shape, topo, steps, planted = base.with_(n_nodes=1), inputs.chain_tree(1), 6, False
    elif case == "one-token-prompt":
        shape, steps, planted = base.with_(prompt_len=1), 5, True
        topo = inputs.make_tree(shape.n_nodes, shape.topk)
    elif case == "max-nodes-128":
        shape = base.with_(n_nodes=128, topk=(16, 8, 4, 2))
        topo, steps, planted = inputs.make_tree(128, shape.topk), 4, True
    elif case == "one-head":
        shape = base.with_(K=1, topk=(4,), n_nodes=5)
        topo, steps, planted = inputs.make_tree(5, shape.topk), 5, True
    else:
        shape = base.with_(K=8, topk=(16,) * 8, n_nodes=96)
        topo, steps, planted = inputs.make_tree(96, shape.topk), 3, True
    model, orc = _setup(shape, topo)
    prompt = inputs.make_prompt(shape).tolist()
    rep = run_parity(model, orc, shape, topo, prompt, steps, TOL_F32, TIE_F32, planted)
    print(rep)
    assert rep.steps == steps
    if case == "root-only-tree":
        assert rep.accepted == [1] * steps
    model.close()


def test_small_bf16_max_nodes_128():
    """128 tree rows on the tensor-core path: single-block stages in the projections, two row blocks per attention cluster."""
    shape = inputs.get_shape("small_bf16").with_(n_nodes=128, topk=(16, 8, 4, 2))
    topo = inputs.make_tree(128, shape.topk)
    model, orc = _setup(shape, topo)
    rep = run_parity(model, orc, shape, topo, inputs.make_prompt(shape).tolist(), 3, TOL_BF16, TIE_BF16, True)
    print(rep)
    model.close()
