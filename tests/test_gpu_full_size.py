"""Parity at the benchmark's full size and at the other large shapes.

The 7B-shape test runs the exact configuration bench.py times (32 layers, d = 4096, vocab 32000, 64-node
tree, 512-token prompt, tensor-core projections, CUDA-graph step) and compares it with the float32 CPU
oracle on the same seeded weights: root token, draft logits and candidates, all 64 verified rows, acceptance
and the compacted cache, for one natural and one planted step.  The 13B / 33B shapes are checked at two
layers of depth (their widths, head counts and tile counts are what differs from 7B).
"""
import pytest
import torch

import inputs
from oracle import amphista_oracle as ao
from tests.parity import run_parity

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
TIE_BF16 = 1e-3


def tol_plain(n_layers: int) -> float:
    """Against the oracle that keeps every activation in float32.  The bf16 storage points (projection
    inputs, rotated queries, KV rows) inject an error that accumulates like a random walk over the layers
    of a random-init model: measured 1.1e-2 at 2 layers, 2.1e-2 at 8, 3.5e-2 at 16, 4.0e-2 at 32 (7B
    widths), and reproduced on the CPU by the oracle's bf16-storage mode.  2e-2 holds up to 4 layers."""
    return TOL_BF16 * max(1.0, (n_layers / 4.0) ** 0.5)


def tol_draft(n_layers: int) -> float:
    """The draft module sits on top of the target's last hidden state and adds two decoder layers, the head
    MLPs, the attention block and an un-normalised vocabulary projection (draft logits of a random-init
    model have a standard deviation of 11 against 1.3 for the target).  With N(0, 0.02) weights every linear
    map of width d has gain 0.02 * sqrt(d) (1.28 at 4096, 1.63 at 6656), so these random-init stacks amplify
    the bf16 storage rounding strongly: measured against the plain oracle 6e-2 .. 0.12 (7B widths, 2-layer
    target), 0.24 (33B widths, 2 layers), 0.25 .. 0.40 (7B, 32 layers).  At these widths closeness of the draft
    tensors is therefore only bounded loosely (0.6; unrelated outputs give about 1.4); the draft module's
    arithmetic is pinned tightly by the small-shape tests (1e-5 in fp32, 2e-2 in bf16)."""
    return 0.6


def _run(shape, steps, planted, prompt_len=None, kv_layers=(0, -1), storage=None):
    from paper_2406_13170_b200 import Amphista
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    w_gpu = inputs.make_weights(shape, seed=0, device="cuda:0")
    w_cpu = {k: v.cpu() for k, v in w_gpu.items()}                 # same generator; device independence is tested elsewhere
    probe = inputs.normal_tensor(w_cpu["layers.0.wq"].shape, 0.02, 0, "layers.0.wq", dtype=torch.bfloat16)
    assert torch.equal(probe, w_cpu["layers.0.wq"])
    model = Amphista(shape, topo, w_gpu)
    orc = ao.Oracle(shape, w_cpu, dtype=torch.float32, storage=storage)
    tol = tol_plain(shape.n_layers)
    prompt = inputs.make_prompt(shape, n=prompt_len or shape.prompt_len).tolist()
    rep = run_parity(model, orc, shape, topo, prompt, steps, tol, TIE_BF16, planted, kv_check_layers=kv_layers,
                     tol_draft=tol_draft(shape.n_layers))
    print(shape.name, rep)
    # the same context must also run through amph_step (graph replay) and stay consistent with its own state
    out_tok = torch.zeros(shape.K + 1, dtype=torch.int32, device="cuda:0")
    out_n = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    C0 = model.get_state()[0]
    for _ in range(3):
        model.step(out_tok, out_n)
    model.synchronize()
    C1 = model.get_state()[0]
    assert 3 <= C1 - C0 <= 3 * (shape.K + 1) and 1 <= int(out_n[0]) <= shape.K + 1
    model.close()
    return rep


def test_7b_shape_full_depth():
    shape = inputs.get_shape("7b")
    rep = _run(shape, 2, True)
    assert rep.steps == 2 and max(rep.accepted) >= 2


@pytest.mark.parametrize("storage", [None, torch.bfloat16], ids=["plain-oracle", "bf16-storage-oracle"])
@pytest.mark.parametrize("name", ["7b", "13b", "33b"])
def test_large_shapes_two_layers(name, storage):
    shape = inputs.get_shape(name).with_(n_layers=2, prompt_len=70)
    rep = _run(shape, 2, True, kv_layers=(0, 1), storage=storage)
    assert rep.steps == 2
