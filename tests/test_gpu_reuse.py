"""A context is reused for several sequences, and the path is deterministic: the same inputs give bit-identical
tokens, logits and cache rows from run to run, with the CUDA-graph replay of amph_step and with its kernels launched
one by one (split-K partial sums are always added in a fixed order; there are no floating-point atomics)."""
import pytest
import torch

import inputs

pytestmark = pytest.mark.gpu


def _run(model, shape, prompt, steps, use_step):
    K, V, d = shape.K, shape.vocab, shape.d_model
    root = model.prefill(prompt)
    out_tok = torch.zeros(K + 1, dtype=torch.int32, device="cuda:0")
    out_n = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    toks = [root]
    for _ in range(steps):
        if use_step:
            model.step(out_tok, out_n)
        else:
            model.draft()
            model.verify_tree()
            model.accept(out_tok, out_n)
        torch.cuda.synchronize()
        toks += out_tok[: int(out_n[0])].tolist()
    C, root, _ = model.get_state()
    kv = model.get_tensor("kv.k.0", (C, d)).clone()
    dl = model.get_tensor("d_logits", (K, V)).clone()
    return toks, C, root, kv, dl


@pytest.mark.parametrize("name", ["tiny", "small_bf16"])
def test_reuse_and_bitwise_determinism(name):
    from paper_2406_13170_b200 import Amphista
    shape = inputs.get_shape(name)
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    w = inputs.make_weights(shape, seed=0, device="cuda:0")
    p1 = inputs.make_prompt(shape).tolist()
    p2 = [(t * 7 + 3) % shape.vocab for t in p1[: len(p1) // 2]]
    m = Amphista(shape, topo, w)
    a = _run(m, shape, p1, 4, use_step=True)
    b = _run(m, shape, p2, 3, use_step=True)          # a second sequence in the same context (prefill resets it)
    m.reset()
    c = _run(m, shape, p1, 4, use_step=True)          # the first one again, after an explicit reset
    assert a[0] == c[0] and a[1:3] == c[1:3]
    assert torch.equal(a[3], c[3]) and torch.equal(a[4], c[4])
    assert b[0] != a[0]
    m.close()
    # kernels launched one by one (no graph), phases called separately: same bits
    m2 = Amphista(shape, topo, w, flags=2)
    e = _run(m2, shape, p1, 4, use_step=False)
    assert e[0] == a[0] and e[1:3] == a[1:3]
    assert torch.equal(e[3], a[3]) and torch.equal(e[4], a[4])
    m2.close()
