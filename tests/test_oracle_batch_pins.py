"""Pins of the batched CPU oracle (Section 4.4: sentences of different lengths padded to a common length, the last
valid token of each tracked).  Nothing here touches the CUDA library.

The padded, masked formulation must give every sentence exactly what it gets when decoded alone by the
single-sequence oracle (itself pinned in test_oracle_pins.py): padding rows, padding slots and the other sentences
of the batch must have no influence.  A wrong last-valid index, a mask that lets padding into a softmax, a slot
offset that uses the padded instead of the own length, or a compaction that moves another sentence's rows fails here.
"""
import pytest
import torch

import inputs
from inputs.configs import ModelShape
from oracle import amphista_oracle as ao
from oracle import amphista_batch_oracle as bo

MICRO = ModelShape("micro", 2, 64, 2, 32, 96, 50, "fp32", topk=(3, 2, 2, 1), n_nodes=12, prompt_len=9, steps=6)


def _prompts(shape, lens, seed=1):
    return [inputs.make_prompt(shape.with_(prompt_len=n), seed=seed + i).tolist() for i, n in enumerate(lens)]


def _plant(t, future, leaf):
    ov = [-1] * t.n_nodes
    for i, n in enumerate(t.ancestors[leaf]):
        if i > 0 and i - 1 < len(future):
            ov[n] = future[i - 1]
    return ov


@pytest.mark.parametrize("lens", [(9, 4, 13), (1, 7), (6, 6, 6, 6)], ids=["ragged-3", "one-token-and-7", "equal-4"])
def test_batched_step_equals_each_sentence_alone(lens):
    shape = MICRO
    w = inputs.make_weights(shape, seed=0, std=0.3)                 # large weights: softmaxes far from uniform
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    t = ao.tree_tables(topo.parent, topo.depth, topo.rank)
    single = ao.Oracle(shape, w, dtype=torch.float64)
    batch = bo.BatchOracle(shape, w, dtype=torch.float64)
    prompts = _prompts(shape, lens)
    B = len(prompts)
    sts = [single.prefill(p) for p in prompts]
    bs = batch.prefill(prompts)
    assert bs.root == [s.root for s in sts] and bs.C == [s.C for s in sts]
    for b in range(B):
        assert torch.allclose(bs.last_logits[b], sts[b].last_logits, atol=1e-10)
    futures = [single.greedy_ar(p, 40) for p in prompts]
    done = [0] * B
    accepted = []
    emitted_all = [[] for _ in range(B)]
    for i in range(4):
        # different sentences accept different numbers of tokens: plant continuations of different depths
        ovs = []
        for b in range(B):
            leaf = t.leaves[(i + 2 * b) % len(t.leaves)]
            ovs.append(_plant(t, futures[b][done[b] + 1: done[b] + 1 + t.depth[leaf]], leaf) if (i + b) % 3 else None)
        taps_b = [dict() for _ in range(B)]
        out_b = batch.step(bs, t, ovs, taps_b)
        for b in range(B):
            taps = {}
            out = single.step(sts[b], t, ovs[b], taps)
            assert out_b[b] == out, f"step {i} sentence {b}"
            assert taps_b[b]["path"] == taps["path"] and taps_b[b]["next_root"] == taps["next_root"]
            assert taps_b[b]["topk_ids"] == taps["topk_ids"] and taps_b[b]["toks"] == taps["toks"]
            for key in ("h1", "h2", "Hp", "attn_o", "d_logits", "hid", "logits"):
                assert torch.allclose(taps_b[b][key], taps[key], atol=1e-9), f"step {i} sentence {b}: {key}"
            assert (bs.C[b], bs.root[b]) == (sts[b].C, sts[b].root)
            done[b] += len(out)
            emitted_all[b] += out
            accepted.append(len(out))
    assert len(set(bs.C)) > 1 or len(set(lens)) == 1 and len(set(accepted)) > 1     # the batch really became ragged
    # committed caches: every valid slot equals the sentence's own cache, everything after it is padding (zero)
    for b in range(B):
        for l in range(shape.n_layers):
            k_ref = torch.stack(sts[b].kv[l].k[:sts[b].C])
            assert torch.allclose(bs.K[l][b, :bs.C[b]], k_ref, atol=1e-9)
            assert float(bs.K[l][b, bs.C[b]:].abs().max()) == 0.0 if bs.K[l].shape[1] > bs.C[b] else True
        for s in range(shape.n_sal):
            n_rows = len(sts[b].sal_kv[s].k)
            assert torch.allclose(bs.sal_K[s][b, :n_rows], torch.stack(sts[b].sal_kv[s].k), atol=1e-9)
    # and the whole run is lossless for every sentence (Sections 1-2)
    for b in range(B):
        assert emitted_all[b] == futures[b][:done[b]]


def test_batched_output_is_lossless_and_independent_of_the_neighbours():
    """The tokens a sentence emits equal plain greedy decoding of the target whatever shares the batch with it."""
    shape = MICRO
    w = inputs.make_weights(shape, seed=0, std=0.3)
    topo = inputs.make_tree(shape.n_nodes, shape.topk)
    t = ao.tree_tables(topo.parent, topo.depth, topo.rank)
    single = ao.Oracle(shape, w, dtype=torch.float64)
    batch = bo.BatchOracle(shape, w, dtype=torch.float64)
    pa, pb, pc = _prompts(shape, (5, 11, 8))
    want = single.greedy_ar(pa, 30)
    for others in ([pb], [pc, pb], [pb, pb, pc]):
        prompts = [pa] + others
        bs = batch.prefill(prompts)
        got = []
        fut = [single.greedy_ar(p, 30) for p in prompts]
        done = [0] * len(prompts)
        for i in range(4):
            ovs = [_plant(t, fut[b][done[b] + 1: done[b] + 5], t.leaves[(i + b) % len(t.leaves)]) for b in range(len(prompts))]
            out = batch.step(bs, t, ovs)
            for b in range(len(prompts)):
                done[b] += len(out[b])
            got += out[0]
        assert got == want[:len(got)] and len(got) > 4
