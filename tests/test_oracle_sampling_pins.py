"""Pins of the sampling oracle (temperature T > 0; Table 2, Sections 1-2).  Nothing here touches the CUDA library.

What must hold whatever the implementation: the generator reproduces its published known-answer vectors; the tokens a
step emits are distributed exactly as ancestral sampling from the target at temperature T (the "lossless" property the
paper cites for rejection sampling), shown by enumerating every cell of the uniforms on a small vocabulary; T -> 0 is
greedy decoding; the sequential rejection form equals the form with unscaled uniforms.
"""
import itertools
import os

import pytest
import torch

from oracle import amphista_oracle as ao
from oracle import amphista_sampling as sm

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_philox_known_answers():
    n = 0
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        if not line.startswith("kat"):
            continue
        w = [int(x, 16) for x in line.split()[1:]]
        assert sm.philox4x32_10(w[0:4], w[4:6]) == w[6:10]
        n += 1
    assert n == 3


def test_uniforms_are_24_bit_and_distinct_per_counter():
    us = [sm.uniform(12345, s, q, n) for s in range(4) for q in range(2) for n in range(16)]
    assert all(0.0 <= u < 1.0 and float(torch.tensor(u, dtype=torch.float32)) == u and (u * 2 ** 24) % 1 == 0 for u in us)
    assert len(set(us)) == len(us)
    assert sm.uniform(1, 0, 0, 0) != sm.uniform(2, 0, 0, 0) != sm.uniform(1 + (1 << 32), 0, 0, 0)
    assert sm.uniform(7, 3, 0, 5, stream=0) != sm.uniform(7, 3, 0, 5, stream=1)
    many = [sm.uniform(99, s, 0, n) for s in range(64) for n in range(64)]
    assert abs(sum(many) / len(many) - 0.5) < 0.02


def _tree():
    #        0
    #      /   \
    #     1     2
    #    / \    |
    #   3   4   5
    parent, depth, rank = [-1, 0, 0, 1, 1, 2], [0, 1, 1, 2, 2, 2], [0, 0, 1, 0, 1, 0]
    return ao.tree_tables(parent, depth, rank)


def _cells(p, toks, children):
    """Boundaries of the uniform at one node: the cumulative sums in the order children's tokens, then other ids."""
    order = []
    for c in children:
        if toks[c] not in order:
            order.append(toks[c])
    order += [y for y in range(p.numel()) if y not in order]
    edges = [0.0]
    for y in order:
        edges.append(edges[-1] + float(p[y]))
    edges[-1] = 1.0
    return [(a, b) for a, b in zip(edges[:-1], edges[1:]) if b > a]


@pytest.mark.parametrize("T", [0.7, 1.0, 0.25])
def test_emitted_tokens_follow_the_target_distribution_exactly(T):
    """Enumerates every cell of every uniform on the walked path and adds up the cells' volumes per outcome (the new
    tokens of the step: accepted tokens, then the next root).  The result must equal ancestral sampling from
    softmax(logits / T): draw y ~ p(node); if y is a child's token continue at that child, else stop."""
    torch.manual_seed(3)
    t = _tree()
    V = 6
    logits = torch.randn(t.n_nodes, V, dtype=torch.float64) * 2.0
    toks = [0, 2, 4, 1, 5, 3]
    got = {}

    def walk(n, u_known, vol, seq):
        p = sm.target_probs(logits[n], T)
        for a, b in _cells(p, toks, sm.children_of(t, n)):
            u = [0.5] * t.n_nodes
            for k, v in u_known.items():
                u[k] = v
            u[n] = 0.5 * (a + b)
            L, path, emitted, nxt = sm.accept_sampled(toks, logits, t, T, u)
            d = len(seq)                       # tokens already decided below the root
            if len(path) > d + 1:              # moved on to a child of n
                c = path[d + 1]
                walk(c, {**u_known, n: u[n]}, vol * (b - a), seq + [toks[c]])
            else:
                key = tuple(seq + [nxt])
                got[key] = got.get(key, 0.0) + vol * (b - a)

    walk(0, {}, 1.0, [])
    want = {}

    def ancestral(n, prob, seq):
        p = sm.target_probs(logits[n], T)
        kids = {toks[c]: c for c in reversed(sm.children_of(t, n))}
        for y in range(V):
            if y in kids:
                ancestral(kids[y], prob * float(p[y]), seq + [y])
            else:
                want[tuple(seq + [y])] = want.get(tuple(seq + [y]), 0.0) + prob * float(p[y])

    ancestral(0, 1.0, [])
    assert set(got) == set(want)
    assert abs(sum(got.values()) - 1.0) < 1e-12
    for k in want:
        assert abs(got[k] - want[k]) < 1e-12, (k, got[k], want[k])
    # and the first new token alone has the target's own distribution at the root
    p0 = sm.target_probs(logits[0], T)
    for y in range(V):
        assert abs(sum(v for k, v in got.items() if k[0] == y) - float(p0[y])) < 1e-12


def test_temperature_to_zero_is_greedy():
    torch.manual_seed(5)
    t = _tree()
    for trial in range(50):
        logits = torch.randn(t.n_nodes, 9, dtype=torch.float64) * 3.0
        amax = [ao.argmax_lowest(logits[n]) for n in range(t.n_nodes)]
        toks = [0] + [int(x) for x in torch.randint(0, 9, (t.n_nodes - 1,))]
        if trial % 2:                                    # plant the greedy continuation on the path 0 -> 1 -> 4
            toks[1], toks[4] = amax[0], amax[1]
        if toks[1] == toks[2] or toks[3] == toks[4]:
            continue
        u = [float(x) for x in torch.rand(t.n_nodes, dtype=torch.float64) * 0.98 + 0.01]
        assert sm.accept_sampled(toks, logits, t, 1e-3, u) == ao.Oracle.accept(toks, amax, t)


def test_sequential_rejection_form_equals_unscaled_form():
    torch.manual_seed(7)
    t = _tree()
    for trial in range(300):
        V = 12
        logits = torch.randn(t.n_nodes, V, dtype=torch.float64) * 2.0
        toks = [0] + [int(x) for x in torch.randperm(V)[:t.n_nodes - 1]]
        u = [float(x) for x in torch.rand(t.n_nodes, dtype=torch.float64)]
        margins = []
        flat = sm.accept_flat(toks, logits, t, 0.7, u)
        sm.choices_flat(toks, logits, t, 0.7, u, margins)
        if min(margins) < 1e-9:
            continue
        assert sm.accept_sampled(toks, logits, t, 0.7, u) == flat
