"""CPU oracle for Amphista decoding at a sampling temperature T > 0 (arXiv 2406.13170, Table 2; Sections 1-2).

TEST INFRASTRUCTURE ONLY (imported by the tests alone; the product path never calls it).

The paper reports speed-ups under random sampling (T = 0.7) and states, with Leviathan et al., that speculative
decoding with a rejection-sampling strategy leaves the target's output distribution unchanged, but it does not
print the rule it applies to a candidate tree.  The reading taken here: the tree's candidates are deterministic
(the drafting heads' top-k lists), so each proposal is a point mass, and the rejection-sampling test of Section 2
reduces to the following walk from the root, with p = softmax(logits of the current node / T):

    rem = 1                                   # mass of the residual distribution
    r   = u(node)                             # one uniform per tree node
    for each child c of the node, in node order, carrying a token x not tried at this node yet:
        a = p(x) / rem                        # acceptance probability min(1, p/q) of a point-mass proposal q = 1[x]
        if r < a:   accept x, move to c, start over there with that node's own uniform
        r = (r - a) / (1 - a)                 # given the rejection, uniform on [0, 1) again
        rem = rem - p(x)                      # residual norm(max(0, p - q)): p without x, renormalised
    (every child rejected, or a leaf)         # the next root is drawn from the residual distribution by inverse
    next_root = first id y, ascending, not tried, with sum_{y' <= y, not tried} p(y') / rem > r          # transform

The emitted tokens (root, accepted tokens) and the next root are then distributed exactly as ancestral sampling
from the target at temperature T (pinned by exhaustive enumeration in the tests), and T -> 0 is greedy decoding.
`accept_flat` is the same rule with the uniform left unscaled (child i is accepted iff u < p(x_1) + .. + p(x_i)),
the form an implementation without divisions takes; the tests show the two agree.

Uniforms come from Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel Random Numbers: As Easy as 1, 2, 3", SC'11),
a counter-based generator: u(seed, step, sequence, node, stream) = top 24 bits of the first output word of
philox(counter = (node, step, sequence, stream), key = (seed mod 2^32, seed div 2^32)) times 2^-24.  stream 0 serves the
tree nodes of decoding step `step` (the number of acceptances the sequence has seen), stream 1 the token sampled after the prompt.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch

from oracle.amphista_oracle import TreeTables

_M0, _M1, _W0, _W1 = 0xD2511F53, 0xCD9E8D57, 0x9E3779B9, 0xBB67AE85
_MASK = 0xFFFFFFFF


def philox4x32_10(counter: Sequence[int], key: Sequence[int]) -> List[int]:
    """Ten rounds of the Philox-4x32 bijection: each round multiplies counter words 0 and 2 by two fixed odd
    constants (64-bit products), crosses the halves and mixes in the key, which is bumped by the Weyl constants
    between rounds."""
    c = [int(x) & _MASK for x in counter]
    k = [int(x) & _MASK for x in key]
    for r in range(10):
        if r > 0:
            k = [(k[0] + _W0) & _MASK, (k[1] + _W1) & _MASK]
        p0, p1 = _M0 * c[0], _M1 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & _MASK, (p0 >> 32) ^ c[3] ^ k[1], p0 & _MASK]
    return c


def uniform(seed: int, step: int, seq: int, node: int, stream: int = 0) -> float:
    """A uniform on [0, 1) with 24 random bits (exactly representable in float32)."""
    w = philox4x32_10([node, step, seq, stream], [seed & _MASK, (seed >> 32) & _MASK])[0]
    return (w >> 8) * 2.0 ** -24


def node_uniforms(seed: int, step: int, seq: int, n_nodes: int) -> List[float]:
    return [uniform(seed, step, seq, n, 0) for n in range(n_nodes)]


def target_probs(logits_row: torch.Tensor, T: float) -> torch.Tensor:
    """softmax(logits / T) in float64 (max subtracted first)."""
    z = logits_row.to(torch.float64) / T
    e = torch.exp(z - z.max())
    return e / e.sum()


def children_of(t: TreeTables, n: int) -> List[int]:
    return [c for c in range(n + 1, t.n_nodes) if t.parent[c] == n]


def _residual_sample(p: torch.Tensor, tried: Sequence[int], r: float, rem: float) -> int:
    acc = 0.0
    last = -1
    tried = set(tried)
    pl = p.tolist()
    for y in range(len(pl)):
        if y in tried:
            continue
        last = y
        acc += pl[y] / rem
        if acc > r:
            return y
    return last                                  # rounding left r above the total: the last admissible id


def accept_sampled(toks: Sequence[int], logits: torch.Tensor, t: TreeTables, T: float, u: Sequence[float]
                   ) -> Tuple[int, List[int], List[int], int]:
    """The walk of the module docstring.  toks [N] tree tokens, logits [N, V] target logits after each node,
    u [N] one uniform per node.  Returns (L, path node ids, emitted tokens, next_root) like Oracle.accept."""
    n = 0
    path = [0]
    while True:
        p = target_probs(logits[n], T)
        rem, r = 1.0, float(u[n])
        tried: List[int] = []
        moved = False
        for c in children_of(t, n):
            x = int(toks[c])
            if x in tried:
                continue
            a = float(p[x]) / rem if rem > 0.0 else 0.0
            if r < a:
                n = c
                path.append(c)
                moved = True
                break
            r = (r - a) / (1.0 - a) if a < 1.0 else 0.0
            rem -= float(p[x])
            tried.append(x)
        if not moved:
            nxt = _residual_sample(p, tried, r, rem)
            return len(path), path, [int(toks[m]) for m in path], nxt


def choice_flat(toks: Sequence[int], logits_row: torch.Tensor, children: Sequence[int], T: float, u: float,
                margin: List[float] = None) -> int:
    """The token the target "chooses" after one node, with the uniform left unscaled: walking the vocabulary in the
    order (children's tokens in node order, then every other id ascending), the first token whose cumulative
    probability exceeds u.  A child is accepted iff the choice is its token.  If `margin` is given, the distance of u
    to the nearest decision boundary is appended (how far floating-point rounding is from changing the outcome)."""
    p = target_probs(logits_row, T).tolist()
    acc = 0.0
    tried: List[int] = []
    for c in children:
        x = int(toks[c])
        if x in tried:
            continue
        lo = acc
        acc += p[x]
        tried.append(x)
        if u < acc:
            if margin is not None:
                margin.append(min(acc - u, u - lo if lo > 0.0 else 1.0))
            return x
    ts = set(tried)
    last = -1
    for y in range(len(p)):
        if y in ts:
            continue
        last = y
        lo = acc
        acc += p[y]
        if acc > u:
            if margin is not None:
                margin.append(min(acc - u, u - lo))
            return y
    if margin is not None:
        margin.append(0.0)
    return last


def choices_flat(toks: Sequence[int], logits: torch.Tensor, t: TreeTables, T: float, u: Sequence[float],
                 margins: List[float] = None) -> List[int]:
    """choice_flat for every node of the tree (the per-node form a parallel implementation computes)."""
    out = []
    for n in range(t.n_nodes):
        m: List[float] = []
        out.append(choice_flat(toks, logits[n], children_of(t, n), T, float(u[n]), m))
        if margins is not None:
            margins.append(m[0])
    return out


def accept_flat(toks: Sequence[int], logits: torch.Tensor, t: TreeTables, T: float, u: Sequence[float]):
    """Acceptance through the per-node choices: node c is matched iff its token is the choice at its parent; the
    accepted path is the deepest fully matched one; the next root is the choice at its end."""
    from oracle.amphista_oracle import Oracle
    return Oracle.accept(toks, choices_flat(toks, logits, t, T, u), t)


def sample_root(st, T: float, seed: int, seq: int = 0, logits_row: torch.Tensor = None) -> int:
    """The token after the prompt at temperature T: an inverse-transform draw from softmax(last logits / T) with the
    generator's stream 1 (step 0, node 0).  Replaces the greedy root of a freshly prefilled oracle state `st`
    (amphista_oracle.State), including the token id queued with the last pending row.  logits_row: the logits to
    draw from (default: the state's own)."""
    row = st.last_logits if logits_row is None else logits_row
    root = choice_flat([], row, [], T, uniform(seed, 0, seq, 0, stream=1))
    st.root = root
    h, _, pos = st.pending[-1]
    st.pending[-1] = (h, root, pos)
    return root
