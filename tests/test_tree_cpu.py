"""Pins for freq, top-k successors and the Prim tree draft of the oracle (Appendix A.1/A.2,
Algorithms 4 and 5): occurrence counts by exhaustive search, hand-worked example, best-first property."""
import itertools
import random

import numpy as np

import oracle
from oracle import tree


def _occurrences(x, w):
    n, m = len(x), len(w)
    return sum(1 for i in range(n - m + 1) if x[i:i + m] == w)


def _longest_string(S, x, s):
    e, l = S.min_endpos(s), S.length(s)
    return x[e - l:e]


def test_freq_is_the_number_of_occurrences():
    rng = random.Random(4)
    for _ in range(60):
        n = rng.randint(1, 40)
        x = [rng.randrange(rng.randint(1, 4)) for _ in range(n)]
        S = oracle.Sam(x)
        f = S.freq()
        assert f[0] == n
        for s in range(1, S.n_states):
            assert f[s] == _occurrences(x, _longest_string(S, x, s)), (x, s)
        # a state's occurrences continue into its successors, except the one at the end of the text
        for s in range(1, S.n_states):
            w = _longest_string(S, x, s)
            at_end = 1 if x[n - len(w):] == w else 0
            assert f[s] == at_end + sum(f[u] for u in S.edges(s).values())


def test_abcbc_freq_and_topk():
    # A=0 B=1 C=2; states as in tests/golden/abcbc_automaton.txt
    x = [0, 1, 2, 1, 2]
    S = oracle.Sam(x)
    f = S.freq()
    # "A" once, "AB" once, "ABC" once, "ABCB" once, "B" twice (clone 5), "ABCBC" once, "BC"/"C" twice (clone 7)
    assert f.tolist() == [5, 1, 1, 1, 1, 2, 1, 2]
    assert S.topk(f, 0, 2) == [(1, 5), (2, 7)]            # B and C occur twice, A once; tie -> smaller token
    assert S.topk(f, 0, 3) == [(1, 5), (2, 7), (0, 1)]
    assert S.topk(f, 5, 4) == [(2, 7)] and S.topk(f, 6, 4) == []
    # Prim from the state of "B" (5), start token B: B(1.0) -> C(2/2) -> B(1/2) -> C(1/2 * 1/1)
    toks, par, pr = tree.prim_tree(S, f, 5, 1, 8, 2)
    assert toks == [1, 2, 1, 2] and par == [-1, 0, 1, 2]
    assert [float(p) for p in pr] == [1.0, 1.0, 0.5, 0.5]


def test_topk_is_the_k_most_frequent_successors():
    rng = random.Random(9)
    for _ in range(40):
        x = [rng.randrange(5) for _ in range(rng.randint(5, 80))]
        S = oracle.Sam(x)
        f = S.freq()
        for s in range(S.n_states):
            ed = sorted(S.edges(s).items(), key=lambda tu: (-f[tu[1]], tu[0]))
            for k in (1, 2, 4):
                assert S.topk(f, s, k) == ed[:k]


def test_prim_pops_the_most_probable_nodes_first():
    """Path probabilities only shrink along a path, so best-first expansion returns nodes in
    non-increasing probability, and (absent ties at the cut) exactly the max_size most probable
    nodes of the full top-k tree."""
    rng = random.Random(2)
    f32 = np.float32
    for _ in range(30):
        x = [rng.randrange(3) for _ in range(rng.randint(8, 60))]
        S = oracle.Sam(x)
        f = S.freq()
        k, max_size = rng.randint(1, 3), rng.randint(1, 12)
        s = rng.randrange(1, S.n_states)
        toks, par, pr = tree.prim_tree(S, f, s, 9, max_size, k)
        assert all(pr[i] >= pr[i + 1] for i in range(len(pr) - 1))
        assert par[0] == -1 and all(0 <= par[i] < i for i in range(1, len(par)))
        # enumerate the full tree to depth max_size with the same float32 arithmetic
        nodes = []                                            # (p, path of tokens)
        frontier = [(f32(1.0), s, (9,))]
        for _depth in range(max_size):
            nxt = []
            for p, st, path in frontier:
                nodes.append((p, path))
                for t_n, s_n in S.topk(f, st, k):
                    nxt.append((f32(p * (f32(f[s_n]) / f32(f[st]))), s_n, path + (t_n,)))
            frontier = nxt
        nodes.sort(key=lambda t: -float(t[0]))
        if len(nodes) > len(toks) and nodes[len(toks) - 1][0] == nodes[len(toks)][0]:
            continue                                          # a tie at the cut: several sets are right
        # rebuild each popped node's path and compare as sets
        paths = []
        for i in range(len(toks)):
            path, j = [], i
            while j >= 0:
                path.append(toks[j]); j = par[j]
            paths.append(tuple(reversed(path)))
        assert len(toks) == min(max_size, len(nodes))
        assert set(paths) == {path for _, path in nodes[:len(toks)]}
