"""The library's offline static builder (host C++) against the CPU oracle: same automaton, state
for state and transition for transition, decoded from the very image the device would receive."""
import os
import random

import numpy as np
import pytest

import oracle
import workloads as W
from paper_2411_10666_b200 import binding as sd

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "abcbc_automaton.txt")


def _edge_set(src, tok, tgt):
    return set(zip(src.tolist(), tok.tolist(), tgt.tolist()))


def _oracle_edges(S):
    out = set()
    for s in range(S.n_states):
        for t, u in S.edges(s).items():
            out.add((s, t, u))
    return out


def _compare(text, vocab):
    t = sd.sam_build_static_tables(text, vocab)
    S = oracle.Sam(text)
    link, length, endpos, deg = S.tables()
    assert len(t["length"]) == S.n_states
    assert (t["length"] == length).all() and (t["link"] == link).all()
    assert (t["min_endpos"] == endpos).all() and (t["deg"] == deg).all()
    return t, S


def test_abcbc_golden():
    t = sd.sam_build_static_tables([0, 1, 2, 1, 2], 3)
    rows = [l.split() for l in open(GOLDEN) if l[0].isdigit()]
    for f in rows:
        sid = int(f[0])
        assert (t["length"][sid], t["link"][sid], t["min_endpos"][sid]) == (int(f[1]), int(f[2]), int(f[3]))
    exp = {(int(f[0]), int(a), int(b)) for f in rows if f[4] != "-" for a, b in (e.split(">") for e in f[4].split(","))}
    assert _edge_set(t["edge_src"], t["edge_tok"], t["edge_tgt"]) == exp


@pytest.mark.parametrize("seed", range(5))
def test_random_texts_match_oracle(seed):
    rng = random.Random(seed)
    for n, vocab in [(1, 1), (2, 2), (30, 2), (300, 3), (2000, 4), (5000, 40), (20000, 3000)]:
        x = []
        while len(x) < n:
            if x and rng.random() < 0.3:
                s = rng.randrange(len(x))
                x.extend(x[s:s + rng.randint(1, 12)])
            else:
                x.append(rng.randrange(vocab))
        x = x[:n]
        t, S = _compare(x, vocab)
        assert _edge_set(t["edge_src"], t["edge_tok"], t["edge_tgt"]) == _oracle_edges(S)


def test_adversarial_texts_match_oracle():
    n = 3000
    cases = [
        [0] * n,                                            # a^n
        [0] + [1] * (n - 1),                                # 2n-1 states
        [0] + [1] * (n - 2) + [2],                          # 3n-4 transitions
        [i % 7 for i in range(n)],                          # periodic
        [v for i in range(n // 2) for v in (0, 1 + i)],     # one state with n/2 successors
        list(range(n)),                                     # all distinct
    ]
    for x in cases:
        t, S = _compare(x, max(x) + 1)
        assert _edge_set(t["edge_src"], t["edge_tok"], t["edge_tgt"]) == _oracle_edges(S)


def test_workload_corpus_matches_oracle():
    spec = W.scaled(W.SPECS["c2"], corpus_len=300_000)
    corpus = W.make_corpus(spec)
    t, S = _compare(corpus, spec.vocab)
    assert len(t["edge_src"]) == S.n_transitions
    # spot-check transitions of the busiest states and a random sample
    rng = random.Random(1)
    by_src = {}
    for s, k, u in zip(t["edge_src"].tolist(), t["edge_tok"].tolist(), t["edge_tgt"].tolist()):
        by_src.setdefault(s, {})[k] = u
    busiest = np.argsort(t["deg"])[-20:].tolist()
    for s in busiest + [rng.randrange(S.n_states) for _ in range(2000)]:
        assert by_src.get(s, {}) == S.edges(s)


def test_argument_errors():
    L = sd.lib()
    bad = np.array([0, 5, 1], dtype=np.int32)
    with pytest.raises(sd.SamError) as e:
        sd.sam_build_static_tables(bad, 3)                 # token out of range
    assert e.value.code == -1
    with pytest.raises(sd.SamError):
        sd.sam_build_static_tables(np.zeros(0, dtype=np.int32), 3)
    assert L.sam_strerror(-4) == b"workspace too small or misaligned"
