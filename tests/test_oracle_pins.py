"""Pins for the CPU oracle: it is checked against things other than itself — the worked example
of the paper's Figure 2 string, exhaustive search, counting identities and closed forms."""
import os
import random

import numpy as np
import pytest

import oracle
from oracle import bruteforce as bf

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "abcbc_automaton.txt")


def _parse_golden():
    states, transfers, dynamic = [], [], []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        f = line.split()
        lst = lambda s: [] if s == "-" else [int(v) for v in s.split(",")]
        if f[0] == "T":
            transfers.append((int(f[1]), int(f[2]), int(f[3]), int(f[4]), int(f[5]), lst(f[6])))
        elif f[0] == "D":
            dynamic.append((int(f[1]), int(f[2]), int(f[3]), int(f[4]), lst(f[5])))
        else:
            nxt = {} if f[4] == "-" else {int(a): int(b) for a, b in (e.split(">") for e in f[4].split(","))}
            states.append((int(f[0]), int(f[1]), int(f[2]), int(f[3]), nxt))
    return states, transfers, dynamic


def test_abcbc_automaton_matches_hand_derivation():
    states, _, _ = _parse_golden()
    S = oracle.Sam([0, 1, 2, 1, 2])
    assert S.n_states == len(states) == 8
    assert S.n_transitions == sum(len(s[4]) for s in states) == 9
    for sid, length, link, endpos, nxt in states:
        assert (S.length(sid), S.link(sid), S.min_endpos(sid)) == (length, link, endpos), sid
        assert S.edges(sid) == nxt, sid
    assert S.last == 6


def test_abcbc_static_transfer_and_draft():
    _, transfers, _ = _parse_golden()
    T = [0, 1, 2, 1, 2]
    S = oracle.Sam(T)
    s, l = 0, 0
    for tok, exp_s, exp_l, exp_p, exp_moves, exp_draft in transfers:
        s, l, link_moves, _ = S.transfer(tok, s, l)
        assert (s, l, S.min_endpos(s), link_moves) == (exp_s, exp_l, exp_p, exp_moves)
        p = S.min_endpos(s)
        assert T[p:p + 3] == exp_draft
    # the same first row through the batched step (the dynamic side has nothing to match yet)
    B = oracle.Batch(S, T, 1, 3, 16)
    out = B.step([[1]], [1], 3)
    assert out.match_len.tolist() == [[1, 0]] and out.source.tolist() == [1]
    assert out.draft_tokens.tolist() == [[2, 1, 2]] and out.state.tolist() == [[5, 0]]


def test_abcbc_dynamic_transfer_then_expand():
    _, _, dynamic = _parse_golden()
    B = oracle.Batch(None, None, 1, 3, 16)
    for tok, exp_s, exp_l, exp_p, exp_draft in dynamic:
        out = B.step([[tok]], [1], 3)
        assert out.match_len[0, 1] == exp_l and out.state[0, 1] == exp_s
        assert B.dynamic(0).min_endpos(exp_s) == exp_p
        dl = int(out.draft_len[0])
        assert out.draft_tokens[0, :dl].tolist() == exp_draft
        assert (out.draft_tokens[0, dl:] == -1).all()
        assert out.source[0] == (2 if exp_l > 0 else 0)


def _random_text(rng, n, vocab, copy_p=0.3):
    x = []
    while len(x) < n:
        if x and rng.random() < copy_p:
            s = rng.randrange(len(x))
            ln = rng.randint(1, 8)
            for k in range(ln):
                if len(x) < n:
                    x.append(x[s + k] if s + k < len(x) else rng.randrange(vocab))
        else:
            x.append(rng.randrange(vocab))
    return x


@pytest.mark.parametrize("seed", range(8))
def test_step_equals_exhaustive_search(seed):
    """>= 10 000 tiny random cases in total: every reported quantity equals its definition."""
    rng = random.Random(1000 + seed)
    n_cases = 0
    for _ in range(160):
        vocab = rng.randint(2, 4)
        N = rng.randint(0, 64)
        k_total = rng.randint(1, 64)
        L = rng.randint(1, 8)
        l_bias = rng.randint(0, 2)
        min_match = rng.randint(0, 3)
        corpus = _random_text(rng, N, vocab)
        x = _random_text(rng, k_total, vocab)
        if corpus and rng.random() < 0.5:            # splice corpus spans into x so static wins sometimes
            s = rng.randrange(len(corpus)); ln = rng.randint(1, 12)
            at = rng.randrange(len(x))
            x[at:at + ln] = corpus[s:s + ln]
            x = x[:k_total]
        S = oracle.Sam(corpus) if N > 0 else None
        B = oracle.Batch(S, corpus if N > 0 else None, 1, vocab, k_total, l_bias, min_match)
        k = 0
        while k < len(x):
            m = min(rng.randint(0, 5), len(x) - k)
            stride = max(m, 1)
            toks = x[k:k + m] + [0] * (stride - m)
            out = B.step([toks], [m], L)
            k += m
            exp = bf.retrieve(corpus if N > 0 else None, x, k, L, l_bias, min_match)
            assert out.status[0] == 0
            assert out.match_len[0].tolist() == [exp["l1"], exp["l2"]], (corpus, x[:k])
            assert out.source[0] == exp["source"]
            dl = int(out.draft_len[0])
            assert out.draft_tokens[0, :dl].tolist() == exp["draft"], (corpus, x[:k], exp)
            assert (out.draft_tokens[0, dl:] == -1).all()
            # the reported states carry the earliest end positions
            if S is not None:
                assert S.min_endpos(int(out.state[0, 0])) == exp["e1"]
            assert B.dynamic(0).min_endpos(int(out.state[0, 1])) == exp["e2"]
            n_cases += 1
    assert n_cases >= 1250


@pytest.mark.parametrize("seed", range(6))
def test_states_are_the_endpos_classes(seed):
    """Non-root states <-> classes of substrings with equal end-position sets; each carries the
    class's longest length and earliest end position; distinct substrings = sum(len - len[link])."""
    rng = random.Random(77 + seed)
    for _ in range(40):
        n = rng.randint(1, 28)
        x = _random_text(rng, n, rng.randint(1, 4))
        S = oracle.Sam(x)
        link, length, endpos, deg = S.tables()
        classes = bf.endpos_classes(x)
        got = sorted((int(length[s]), int(endpos[s])) for s in range(1, S.n_states))
        assert got == sorted(classes.values())
        assert int((length[1:] - length[link[1:]]).sum()) == bf.distinct_substrings(x)
        # every transition s -t-> u: appending t to s's longest string gives a string of class u
        for s in range(S.n_states):
            for t, u in S.edges(s).items():
                assert length[u] >= length[s] + 1
                assert length[link[u]] <= (length[link[s]] if s else -1) + 1


@pytest.mark.parametrize("seed", range(4))
def test_size_and_structure_invariants(seed):
    rng = random.Random(5 + seed)
    for n, vocab in [(2, 2), (3, 2), (50, 2), (400, 3), (3000, 50), (20000, 1000)]:
        x = _random_text(rng, n, vocab)
        S = oracle.Sam(x)
        link, length, endpos, deg = S.tables()
        assert S.err == 0
        assert S.n_states <= 2 * n - 1 if n >= 2 else S.n_states == n + 1
        if n >= 3:
            assert S.n_transitions <= 3 * n - 4
        assert int(deg.sum()) == S.n_transitions
        assert link[0] == -1 and length[0] == 0 and endpos[0] == 0
        assert (length[link[1:]] < length[1:]).all()
        assert (length[1:] <= endpos[1:]).all() and (endpos[1:] <= n).all()
        # the string ending at min_endpos with the state's length really is followed as recorded:
        # walking the text from the root reaches a state whose min_endpos is <= the position
        s, l = 0, 0
        for i, t in enumerate(x):
            s, l, _, _ = S.transfer(t, s, l)
            assert l == i + 1 and endpos[s] <= i + 1


def test_worst_case_sizes_are_attained():
    # a b^(n-1) attains 2n-1 states; a b^(n-2) c attains 3n-4 transitions (Blumer et al.)
    for n in (3, 5, 17, 64):
        x = [0] + [1] * (n - 1)
        assert oracle.Sam(x).n_states == 2 * n - 1
        y = [0] + [1] * (n - 2) + [2]
        assert oracle.Sam(y).n_transitions == 3 * n - 4


def test_closed_forms():
    # a^n: n+1 states, no clones; dynamic l2 = k-1 with end position k-1 and a 1-token draft
    n = 40
    S = oracle.Sam([7] * n)
    assert S.n_states == n + 1 and S.counters()["clones"] == 0
    B = oracle.Batch(None, None, 1, 8, n)
    for k in range(1, n + 1):
        out = B.step([[7]], [1], 5)
        assert out.match_len[0, 1] == k - 1
        if k > 1:
            assert B.dynamic(0).min_endpos(int(out.state[0, 1])) == k - 1
            assert out.draft_len[0] == 1 and out.draft_tokens[0, 0] == 7
    # all-distinct tokens: n+1 states, l2 = 0 always, never a draft
    S = oracle.Sam(list(range(n)))
    assert S.n_states == n + 1 and S.n_transitions == 2 * n - 1   # a chain of n edges plus the root's other n-1
    B = oracle.Batch(None, None, 1, n, n)
    for k in range(n):
        out = B.step([[k]], [1], 5)
        assert out.match_len[0, 1] == 0 and out.source[0] == 0 and out.draft_len[0] == 0
    # exact period p with distinct period tokens: l2 = k - p once k > p; draft continues the period
    p = 5
    B = oracle.Batch(None, None, 1, p, 64)
    for k in range(1, 41):
        out = B.step([[(k - 1) % p]], [1], 4)
        assert out.match_len[0, 1] == max(0, k - p)
        if k > p:
            dl = int(out.draft_len[0])
            assert dl == min(4, p)                      # the earliest occurrence ends at k-p; p tokens follow it
            assert out.draft_tokens[0, :dl].tolist() == [(k + i) % p for i in range(dl)]
    # a stream that is a verbatim corpus prefix: l1 = k, e1 = k, draft = the next corpus tokens
    rng = random.Random(3)
    corpus = [rng.randrange(50) for _ in range(300)]
    S = oracle.Sam(corpus)
    B = oracle.Batch(S, corpus, 1, 50, 300, l_bias=0)
    for k in range(1, 200):
        out = B.step([[corpus[k - 1]]], [1], 6)
        assert out.match_len[0, 0] == k
        if out.source[0] == 1:
            assert out.draft_tokens[0].tolist() == corpus[k:k + 6]


def test_transfer_cost_bound():
    """Appendix A.3: over a stream of L tokens the link and next moves total at most 2L and the
    match length rises by at most one per token."""
    rng = random.Random(11)
    corpus = _random_text(rng, 5000, 6)
    S = oracle.Sam(corpus)
    x = _random_text(rng, 4000, 6)
    s = l = 0
    total = 0
    for t in x:
        s2, l2, lm, nm = S.transfer(t, s, l)
        assert l2 <= l + 1 and nm <= 1
        total += lm + nm
        s, l = s2, l2
    assert total <= 2 * len(x)


def test_boundary_conventions():
    B = oracle.Batch(None, None, 4, 10, 4)
    out = B.step([[1, 2, 3], [1, 10, 0], [1, 2, 3], [1, 2, 3]], [3, 2, 4, 3], 2)
    assert out.status.tolist() == [0, 3, 4, 0]
    out = B.step([[1, 2], [1, 1], [1, 1], [5, 0]], [2, 1, 1, 1], 2)
    assert out.status.tolist() == [1, 3, 4, 0]            # sticky, and 3+2 > max_seq_len
    assert out.draft_len.tolist()[:3] == [0, 0, 0] and (out.draft_tokens[:3] == -1).all()
    # count 0 re-emits the current draft
    B = oracle.Batch(None, None, 1, 10, 16)
    a = B.step([[1, 2, 1, 2, 1]], [5], 3)
    b = B.step([[0, 0, 0, 0, 0]], [0], 3)
    assert a.draft_tokens.tolist() == b.draft_tokens.tolist() and a.match_len.tolist() == b.match_len.tolist()
    # reset forgets
    B.reset(0)
    c = B.step([[1]], [1], 3)
    assert c.match_len.tolist() == [[0, 0]]


def test_workload_scale_self_certification():
    """On a generated workload every reported match really is a suffix occurrence at the reported
    end position, and the draft is the continuation there."""
    import workloads as W
    spec = W.scaled(W.SPECS["tiny"], corpus_len=20000, batch=3, prompt_len=64, gen_len=200)
    w = W.make(spec)
    S = oracle.Sam(w.corpus)
    B = oracle.Batch(S, w.corpus, spec.batch, spec.vocab, spec.prompt_len + spec.gen_len)
    L = spec.draft_len
    out = B.step(w.prompts, [spec.prompt_len] * spec.batch, L)
    pos = [spec.prompt_len] * spec.batch
    n_static = 0
    for s in range(w.n_steps):
        out = B.step(w.new_tokens[s], w.counts[s], L)
        for b in range(spec.batch):
            pos[b] += int(w.counts[s, b])
            x = w.seqs[b, :pos[b]]
            l1, l2 = (int(v) for v in out.match_len[b])
            e1 = S.min_endpos(int(out.state[b, 0]))
            e2 = B.dynamic(b).min_endpos(int(out.state[b, 1]))
            assert (w.corpus[e1 - l1:e1] == x[len(x) - l1:]).all()
            assert (x[e2 - l2:e2] == x[len(x) - l2:]).all() and (e2 < len(x) or l2 == 0)
            dl = int(out.draft_len[b])
            if out.source[b] == 1:
                n_static += 1
                assert (out.draft_tokens[b, :dl] == w.corpus[e1:e1 + dl]).all()
            elif out.source[b] == 2:
                assert (out.draft_tokens[b, :dl] == x[e2:e2 + dl]).all()
    assert n_static > 0
    assert B.counters()["tokens"] == spec.batch * (spec.prompt_len + spec.gen_len)


def test_stop_token_cuts_the_draft_at_a_document_separator():
    """Section 3.1 joins the corpus' documents with an EOS symbol; with that symbol as the stop token a
    draft is the definition's draft cut before its first EOS."""
    rng = random.Random(21)
    EOS = 0
    for _ in range(60):
        docs = [[rng.randrange(1, 5) for _ in range(rng.randint(1, 9))] for _ in range(rng.randint(1, 8))]
        corpus = [t for d in docs for t in d + [EOS]]
        x = [rng.randrange(0, 5) for _ in range(rng.randint(1, 30))]
        L = rng.randint(1, 8)
        B = oracle.Batch(oracle.Sam(corpus), corpus, 1, 5, len(x), 0, 1, EOS)
        for k in range(1, len(x) + 1):
            out = B.step([[x[k - 1]]], [1], L)
            exp = bf.retrieve(corpus, x, k, L)
            d = exp["draft"]
            if EOS in d:
                d = d[:d.index(EOS)]
            dl = int(out.draft_len[0])
            assert out.source[0] == exp["source"]
            assert out.draft_tokens[0, :dl].tolist() == d and (out.draft_tokens[0, dl:] == -1).all()
            assert EOS not in out.draft_tokens[0, :dl].tolist()


@pytest.mark.parametrize("threads", [1, 3])
def test_run_of_many_steps_equals_the_definition_and_the_single_steps(threads):
    """Batch.run (all steps of a schedule in one call: what the timed CPU baseline executes) leaves,
    for every sequence, exactly what exhaustive search gives for its whole text, and the same
    outputs, automata and operation counts as feeding the steps one by one."""
    rng = random.Random(77 + threads)
    for _ in range(25):
        vocab, B, K, L = rng.randint(2, 4), rng.randint(1, 4), rng.randint(1, 5), rng.randint(1, 6)
        N, n_steps = rng.randint(0, 50), rng.randint(1, 14)
        l_bias, min_match = rng.randint(0, 2), rng.randint(0, 2)
        corpus = _random_text(rng, N, vocab)
        counts = np.array([[rng.randint(0, K) for _ in range(B)] for _ in range(n_steps)], dtype=np.int32)
        toks = np.array([[[rng.randrange(vocab) for _ in range(K)] for _ in range(B)] for _ in range(n_steps)], dtype=np.int32)
        total = int(counts.sum(axis=0).max()) + 1
        S = oracle.Sam(corpus) if N else None
        whole = oracle.Batch(S, corpus if N else None, B, vocab, total, l_bias, min_match)
        out = whole.run(toks, counts, L, threads)
        single = oracle.Batch(S, corpus if N else None, B, vocab, total, l_bias, min_match)
        for s in range(n_steps):
            ref = single.step(toks[s], counts[s], L)
        for k in ("draft_tokens", "draft_len", "match_len", "source", "state", "status"):
            assert np.array_equal(getattr(out, k), getattr(ref, k)), k
        assert whole.counters() == single.counters()
        for b in range(B):
            x = [int(t) for s in range(n_steps) for t in toks[s, b, :counts[s, b]]]
            exp = bf.retrieve(corpus if N else None, x, len(x), L, l_bias, min_match)
            assert out.match_len[b].tolist() == [exp["l1"], exp["l2"]] and out.source[b] == exp["source"]
            assert out.draft_tokens[b, :out.draft_len[b]].tolist() == exp["draft"]
            assert whole.seq_len(b) == len(x) and whole.dynamic(b).n_states == single.dynamic(b).n_states
