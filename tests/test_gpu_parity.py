"""GPU parity: the CUDA library against the CPU oracle, bit for bit, through the C ABI."""
import os
import random

import numpy as np
import pytest

import oracle
import workloads as W
from _parity import assert_dynamic_automata_equal, assert_same, gpu_run, oracle_run

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "abcbc_automaton.txt")


@pytest.fixture(scope="module")
def P():
    import torch
    assert torch.cuda.is_available(), "the gpu tests need a CUDA device"
    import paper_2411_10666_b200 as pkg
    pkg.lib()
    return pkg


def _steps_from_text(x, rng, kmax):
    """Split a token list into (new_tokens [S,1,K], counts [S,1])."""
    rows, cnts, k = [], [], 0
    while k < len(x):
        m = min(rng.randint(0, kmax), len(x) - k)
        rows.append(x[k:k + m] + [-1] * (kmax - m))
        cnts.append(m)
        k += m
    return np.array(rows, dtype=np.int32).reshape(-1, 1, kmax), np.array(cnts, dtype=np.int32).reshape(-1, 1)


def test_abcbc_golden(P):
    T = np.array([0, 1, 2, 1, 2], dtype=np.int32)
    st = P.StaticSam.build(T, 3)
    tb = P.binding.sam_static_tables(st.handle)
    rows = [l.split() for l in open(GOLDEN) if l[0].isdigit()]
    for f in rows:
        sid = int(f[0])
        assert (tb["length"][sid], tb["link"][sid], tb["min_endpos"][sid]) == (int(f[1]), int(f[2]), int(f[3]))
        exp = {} if f[4] == "-" else {int(a): int(b) for a, b in (e.split(">") for e in f[4].split(","))}
        assert P.binding.sam_static_state(st.handle, sid)["next"] == exp
    # static stream B,C,B,A with a disabled dynamic side cannot be had; use l_bias=0 rows where static wins
    trans = [l.split() for l in open(GOLDEN) if l.startswith("T ")]
    dyn = [l.split() for l in open(GOLDEN) if l.startswith("D ")]
    lst = lambda s: [] if s == "-" else [int(v) for v in s.split(",")]
    toks = np.array([[[int(f[1])]] for f in trans], dtype=np.int32)
    res, _ = gpu_run(P, st, 3, np.zeros((1, 0), np.int32), toks, np.ones((len(trans), 1), np.int32), 3, 16)
    for i, f in enumerate(trans):
        assert res["state"][i, 0, 0] == int(f[2]) and res["match_len"][i, 0, 0] == int(f[3])
        if res["source"][i, 0] == 1:
            d = lst(f[6])
            assert res["draft_tokens"][i, 0, :len(d)].tolist() == d and res["draft_len"][i, 0] == len(d)
    assert (res["source"][:, 0] == 1).sum() >= 3
    toks = np.array([[[int(f[1])]] for f in dyn], dtype=np.int32)
    res, batch = gpu_run(P, None, 3, np.zeros((1, 0), np.int32), toks, np.ones((len(dyn), 1), np.int32), 3, 16)
    for i, f in enumerate(dyn):
        assert res["state"][i, 0, 1] == int(f[2]) and res["match_len"][i, 0, 1] == int(f[3])
        d = lst(f[5])
        assert res["draft_len"][i, 0] == len(d) and res["draft_tokens"][i, 0, :len(d)].tolist() == d
    d = batch.dump(0, 16, 16)
    assert d["n_states"] == 8 and d["n_edges"] == 9
    for f in rows:
        sid = int(f[0])
        assert (d["length"][sid], d["link"][sid], d["min_endpos"][sid]) == (int(f[1]), int(f[2]), int(f[3]))


def _rand_text(rng, n, vocab, copy_p):
    x = []
    while len(x) < n:
        if x and rng.random() < copy_p:
            s = rng.randrange(len(x))
            x.extend(x[s:s + rng.randint(1, 20)])
        else:
            x.append(rng.randrange(vocab))
    return x[:n]


@pytest.mark.parametrize("seed", range(6))
def test_random_small_cases_all_outputs_and_automata(P, seed):
    rng = random.Random(100 + seed)
    for case in range(6):
        vocab = rng.choice([2, 3, 5, 50, 1000])
        N = rng.choice([1, 7, 200, 3000])
        n = rng.choice([1, 33, 257, 900])
        L = rng.choice([1, 5, 32, 33, 128])
        kmax = rng.choice([1, 4, 40])
        l_bias, min_match = rng.choice([(0, 1), (0, 0), (2, 1), (0, 3), (5, 5)])
        corpus = np.array(_rand_text(rng, N, vocab, 0.3), dtype=np.int32)
        B = rng.choice([1, 3])
        texts = []
        for b in range(B):
            x = _rand_text(rng, n, vocab, 0.4)
            if N > 20 and rng.random() < 0.7:                # splice corpus spans in
                for _ in range(3):
                    s = rng.randrange(N); ln = rng.randint(2, 40); at = rng.randrange(n)
                    x[at:at + ln] = corpus[s:s + ln].tolist()
                x = x[:n]
            texts.append(x + [0] * (n - len(x)))
        # a common step schedule for all slots
        rows, cnts, k = [], [], 0
        while k < n:
            m = min(rng.randint(0, kmax), n - k)
            rows.append([t[k:k + m] + [-1] * (kmax - m) for t in texts])
            cnts.append([m] * B)
            k += m
        nt = np.array(rows, dtype=np.int32).reshape(len(rows), B, kmax)
        ct = np.array(cnts, dtype=np.int32).reshape(len(rows), B)
        empty = np.zeros((B, 0), np.int32)
        st = P.StaticSam.build(corpus, vocab)
        ref, ob, _ = oracle_run(corpus, vocab, empty, nt, ct, L, n, l_bias, min_match)
        got, batch = gpu_run(P, st, vocab, empty, nt, ct, L, n, l_bias, min_match)
        assert_same(got, ref, "seed %d case %d" % (seed, case))
        assert_dynamic_automata_equal(batch, ob, range(B), n)
        assert (got["status"] == 0).all()


def test_adversarial_sequences(P):
    n = 1500
    cases = [
        [0] * n,
        [0] + [1] * (n - 1),
        [0] + [1] * (n - 2) + [2],
        [i % 7 for i in range(n)],
        [v for i in range(n // 2) for v in (0, 1 + i)],       # a state with n/2 successors: block growth
        list(range(n)),
        [(i * i) % 11 for i in range(n)],
        [v for i in range(n // 3) for v in (0, 1, 2 + i)],
    ]
    rng = random.Random(5)
    for x in cases:
        vocab = max(x) + 1
        nt, ct = _steps_from_text(x, rng, 64)
        empty = np.zeros((1, 0), np.int32)
        ref, ob, _ = oracle_run(None, vocab, empty, nt, ct, 8, n)
        got, batch = gpu_run(P, None, vocab, empty, nt, ct, 8, n)
        assert_same(got, ref)
        assert_dynamic_automata_equal(batch, ob, [0], n)


def test_repeated_passages_dynamic_runs(P):
    """Passages repeated once, twice and three times, with contexts of different lengths before them,
    self-overlapping repeats, periodic stretches and repeats of the very beginning of the text: the
    cases in which the step kernel extends several cloning tokens side by side.  Every output and the
    whole automaton equal the oracle's."""
    rng = random.Random(11)
    n = 1400
    for vocab, kmax in [(3, 40), (6, 32), (50, 17), (2000, 40), (2000, 3)]:
        x = [rng.randrange(vocab) for _ in range(60)]
        while len(x) < n:
            kind = rng.random()
            if kind < 0.45:                                   # repeat an earlier span (again and again)
                s = rng.randrange(len(x)); ln = rng.randint(2, 70)
                x.extend(x[s:s + ln])
            elif kind < 0.55:                                 # overlap: the span runs into itself
                back = rng.randint(1, 12); ln = rng.randint(5, 60)
                for _ in range(ln):
                    x.append(x[-back])
            elif kind < 0.62:                                 # the beginning of the text once more
                x.extend(x[:rng.randint(2, 50)])
            else:
                x.extend(rng.randrange(vocab) for _ in range(rng.randint(1, 6)))
        x = x[:n]
        nt, ct = _steps_from_text(x, rng, kmax)
        empty = np.zeros((1, 0), np.int32)
        for L in (1, 32):
            ref, ob, _ = oracle_run(None, vocab, empty, nt, ct, L, n)
            got, batch = gpu_run(P, None, vocab, empty, nt, ct, L, n)
            assert_same(got, ref, "vocab %d kmax %d L %d" % (vocab, kmax, L))
            assert_dynamic_automata_equal(batch, ob, [0], n)
            assert (got["status"] == 0).all()


def test_periodic_passages_and_their_breaks(P):
    """Periodic stretches (period 1 to 9, up to several hundred tokens, also re-entered later) that break off
    with a token the passage never had: Expand then walks down the passage's suffixes a period at a time and
    adds a transition at every state — the longest walks the workloads contain (50 to 100 suffix links).
    Every output and the whole automaton equal the oracle's."""
    rng = random.Random(21)
    n = 2600
    for vocab, kmax in [(3, 16), (12, 40), (300, 7), (5000, 64)]:
        x, motifs = [], []
        while len(x) < n:
            kind = rng.random()
            if kind < 0.5:
                period = rng.randint(1, 9)
                motif = rng.choice(motifs) if motifs and rng.random() < 0.4 else [rng.randrange(vocab) for _ in range(period)]
                motifs.append(motif)
                reps = rng.randint(2, 400 // len(motif))
                x.extend((motif * reps)[:rng.randint(len(motif) + 1, len(motif) * reps)])
            elif kind < 0.7 and len(x) > 20:
                back = rng.randint(1, 9); ln = rng.randint(10, 300)     # a copy that runs into itself
                for _ in range(ln):
                    x.append(x[-back])
            else:
                x.extend(rng.randrange(vocab) for _ in range(rng.randint(1, 5)))
        x = x[:n]
        nt, ct = _steps_from_text(x, rng, kmax)
        empty = np.zeros((1, 0), np.int32)
        ref, ob, _ = oracle_run(None, vocab, empty, nt, ct, 8, n)
        got, batch = gpu_run(P, None, vocab, empty, nt, ct, 8, n)
        assert_same(got, ref, "vocab %d kmax %d" % (vocab, kmax))
        assert_dynamic_automata_equal(batch, ob, [0], n)
        assert (got["status"] == 0).all()


def test_static_matches_in_prefix_states(P):
    """Sequences that copy long stretches of the corpus (the match soon sits in the state of a whole
    corpus prefix, so the static side advances it by comparing with the corpus), including stretches
    that run to the corpus' end, that break off after any number of tokens, and corpora with internal
    repeats.  The periodic corpora ("abab...", "ababc", period 3 with a tail) have prefix states that
    occur several times and have two transitions — the state of "ab" in "ababc" goes on with a and
    with c — so tokens that leave the corpus' own continuation from such a state are covered."""
    rng = random.Random(12)
    made = []
    for vocab, N in [(4, 300), (40, 5000), (3000, 20000)]:
        corpus = []
        while len(corpus) < N:
            if corpus and rng.random() < 0.2:
                s = rng.randrange(len(corpus)); corpus.extend(corpus[s:s + rng.randint(3, 40)])
            else:
                corpus.append(rng.randrange(vocab))
        made.append((vocab, corpus[:N]))
    made.append((3, [0, 1, 0, 1, 2]))                                     # ababc
    made.append((3, [0, 1] * 40))                                         # (ab)^40
    made.append((3, [0, 1] * 30 + [2] + [0, 1] * 20 + [2, 2, 0]))         # two periodic stretches
    made.append((4, [0, 1, 2] * 25 + [3] + [0, 1, 2, 0, 1, 3]))           # period 3 with tails
    for vocab, corpus in made:
        N = len(corpus)
        corpus = np.array(corpus, dtype=np.int32)
        n = 900 if N > 200 else 400
        texts = []
        for b in range(3):
            x = []
            while len(x) < n:
                r = rng.random()
                if r < 0.5:
                    s = rng.randrange(N); x.extend(corpus[s:s + rng.randint(1, 90)].tolist())
                elif r < 0.6:
                    x.extend(corpus[N - rng.randint(1, min(50, N)):].tolist())  # up to the corpus' end
                elif r < 0.7:
                    x.extend(corpus[:rng.randint(1, min(60, N))].tolist())      # from the corpus' start: prefix states
                else:
                    x.extend(rng.randrange(vocab) for _ in range(rng.randint(1, 4)))
            texts.append(x[:n])
        kmax = 32
        rows, cnts, k = [], [], 0
        while k < n:
            m = min(rng.randint(0, kmax), n - k)
            rows.append([t[k:k + m] + [-1] * (kmax - m) for t in texts]); cnts.append([m] * 3); k += m
        nt = np.array(rows, dtype=np.int32).reshape(len(rows), 3, kmax)
        ct = np.array(cnts, dtype=np.int32).reshape(len(rows), 3)
        empty = np.zeros((3, 0), np.int32)
        st = P.StaticSam.build(corpus, vocab)
        for L, stop in ((8, -1), (40, 1)):
            ref, ob, _ = oracle_run(corpus, vocab, empty, nt, ct, L, n, stop_token=stop)
            got, batch = gpu_run(P, st, vocab, empty, nt, ct, L, n, stop_token=stop)
            assert_same(got, ref, "vocab %d N %d L %d" % (vocab, N, L))
            assert got["match_len"][:, :, 0].max() >= min(N, 8)
            assert N < 200 or (got["source"] == 1).any()      # in the short periodic corpora the own text ties or wins


def test_large_batch_is_ordered_by_token_count(P):
    """A batch above the size at which the step first sorts its slots by token count (two kernels per
    step): the results are the same as the oracle's, slot for slot."""
    spec = W.scaled(W.SPECS["c5"], 150_000, 1700, 48, 80)
    w = W.make(spec)
    L, msl = spec.draft_len, spec.prompt_len + spec.gen_len
    st = P.StaticSam.build(w.corpus, spec.vocab)
    ref, ob, _ = oracle_run(w.corpus, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl, threads=4)
    got, batch = gpu_run(P, st, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl)
    assert batch.launches_per_step() == 2
    assert_same(got, ref, "ordered batch")
    assert (got["status"] == 0).all()
    assert_dynamic_automata_equal(batch, ob, [0, 777, spec.batch - 1], msl)


@pytest.mark.parametrize("l_bias,min_match,stop", [(0, 1, -1), (2, 3, 7)])
def test_split_step_for_very_large_batches(P, l_bias, min_match, stop):
    """From 8192 slots on a step runs as the split kernel: the static side of a slot in one block (a lane
    or a warp of it, by token count), the dynamic side in another, the outputs written by whichever
    finishes last.  Every output of every step equals the oracle's, slot for slot, and so do sampled
    dynamic automata; counts include 0 and the prompt is fed in one step (hundreds of tokens per slot)."""
    spec = W.scaled(W.SPECS["c5"], 200_000, 8300, 130, 90)
    w = W.make(spec)
    L, msl = spec.draft_len, spec.prompt_len + spec.gen_len
    counts = w.counts.copy()
    counts[3, ::7] = 0                                      # some slots sit a step out (their tokens are dropped)
    st = P.StaticSam.build(w.corpus, spec.vocab)
    ref, ob, _ = oracle_run(w.corpus, spec.vocab, w.prompts, w.new_tokens, counts, L, msl, l_bias, min_match,
                            threads=8, stop_token=stop)
    got, batch = gpu_run(P, st, spec.vocab, w.prompts, w.new_tokens, counts, L, msl, l_bias, min_match, stop_token=stop)
    assert batch.launches_per_step() == 2
    assert_same(got, ref, "split step")
    assert (got["status"] == 0).all()
    assert (got["source"] == 1).any() and (got["source"] == 2).any()
    assert_dynamic_automata_equal(batch, ob, [0, 4097, spec.batch - 1], msl)


def test_very_large_batch_without_a_static_automaton(P):
    """8300 slots and no static automaton: nothing to split, the two-warp kernel runs with sorted slots;
    the dynamic side alone drafts, as the oracle does."""
    spec = W.scaled(W.SPECS["c4"], 1000, 8300, 100, 60)
    w = W.make(spec)
    L, msl = spec.draft_len, spec.prompt_len + spec.gen_len
    ref, ob, _ = oracle_run(None, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl, threads=8)
    got, batch = gpu_run(P, None, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl)
    assert batch.launches_per_step() == 2
    assert_same(got, ref, "no static automaton")
    assert (got["source"] == 2).any() and not (got["source"] == 1).any()
    assert_dynamic_automata_equal(batch, ob, [0, 8299], msl)


def test_split_step_reports_failed_slots_like_the_oracle(P):
    """Bad counts, bad tokens and texts that outgrow max_seq_len in a batch of 8300: the refused slots are
    frozen with the oracle's status codes, the others are unaffected."""
    spec = W.scaled(W.SPECS["c5"], 100_000, 8300, 24, 40)
    w = W.make(spec)
    L, msl = spec.draft_len, spec.prompt_len + spec.gen_len - 9     # the last tokens do not fit: status 1
    counts, toks = w.counts.copy(), w.new_tokens.copy()
    counts[1, 5] = -3; counts[2, 77] = spec.accept_max + 1          # status 4
    toks[1, 100, 0] = spec.vocab; toks[2, 8200, 0] = -1             # status 3
    st = P.StaticSam.build(w.corpus, spec.vocab)
    ref, ob, _ = oracle_run(w.corpus, spec.vocab, w.prompts, toks, counts, L, msl, threads=8)
    got, batch = gpu_run(P, st, spec.vocab, w.prompts, toks, counts, L, msl)
    assert_same(got, ref, "split step, failures")
    assert {1, 3, 4} <= set(np.unique(got["status"]).tolist())


CASES = {
    # name: (spec key, corpus_len, batch, prompt_len, gen_len) — same recipes, smaller sizes
    "tiny_full": ("tiny", None, None, None, None),
    "c2_small": ("c2", 400_000, 16, 512, 700),
    "c3_small": ("c3", 600_000, 24, 600, 900),
    "c4_small": ("c4", 200_000, 32, 1500, 700),
    "c5_small": ("c5", 500_000, 96, 500, 500),
}


@pytest.mark.parametrize("name", list(CASES))
def test_workload_recipes(P, name):
    key, N, B, pl, gl = CASES[name]
    spec = W.scaled(W.SPECS[key], N, B, pl, gl)
    w = W.make(spec)
    L = spec.draft_len
    msl = spec.prompt_len + spec.gen_len
    st = P.StaticSam.build(w.corpus, spec.vocab)
    ref, ob, S = oracle_run(w.corpus, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl, threads=4)
    got, batch = gpu_run(P, st, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl)
    assert_same(got, ref, name)
    assert (got["status"] == 0).all()
    assert_dynamic_automata_equal(batch, ob, [0, spec.batch - 1], msl)
    assert (got["source"] == 1).any() or key == "c4"
    assert (got["source"] == 2).any()
    info = st.info
    assert info.n_states == S.n_states and info.n_transitions == S.n_transitions


def test_multi_document_corpus_with_stop_token(P):
    """A corpus of documents joined by an end-of-sequence token, with that token as the drafts' stop
    token (Section 3.1): every output equals the oracle's, no draft crosses a document boundary, and
    some drafts are in fact cut short by a separator."""
    spec = W.scaled(W.DOCS, 600_000, 24, 500, 700)
    w = W.make(spec)
    L, msl = spec.draft_len, spec.prompt_len + spec.gen_len
    st = P.StaticSam.build(w.corpus, spec.vocab)
    ref, ob, S = oracle_run(w.corpus, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl, threads=4, stop_token=spec.eos)
    got, batch = gpu_run(P, st, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl, stop_token=spec.eos)
    assert_same(got, ref, "docs")
    assert (got["status"] == 0).all() and not (got["draft_tokens"] == spec.eos).any()
    tb = P.binding.sam_static_tables(st.handle)
    stat = got["source"] == 1
    e1 = tb["min_endpos"][got["state"][..., 0]]
    room = np.minimum(L, spec.corpus_len - e1)
    assert (stat & (got["draft_len"] < room)).any()                 # cut by a separator, not by the corpus' end
    assert st.info.n_states == S.n_states and st.info.n_transitions == S.n_transitions


def test_c2_full_size_bench_configuration(P):
    """Config 2 at full size, launched exactly as the benchmark launches it (prefill step, then one
    launch per decoding step through sam_run_steps): every output of every step equals the oracle."""
    spec = W.SPECS["c2"]
    w = W.make(spec)
    L, msl = spec.draft_len, spec.prompt_len + spec.gen_len
    st = P.StaticSam.build(w.corpus, spec.vocab)
    ref, ob, S = oracle_run(w.corpus, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl, threads=8)
    got, batch = gpu_run(P, st, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl)
    assert_same(got, ref, "c2 full")
    assert st.info.n_states == S.n_states
    # self-certifying sample: the reported match is a suffix occurrence at the reported end position
    rng = random.Random(2)
    tb = P.binding.sam_static_tables(st.handle)
    pos = np.full(spec.batch, spec.prompt_len) + np.cumsum(w.counts, axis=0)
    for _ in range(300):
        s = rng.randrange(w.n_steps); b = rng.randrange(spec.batch)
        k = int(pos[s, b]); x = w.seqs[b, :k]
        l1 = int(got["match_len"][s + 1, b, 0]); e1 = int(tb["min_endpos"][got["state"][s + 1, b, 0]])
        assert (w.corpus[e1 - l1:e1] == x[k - l1:]).all()
        if got["source"][s + 1, b] == 1:
            dl = int(got["draft_len"][s + 1, b])
            assert (got["draft_tokens"][s + 1, b, :dl] == w.corpus[e1:e1 + dl]).all()


def _mem_available_gb():
    try:
        for line in open("/proc/meminfo"):
            if line.startswith("MemAvailable:"):
                return int(line.split()[1]) / 1e6
    except OSError:
        pass
    return 1e9


# host memory (GB) the two independent automata of a full-size case need side by side, with margin
FULL_SIZE_HOST_GB = {"c4": 4, "c3": 60, "c5": 110}


@pytest.mark.parametrize("key", ["c4", "c3", "c5"])
def test_full_size_configs(P, key):
    """The recipe at its full size, launched as the benchmark launches it (prefill step, then every
    decoding step through sam_run_steps; the slot-ordering launch included for c5): every output of
    every step equals the oracle's, and the library's static automaton has the oracle's number of
    states and transitions.  The oracle's automaton is built in a thread while the library builds its
    own and the GPU runs.  Skipped only when the host cannot hold both automata."""
    import threading
    import torch
    avail = _mem_available_gb()
    free_dev = torch.cuda.mem_get_info()[0] / 1e9
    if avail < FULL_SIZE_HOST_GB[key]:
        pytest.skip("host has %.0f GB available; %s at full size needs about %d GB" % (avail, key, FULL_SIZE_HOST_GB[key]))
    spec = W.SPECS[key]
    if free_dev < spec.corpus_len * 100e-9 + 6:
        pytest.skip("device has %.0f GB free; %s at full size needs about %.0f GB" % (free_dev, key, spec.corpus_len * 100e-9 + 6))
    w = W.make(spec)
    L, msl = spec.draft_len, spec.prompt_len + spec.gen_len
    box = {}

    def build_oracle():
        try:
            box["S"] = oracle.Sam(w.corpus)
        except BaseException as ex:                     # re-raised in the test's own thread
            box["err"] = ex

    th = threading.Thread(target=build_oracle)
    th.start()
    st = P.StaticSam.build(w.corpus, spec.vocab)
    got, batch = gpu_run(P, st, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl)
    assert batch.launches_per_step() == (2 if spec.batch >= 1536 else 1)
    th.join()
    if "err" in box:
        raise box["err"]
    ref, ob, S = oracle_run(w.corpus, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl, static=box["S"],
                            threads=os.cpu_count())
    assert_same(got, ref, key)
    assert (got["status"] == 0).all()
    assert st.info.n_states == S.n_states and st.info.n_transitions == S.n_transitions


def test_runs_of_new_tokens_across_slabs_and_crowded_root_buckets(P):
    """The parallel path for runs of new tokens: runs that straddle a slab boundary (4 KiB slabs hold
    128 records), chunks with repeated tokens, and tiny root tables where many tokens share a bucket."""
    rng = random.Random(77)
    empty = lambda B: np.zeros((B, 0), np.int32)
    # all-distinct text in steps of 24 (128 is not a multiple of 24) and of 100 (several chunks of 32)
    for step in (24, 100):
        n = 1000
        x = list(range(n)); rng.shuffle(x)
        rows = [x[i:i + step] + [-1] * (step - len(x[i:i + step])) for i in range(0, n, step)]
        nt = np.array(rows, dtype=np.int32).reshape(len(rows), 1, step)
        ct = np.array([min(step, n - i) for i in range(0, n, step)], dtype=np.int32).reshape(-1, 1)
        ref, ob, _ = oracle_run(None, n, empty(1), nt, ct, 8, n)
        got, batch = gpu_run(P, None, n, empty(1), nt, ct, 8, n, slab_bytes=4096)
        assert_same(got, ref)
        assert_dynamic_automata_equal(batch, ob, [0], n)
    # short sequences (root table of 64 entries = 8 buckets): distinct tokens, then tokens with repeats
    for case in range(120):
        n = rng.randint(8, 32)
        vocab = 100000
        if case % 2 == 0:
            x = rng.sample(range(vocab), n)
        else:
            pool = rng.sample(range(vocab), rng.randint(3, n))
            x = [rng.choice(pool) for _ in range(n)]
        B = 3
        xs = [x, x[::-1], x[n // 2:] + x[:n // 2]]
        k = rng.choice([n, 7, 32])
        rows, cnts = [], []
        for i in range(0, n, k):
            rows.append([t[i:i + k] + [-1] * (k - len(t[i:i + k])) for t in xs]); cnts.append([min(k, n - i)] * B)
        nt = np.array(rows, dtype=np.int32); ct = np.array(cnts, dtype=np.int32)
        ref, ob, _ = oracle_run(None, vocab, empty(B), nt, ct, 4, n)
        got, batch = gpu_run(P, None, vocab, empty(B), nt, ct, 4, n)
        assert_same(got, ref, "case %d" % case)
        assert_dynamic_automata_equal(batch, ob, range(B), n)


def test_pool_exhaustion_leaves_other_slots_exact(P):
    """When the shared pool runs dry some slots stop with status 1; the slots that did not stop still
    agree with the oracle on everything."""
    rng = random.Random(8)
    vocab, n, L, B = 3000, 1200, 8, 6
    nt = np.array([[rng.randrange(vocab) for _ in range(n)] for _ in range(B)], dtype=np.int32)
    step = 60
    rows = nt.reshape(B, n // step, step).transpose(1, 0, 2).copy()
    ct = np.full((n // step, B), step, dtype=np.int32)
    ref, _, _ = oracle_run(None, vocab, np.zeros((B, 0), np.int32), rows, ct, L, n)
    got, _ = gpu_run(P, None, vocab, np.zeros((B, 0), np.int32), rows, ct, L, n, slab_bytes=4096, pool_slabs=40)
    st = got["status"]
    assert set(np.unique(st).tolist()) <= {0, 1} and (st[-1] == 1).any() and (st[0] == 0).all()
    ok = st == 0
    for k in ("draft_len", "match_len", "source", "state", "draft_tokens"):
        assert np.array_equal(got[k][ok], ref[k][ok]), k
    assert (got["draft_len"][~ok] == 0).all()
    # once stopped, always stopped
    assert (np.diff((st != 0).astype(int), axis=0) >= 0).all()
