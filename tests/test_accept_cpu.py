"""Pins for the oracle's greedy verification and auxiliary selection (definitions of Sections 2.2
and 3.4 on hand-made cases), and the closed decoding loop's basic accounting."""
import numpy as np

import oracle
import workloads as W
from oracle import accept


def test_accept_greedy_hand_cases():
    draft = np.array([[5, 6, 7, 8], [5, 6, 7, 8], [5, 6, 7, 8], [5, 6, 7, 8], [9, 9, 9, 9]], dtype=np.int32)
    dlen = np.array([4, 4, 2, 0, 4], dtype=np.int32)
    target = np.array([[5, 6, 7, 8, 1],      # whole draft confirmed: 4 + the target's next token
                       [5, 6, 0, 8, 1],      # third token differs: 2 confirmed, the target's own third token follows
                       [5, 6, 7, 8, 1],      # only two drafted
                       [3, 6, 7, 8, 1],      # nothing drafted: one plain decoding step
                       [5, 6, 7, 8, 1]], dtype=np.int32)   # first token differs
    nt, cnt, acc = accept.accept_greedy(draft, dlen, target)
    assert cnt.tolist() == [5, 3, 3, 1, 1] and acc.tolist() == [4, 2, 2, 0, 0]
    assert nt[0].tolist() == [5, 6, 7, 8, 1] and nt[1].tolist() == [5, 6, 0, -1, -1]
    assert nt[2].tolist() == [5, 6, 7, -1, -1] and nt[3].tolist() == [3, -1, -1, -1, -1] and nt[4, 0] == 5
    # caps: per-slot limit and row width
    nt, cnt, acc = accept.accept_greedy(draft, dlen, target, max_new=[2, 0, 9, 1, 1], stride=3)
    assert cnt.tolist() == [2, 0, 3, 1, 1] and acc.tolist() == [2, 0, 2, 0, 0]
    assert nt.shape == (5, 3) and nt[1].tolist() == [-1, -1, -1]


def test_select_auxiliary_hand_cases():
    draft = np.array([[1, 2, -1], [-1, -1, -1], [-1, -1, -1]], dtype=np.int32)
    d, dl, src = accept.select_auxiliary(draft, [2, 0, 0], [2, 0, 0], np.array([[7, 7, 7], [8, 9, 0], [4, 4, 4]]), [3, 2, 0])
    assert d.tolist() == [[1, 2, -1], [8, 9, -1], [-1, -1, -1]] and dl.tolist() == [2, 2, 0] and src.tolist() == [2, 3, 0]


def test_decode_loop_reconstructs_the_sequences():
    spec = W.scaled(W.SPECS["tiny"], corpus_len=20000, batch=3, prompt_len=50, gen_len=150)
    w = W.make(spec)
    S = oracle.Sam(w.corpus)
    total = spec.prompt_len + spec.gen_len
    ob = oracle.Batch(S, w.corpus, spec.batch, spec.vocab, total)
    log, pos = accept.decode_loop(ob, w.seqs, spec.prompt_len, spec.draft_len, spec.draft_len + 1)
    assert (pos == total).all()
    for b in range(spec.batch):
        assert ob.seq_len(b) == total                      # every token went through the automata once
    acc = np.array([r["accepted"] for r in log]); cnt = np.array([r["counts"] for r in log])
    assert ((cnt == acc + 1) | (cnt == 0) | (cnt.cumsum(0) + spec.prompt_len == total)).all()
    assert acc.sum() > 0 and len(log) < spec.gen_len       # drafts were accepted: fewer steps than tokens
    # an accepted draft token is by construction the true continuation
    p = np.full(spec.batch, spec.prompt_len)
    for r in log:
        for b in range(spec.batch):
            a = int(r["accepted"][b])
            assert (r["draft_tokens"][b, :a] == w.seqs[b, p[b]:p[b] + a]).all()
        p = p + r["counts"]
