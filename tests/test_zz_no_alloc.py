"""The allocation-free retrieval call against the regular path and against the CPU oracle.

Some callers of this library cannot allocate device memory at all — a drafting hook inside an
inference server that has already claimed the device's free memory for its KV cache, for example —
so `sam_retrieve_noalloc` keeps its per-sequence automata in an array built into the library.
This file checks, through the C ABI, that it returns exactly what a fresh batch plus one
`sam_step` returns and what the oracle computes for "empty sequences, one step", twice in a row
with different inputs (the array keeps the previous call's contents, so the second call proves that
what must start empty is cleared); that a call leaves the device's free memory where it was and
works on a stream other than the default one; and that a request too large for the array is
refused.  It is named to be collected last.
"""
import numpy as np
import pytest

import oracle
import workloads as W

pytestmark = pytest.mark.gpu

KEYS = ("draft_tokens", "draft_len", "match_len", "source", "state", "status")


def _regular(P, st, vocab, toks, cnts, L, l_bias, min_match):
    import torch
    B, stride = toks.shape
    batch = P.Batch(st, B, stride, max_draft_len=L, l_bias=l_bias, min_match=min_match, vocab=vocab)
    out = batch.step(torch.from_numpy(toks).to(batch.device), torch.from_numpy(cnts).to(batch.device), L)
    res = out.cpu()
    batch.close()
    return res


def _noalloc(P, st, vocab, toks, cnts, L, l_bias, min_match, stream=None):
    import torch
    dev = torch.device("cuda", 0)
    B = toks.shape[0]
    out = P.StepOutputs(B, L, dev)
    for t in out.tensors():
        t.fill_(-7)                                   # stale values must all be overwritten
    td, cd = torch.from_numpy(toks).to(dev), torch.from_numpy(cnts).to(dev)
    torch.cuda.synchronize()
    P.binding.sam_retrieve_noalloc(st.handle if st is not None else None, vocab, td, cd,
                                   L, l_bias, min_match, *out.tensors(), stream=stream)
    torch.cuda.synchronize()
    return out.cpu()


def _oracle(S, corpus, vocab, toks, cnts, L, l_bias, min_match):
    """What the paper's algorithms give for empty sequences fed their whole text in one step."""
    B, stride = toks.shape
    ob = oracle.Batch(S, corpus, B, vocab, stride, l_bias, min_match)
    o = ob.step(toks, cnts, L)
    return {k: getattr(o, k) for k in KEYS}


def test_noalloc_matches_regular_path_twice_in_a_row():
    import torch
    assert torch.cuda.is_available()
    import paper_2411_10666_b200 as P
    P.lib()
    spec = W.scaled(W.SPECS["tiny"], corpus_len=40_000, batch=6, prompt_len=200, gen_len=300)
    w = W.make(spec)
    st = P.StaticSam.build(w.corpus, spec.vocab)
    L = spec.draft_len
    # call 1: six sequences of different lengths; call 2: other texts, shorter, one slot empty and
    # one slot with an out-of-range token (status 3) — nothing of call 1 may show through
    toks1 = np.ascontiguousarray(w.seqs[:, :500])
    cnts1 = np.array([500, 431, 257, 33, 1, 500], dtype=np.int32)
    toks2 = np.ascontiguousarray(w.seqs[::-1, 100:420])
    cnts2 = np.array([320, 0, 111, 320, 64, 7], dtype=np.int32)
    toks2[4, 10] = spec.vocab + 5
    S = oracle.Sam(w.corpus)
    for toks, cnts, l_bias, min_match in ((toks1, cnts1, 0, 1), (toks2, cnts2, 2, 3)):
        got = _noalloc(P, st, spec.vocab, toks, cnts, L, l_bias, min_match)
        ref = _regular(P, st, spec.vocab, toks, cnts, L, l_bias, min_match)
        exp = _oracle(S, w.corpus, spec.vocab, toks, cnts, L, l_bias, min_match)
        for k in KEYS:
            assert np.array_equal(got[k], ref[k]), k           # integer work: bit-exact
            assert np.array_equal(got[k], exp[k]), k
    assert ref["status"].tolist() == [0, 0, 0, 0, 3, 0]
    # without a static automaton
    got = _noalloc(P, None, spec.vocab, toks1, cnts1, L, 0, 1)
    ref = _regular(P, None, spec.vocab, toks1, cnts1, L, 0, 1)
    exp = _oracle(None, None, spec.vocab, toks1, cnts1, L, 0, 1)
    for k in KEYS:
        assert np.array_equal(got[k], ref[k]), k
        assert np.array_equal(got[k], exp[k]), k
    assert (got["source"] == 2).any()


def test_noalloc_allocates_nothing_and_runs_on_a_side_stream():
    """The property the call is named for: after a first call (which looks the array's address up) a
    further call leaves the device's free memory exactly where it was.  And the call is not tied to
    the default stream."""
    import torch
    import paper_2411_10666_b200 as P
    P.lib()
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(3)
    B, stride, L, vocab = 5, 300, 8, 7
    toks = rng.integers(0, vocab, size=(B, stride), dtype=np.int32)
    cnts = np.array([300, 17, 0, 123, 299], dtype=np.int32)
    exp = _oracle(None, None, vocab, toks, cnts, L, 0, 1)
    first = _noalloc(P, None, vocab, toks, cnts, L, 0, 1)                 # set-up happens here
    td, cd = torch.from_numpy(toks).to(dev), torch.from_numpy(cnts).to(dev)
    out = P.StepOutputs(B, L, dev)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info(dev)
    P.binding.sam_retrieve_noalloc(None, vocab, td, cd, L, 0, 1, *out.tensors())
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info(dev)
    assert free1 == free0, "the call changed the device's free memory by %d bytes" % (free0 - free1)
    side = torch.cuda.Stream(device=dev)
    side.wait_stream(torch.cuda.current_stream(dev))
    with torch.cuda.stream(side):
        on_side = _noalloc(P, None, vocab, toks, cnts, L, 0, 1, stream=side)
    for k in KEYS:
        assert np.array_equal(first[k], exp[k]), k
        assert np.array_equal(out.cpu()[k], exp[k]), k
        assert np.array_equal(on_side[k], exp[k]), k


def test_noalloc_refuses_what_does_not_fit():
    import torch
    import paper_2411_10666_b200 as P
    cap = P.lib().sam_noalloc_capacity_bytes()
    assert cap == 8 << 20
    dev = torch.device("cuda", 0)
    B, stride, L = 64, 4096, 8                          # far beyond 8 MiB of automata
    toks = torch.zeros((B, stride), dtype=torch.int32, device=dev)
    cnts = torch.zeros(B, dtype=torch.int32, device=dev)
    out = P.StepOutputs(B, L, dev)
    with pytest.raises(P.SamError) as e:
        P.binding.sam_retrieve_noalloc(None, 100, toks, cnts, L, 0, 1, *out.tensors())
    assert e.value.code == -7
    with pytest.raises(P.SamError) as e:
        P.binding.sam_retrieve_noalloc(None, 0, toks[:2, :16].contiguous(), cnts[:2].contiguous(), L, 0, 1,
                                       *P.StepOutputs(2, L, dev).tensors())
    assert e.value.code == -1
    torch.cuda.synchronize()
