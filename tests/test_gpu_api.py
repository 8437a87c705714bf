"""GPU tests of the boundary's conventions: per-slot status codes, freezing, reset and slab reuse,
count 0, the host-array step, image save/load, pool exhaustion.  Expected values come from the
oracle or are stated outright; nothing here expects a fault."""
import os
import random

import numpy as np
import pytest

import oracle
import workloads as W
from _parity import KEYS, assert_dynamic_automata_equal, assert_same, gpu_run, oracle_run

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    import torch
    assert torch.cuda.is_available()
    import paper_2411_10666_b200 as pkg
    pkg.lib()
    return pkg


def _t(a, dev):
    import torch
    return torch.from_numpy(np.ascontiguousarray(np.asarray(a, dtype=np.int32))).to(dev)


def test_status_codes_freeze_and_match_oracle(P):
    vocab, msl, L = 10, 6, 4
    steps = [
        ([[1, 2, 3], [1, 10, 0], [1, 2, 3], [1, 2, 3]], [3, 2, 4, 3]),     # ok, bad token, bad count, ok
        ([[1, 2, 1], [1, 1, 1], [1, 1, 1], [5, 0, 0]], [3, 1, 1, 1]),      # ok (6 tokens), frozen, frozen, ok
        ([[1, 0, 0], [1, 1, 1], [1, 1, 1], [5, 0, 0]], [1, 0, -1, 0]),     # capacity, frozen, frozen, count 0
    ]
    nt = np.array([s[0] for s in steps], dtype=np.int32)
    ct = np.array([s[1] for s in steps], dtype=np.int32)
    empty = np.zeros((4, 0), np.int32)
    ref, _, _ = oracle_run(None, vocab, empty, nt, ct, L, msl)
    got, batch = gpu_run(P, None, vocab, empty, nt, ct, L, msl)
    assert_same(got, ref)
    assert got["status"].tolist() == [[0, 3, 4, 0], [0, 3, 4, 0], [1, 3, 4, 0]]
    assert (got["draft_tokens"][2, :3] == -1).all() and (got["draft_len"][2, :3] == 0).all()
    # the failed step changed nothing: slot 0 still holds 6 tokens
    assert batch.dump(0, 16, 32)["n_tokens"] == 6


def test_argument_errors_launch_nothing(P):
    import torch
    b = P.Batch(None, 2, 16, max_draft_len=8, vocab=5)
    dev = b.device
    toks, cnt = _t([[1, 2], [3, 4]], dev), _t([2, 2], dev)
    out = P.StepOutputs(2, 8, dev)
    L = P.lib()
    args = [toks.data_ptr(), 2, cnt.data_ptr(), 8] + [t.data_ptr() for t in out.tensors()] + [None]
    assert L.sam_step(b.handle, *args) == 0
    bad = list(args); bad[3] = 9                                   # L > max_draft_len
    assert L.sam_step(b.handle, *bad) == -1
    bad = list(args); bad[1] = 0                                   # stride < 1
    assert L.sam_step(b.handle, *bad) == -1
    bad = list(args); bad[4] = None                                # null output
    assert L.sam_step(b.handle, *bad) == -1
    ws = torch.empty(1024, dtype=torch.uint8, device=dev)
    h = P.binding.c_void_p()
    o = P.BatchOpts(2, 16, 8, 0, 1, 5, 0, 0, 0)
    assert L.sam_batch_create(None, P.binding.byref(o), ws.data_ptr(), ws.numel(), None, P.binding.byref(h)) == -4
    torch.cuda.synchronize()
    assert batch_ok(P, b)


def batch_ok(P, b):
    tot, free = b.pool_info()
    return 0 <= free <= tot


def test_reset_returns_slabs_and_slots_restart(P):
    import torch
    rng = random.Random(3)
    vocab, n, L, B = 40, 600, 8, 6
    texts = [[rng.randrange(vocab) for _ in range(n)] for _ in range(B)]
    nt = np.array(texts, dtype=np.int32)
    b = P.Batch(None, B, n, max_draft_len=L, vocab=vocab, slab_bytes=4096)
    tot, free0 = b.pool_info()
    assert free0 == tot
    full = np.full(B, n, dtype=np.int32)
    o1 = b.step(_t(nt, b.device), _t(full, b.device), L).cpu()
    _, free1 = b.pool_info()
    assert free1 < free0
    b.reset([1, 4])
    _, free2 = b.pool_info()
    assert free1 < free2 < free0
    # slots 1 and 4 start over with other text; the rest are untouched (count 0 re-emits)
    nt2 = nt.copy(); nt2[1] = nt[2]; nt2[4] = nt[0]
    cnt = np.zeros(B, dtype=np.int32); cnt[[1, 4]] = n
    o2 = b.step(_t(nt2, b.device), _t(cnt, b.device), L).cpu()
    for k in KEYS:
        assert np.array_equal(o2[k][[0, 2, 3, 5]], o1[k][[0, 2, 3, 5]]), k
        assert np.array_equal(o2[k][1], o1[k][2]) and np.array_equal(o2[k][4], o1[k][0]), k
    b.reset()
    _, free3 = b.pool_info()
    assert free3 == tot
    o3 = b.step(_t(nt, b.device), _t(full, b.device), L).cpu()
    for k in KEYS:
        assert np.array_equal(o3[k], o1[k])


def test_pool_exhaustion_is_a_status_not_a_fault(P):
    rng = random.Random(4)
    vocab, n, L, B = 500, 2000, 8, 4
    nt = np.array([[rng.randrange(vocab) for _ in range(n)] for _ in range(B)], dtype=np.int32)
    b = P.Batch(None, B, n, max_draft_len=L, vocab=vocab, slab_bytes=4096, pool_slabs=20)
    o = b.step(_t(nt, b.device), _t(np.full(B, n), b.device), L).cpu()
    assert (o["status"] == 1).any()                     # 4 x 2000 tokens cannot fit 20 slabs of 4 KiB
    assert set(o["status"].tolist()) <= {0, 1}
    assert (o["draft_len"][o["status"] == 1] == 0).all()
    o2 = b.step(_t(nt[:, :1], b.device), _t(np.zeros(B), b.device), L).cpu()
    assert np.array_equal(o2["status"], o["status"])   # sticky
    b.reset()
    ok = b.step(_t(nt[:, :50], b.device), _t(np.full(B, 50), b.device), L).cpu()
    assert (ok["status"] == 0).all()


def test_host_step_equals_device_step(P):
    import torch
    spec = W.scaled(W.SPECS["tiny"], corpus_len=30000, batch=5, prompt_len=40, gen_len=120)
    w = W.make(spec)
    L, msl = spec.draft_len, spec.prompt_len + spec.gen_len
    st = P.StaticSam.build(w.corpus, spec.vocab)
    ref, _, _ = oracle_run(w.corpus, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl)
    b = P.Batch(st, spec.batch, msl, max_draft_len=L, max_host_stride=spec.prompt_len)
    B = spec.batch
    mk = lambda *s: torch.empty(s, dtype=torch.int32).pin_memory()
    out = dict(draft_tokens=mk(B, L), draft_len=mk(B), match_len=mk(B, 2), source=mk(B), state=mk(B, 2), status=mk(B))
    steps = [(w.prompts, np.full(B, spec.prompt_len, dtype=np.int32))] + \
            [(w.new_tokens[s], w.counts[s]) for s in range(w.n_steps)]
    prepared = {}                                       # the bound form of the call, one per stride
    for i, (toks, cnt) in enumerate(steps):
        toks = np.ascontiguousarray(toks)
        if i % 2 == 0:
            P.binding.sam_step_host(b.handle, toks, toks.shape[1], np.ascontiguousarray(cnt), L,
                                    *[out[k] for k in KEYS])
        else:
            if toks.shape[1] not in prepared:
                prepared[toks.shape[1]] = P.binding.sam_step_host_prepared(b.handle, toks.shape[1], L, *[out[k] for k in KEYS])
            prepared[toks.shape[1]](toks, np.ascontiguousarray(cnt))
        for k in KEYS:
            assert np.array_equal(out[k].numpy(), ref[k][i]), (i, k)
    with pytest.raises(P.SamError):
        big = np.zeros((B, spec.prompt_len + 1), dtype=np.int32)
        P.binding.sam_step_host(b.handle, big, big.shape[1], np.zeros(B, np.int32), L, *[out[k] for k in KEYS])


@pytest.mark.parametrize("B", [600, 1700, 8300])
def test_host_step_large_with_pinned_and_pageable_arrays(P, B):
    """Large host steps: page-locked caller arrays are read and written in place, pageable ones go
    through the staging area (and, at this size, two DMA copies or the mapped staging area — the DMA path
    runs the device step as it is: slot ordering at 1700 slots, the split step at 8300; the in-place paths
    run one unordered two-warp launch whatever the batch).  All equal the oracle."""
    import torch
    spec = W.scaled(W.SPECS["c5"], corpus_len=60_000, batch=B, prompt_len=24, gen_len=40)
    w = W.make(spec)
    L, msl = spec.draft_len, spec.prompt_len + spec.gen_len
    st = P.StaticSam.build(w.corpus, spec.vocab)
    ref, _, _ = oracle_run(w.corpus, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl, threads=4)
    steps = [(w.prompts, np.full(B, spec.prompt_len, dtype=np.int32))] + \
            [(w.new_tokens[s], w.counts[s]) for s in range(w.n_steps)]
    for pinned in (True, False):
        b = P.Batch(st, B, msl, max_draft_len=L, max_host_stride=spec.prompt_len)
        mk = (lambda *s: torch.empty(s, dtype=torch.int32).pin_memory()) if pinned else (lambda *s: torch.empty(s, dtype=torch.int32))
        out = dict(draft_tokens=mk(B, L), draft_len=mk(B), match_len=mk(B, 2), source=mk(B), state=mk(B, 2), status=mk(B))
        for i, (toks, cnt) in enumerate(steps):
            t = torch.from_numpy(np.ascontiguousarray(toks)); c = torch.from_numpy(np.ascontiguousarray(cnt))
            if pinned:
                t, c = t.pin_memory(), c.pin_memory()
            P.binding.sam_step_host(b.handle, t, t.shape[1], c, L, *[out[k] for k in KEYS])
            for k in KEYS:
                assert np.array_equal(out[k].numpy(), ref[k][i]), (pinned, i, k)
        b.close()


def test_cached_static_automaton_is_built_once_then_loaded(P, tmp_path):
    """StaticSam.cached keeps the built image under a name derived from the corpus: the first call builds and
    saves, the second loads the same automaton, another corpus gets another file, a damaged file is rebuilt."""
    spec = W.scaled(W.SPECS["c2"], corpus_len=90_000, batch=3, prompt_len=60, gen_len=120)
    w = W.make(spec)
    L, msl = spec.draft_len, spec.prompt_len + spec.gen_len
    d = str(tmp_path / "cache")
    st1, how1 = P.StaticSam.cached(w.corpus, spec.vocab, d)
    st2, how2 = P.StaticSam.cached(w.corpus, spec.vocab, d)
    assert (how1, how2) == ("built", "loaded") and len(os.listdir(d)) == 1
    r1, _ = gpu_run(P, st1, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl)
    r2, _ = gpu_run(P, st2, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl)
    assert_same(r2, r1)
    other = w.corpus.copy(); other[5] = (other[5] + 1) % spec.vocab
    _, how3 = P.StaticSam.cached(other, spec.vocab, d)
    assert how3 == "built" and len(os.listdir(d)) == 2
    path = os.path.join(d, sorted(os.listdir(d))[0])
    raw = bytearray(open(path, "rb").read()); raw[len(raw) // 2] ^= 0x10
    open(path, "wb").write(bytes(raw))
    hows = {P.StaticSam.cached(c, spec.vocab, d)[1] for c in (w.corpus, other)}
    assert hows == {"built", "loaded"}                      # the damaged one was rebuilt, the other loaded


def test_image_save_load_roundtrip(P, tmp_path):
    spec = W.scaled(W.SPECS["c2"], corpus_len=120_000, batch=4, prompt_len=100, gen_len=200)
    w = W.make(spec)
    L, msl = spec.draft_len, spec.prompt_len + spec.gen_len
    st = P.StaticSam.build(w.corpus, spec.vocab)
    path = str(tmp_path / "static.sam")
    st.save(path)
    st2 = P.StaticSam.load(path)
    a, b = st.info, st2.info
    assert (a.n_states, a.n_transitions, a.hash_buckets, a.vocab) == (b.n_states, b.n_transitions, b.hash_buckets, b.vocab)
    r1, _ = gpu_run(P, st, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl)
    r2, _ = gpu_run(P, st2, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl)
    assert_same(r2, r1)
    raw = bytearray(open(path, "rb").read())
    raw[len(raw) // 2] ^= 0x40
    open(path, "wb").write(bytes(raw))
    with pytest.raises(P.SamError) as e:
        P.StaticSam.load(path)
    assert e.value.code == -6
    with pytest.raises(P.SamError) as e:
        P.StaticSam.load(str(tmp_path / "missing.sam"))
    assert e.value.code == -5


def test_static_tables_match_oracle_on_device(P):
    spec = W.scaled(W.SPECS["tiny"], corpus_len=50_000)
    corpus = W.make_corpus(spec)
    st = P.StaticSam.build(corpus, spec.vocab)
    S = oracle.Sam(corpus)
    link, length, endpos, deg = S.tables()
    tb = P.binding.sam_static_tables(st.handle)
    assert np.array_equal(tb["length"], length) and np.array_equal(tb["link"], link)
    assert np.array_equal(tb["min_endpos"], endpos) and np.array_equal(tb["deg"], deg)
    busiest = np.argsort(deg)[-5:].tolist()
    rng = random.Random(0)
    for s in busiest + [rng.randrange(S.n_states) for _ in range(30)]:
        got = P.binding.sam_static_state(st.handle, s, max_edges=int(deg[s]) + 1)
        assert got["next"] == S.edges(s), s


def test_probes_report_plausible_numbers(P):
    import torch
    buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for g in (32, 64, 128):
        gbps, mreq = P.binding.sam_probe_random_read(buf, g, iters=2)
        assert 10 < gbps < 20000 and mreq > 0
    ns1 = P.binding.sam_probe_chase(buf, 20000, chains=1)
    ns64 = P.binding.sam_probe_chase(buf, 20000, chains=64)
    assert 100 < ns1 < 5000 and 100 < ns64 < 5000


def test_stop_token_matches_oracle(P):
    spec = W.scaled(W.SPECS["tiny"], corpus_len=40_000, batch=6, prompt_len=100, gen_len=300)
    w = W.make(spec)
    L, msl = 40, spec.prompt_len + spec.gen_len
    vals, cnts = np.unique(w.corpus, return_counts=True)
    stop = int(vals[np.argmax(cnts)])                       # the most frequent token plays the separator
    st = P.StaticSam.build(w.corpus, spec.vocab)
    ref, _, _ = oracle_run(w.corpus, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl, stop_token=stop)
    got, _ = gpu_run(P, st, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl, stop_token=stop)
    assert_same(got, ref)
    plain, _ = gpu_run(P, st, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl)
    assert (got["draft_len"] < plain["draft_len"]).any()    # some drafts were cut
    assert not (got["draft_tokens"] == stop).any()
