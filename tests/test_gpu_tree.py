"""GPU: freq, and the best-first tree draft (Algorithm 5) against the oracle — tokens, parents and the
float32 path probabilities bit for bit."""
import random

import numpy as np
import pytest

import oracle
import workloads as W
from oracle import tree

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    import torch
    assert torch.cuda.is_available()
    import paper_2411_10666_b200 as pkg
    pkg.lib()
    return pkg


def _run(P, st, states, starts, max_size, k):
    import torch
    B = len(states)
    dev = torch.device("cuda", 0)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(np.asarray(a, dtype=np.int32))).to(dev)
    toks = torch.empty((B, max_size), dtype=torch.int32, device=dev); par = torch.empty_like(toks)
    pr = torch.empty((B, max_size), dtype=torch.float32, device=dev); sz = torch.empty(B, dtype=torch.int32, device=dev)
    P.binding.sam_tree_draft(st.handle, t(states), t(starts), max_size, k, toks, par, pr, sz)
    torch.cuda.synchronize()
    return toks.cpu().numpy(), par.cpu().numpy(), pr.cpu().numpy(), sz.cpu().numpy()


def _check(P, S, f, st, states, starts, max_size, k):
    toks, par, pr, sz = _run(P, st, states, starts, max_size, k)
    for i, (s, t0) in enumerate(zip(states, starts)):
        if s <= 0:
            assert sz[i] == 0 and (toks[i] == -1).all()
            continue
        et, ep, epr = tree.prim_tree(S, f, s, t0, max_size, k)
        n = len(et)
        assert sz[i] == n, (i, s, sz[i], n)
        assert toks[i, :n].tolist() == et and par[i, :n].tolist() == ep, (i, s)
        assert (toks[i, n:] == -1).all() and (par[i, n:] == -1).all()
        assert np.array_equal(pr[i, :n].view(np.uint32), np.array(epr, dtype=np.float32).view(np.uint32)), (i, s)


def test_abcbc_tree(P):
    x = np.array([0, 1, 2, 1, 2], dtype=np.int32)
    st = P.StaticSam.build(x, 3, tree_topk=2)
    assert st.info.tree_topk == 2
    assert P.binding.sam_static_freq(st.handle).tolist() == [5, 1, 1, 1, 1, 2, 1, 2]
    toks, par, pr, sz = _run(P, st, [5, 0, 7], [1, 0, 2], 8, 2)
    assert sz.tolist() == [4, 0, 3]
    assert toks[0, :4].tolist() == [1, 2, 1, 2] and par[0, :4].tolist() == [-1, 0, 1, 2]
    assert pr[0, :4].tolist() == [1.0, 1.0, 0.5, 0.5]
    with pytest.raises(P.SamError):
        _run(P, st, [5], [1], 8, 3)                          # k beyond what the automaton was built with
    plain = P.StaticSam.build(x, 3)
    with pytest.raises(P.SamError):
        _run(P, plain, [5], [1], 8, 1)                       # no tree data


@pytest.mark.parametrize("seed", range(4))
def test_random_texts(P, seed):
    rng = random.Random(50 + seed)
    for vocab, n in [(2, 40), (3, 300), (6, 3000), (40, 5000)]:
        x = []
        while len(x) < n:
            if x and rng.random() < 0.3:
                s = rng.randrange(len(x)); x.extend(x[s:s + rng.randint(1, 15)])
            else:
                x.append(rng.randrange(vocab))
        x = np.array(x[:n], dtype=np.int32)
        S = oracle.Sam(x)
        f = S.freq()
        for k in (1, 2, 4, 6):
            st = P.StaticSam.build(x, vocab, tree_topk=k)
            assert np.array_equal(P.binding.sam_static_freq(st.handle).astype(np.int64), f)
            states = [rng.randrange(0, S.n_states) for _ in range(40)] + [1, S.n_states - 1, -3]
            starts = [rng.randrange(vocab) for _ in states]
            for max_size in (1, 7, 40, 128):
                _check(P, S, f, st, states, starts, max_size, min(k, rng.randint(1, k)))


def test_workload_states_after_a_decoding_run(P):
    """Trees drafted from the static states a real decoding run ends in (workload recipe c2, reduced)."""
    import torch
    spec = W.scaled(W.SPECS["c2"], corpus_len=300_000, batch=32, prompt_len=256, gen_len=256)
    w = W.make(spec)
    S = oracle.Sam(w.corpus)
    f = S.freq()
    st = P.StaticSam.build(w.corpus, spec.vocab, tree_topk=4)
    assert np.array_equal(P.binding.sam_static_freq(st.handle).astype(np.int64), f)
    batch = P.Batch(st, spec.batch, spec.prompt_len + spec.gen_len, max_draft_len=spec.draft_len)
    dev = batch.device
    batch.step(torch.from_numpy(w.prompts).to(dev), torch.full((spec.batch,), spec.prompt_len, dtype=torch.int32, device=dev),
               spec.draft_len)
    out = batch.run_steps(torch.from_numpy(w.new_tokens[:40]).to(dev), torch.from_numpy(w.counts[:40]).to(dev),
                          spec.draft_len, per_step=False).cpu()
    states = out["state"][:, 0].tolist()
    pos = spec.prompt_len + w.counts[:40].sum(axis=0)
    starts = [int(w.seqs[b, pos[b] - 1]) for b in range(spec.batch)]
    assert any(s > 0 for s in states)
    _check(P, S, f, st, states, starts, 40, 4)
    _check(P, S, f, st, states, starts, 16, 2)
