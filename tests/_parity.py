"""Helpers shared by the GPU parity tests: run a workload through the CUDA library and through
the CPU oracle and compare every output of every step."""
import numpy as np

import oracle

KEYS = ("draft_tokens", "draft_len", "match_len", "source", "state", "status")


def oracle_run(corpus, vocab, prompts, new_tokens, counts, L, max_seq_len, l_bias=0, min_match=1,
               static=None, threads=1, stop_token=-1):
    """Returns (per-step dict of arrays with a leading step axis incl. the prefill step, batch obj)."""
    B = prompts.shape[0]
    S = static if static is not None else (oracle.Sam(corpus) if corpus is not None else None)
    ob = oracle.Batch(S, corpus, B, vocab, max_seq_len, l_bias, min_match, stop_token)
    outs = []
    if prompts.shape[1] > 0:
        outs.append(ob.step(prompts, np.full(B, prompts.shape[1], dtype=np.int32), L, threads))
    for s in range(new_tokens.shape[0]):
        outs.append(ob.step(new_tokens[s], counts[s], L, threads))
    res = {k: np.stack([getattr(o, k) for o in outs]) for k in KEYS}
    return res, ob, S


def gpu_run(P, static, vocab, prompts, new_tokens, counts, L, max_seq_len, l_bias=0, min_match=1, **kw):
    import torch
    B = prompts.shape[0]
    batch = P.Batch(static, B, max_seq_len, max_draft_len=max(L, 1), l_bias=l_bias, min_match=min_match,
                    vocab=vocab, **kw)
    dev = batch.device
    outs = []
    if prompts.shape[1] > 0:
        pt = torch.from_numpy(np.ascontiguousarray(prompts)).to(dev)
        ct = torch.full((B,), prompts.shape[1], dtype=torch.int32, device=dev)
        o = batch.step(pt, ct, L)
        outs.append({k: v[None] for k, v in o.cpu().items()})
    if new_tokens.shape[0] > 0:
        nt = torch.from_numpy(np.ascontiguousarray(new_tokens)).to(dev)
        ct = torch.from_numpy(np.ascontiguousarray(counts)).to(dev)
        o = batch.run_steps(nt, ct, L, per_step=True)
        outs.append(o.cpu())
    torch.cuda.synchronize()
    res = {k: np.concatenate([o[k] for o in outs]) for k in KEYS}
    return res, batch


def assert_same(gpu, ref, what=""):
    for k in KEYS:
        if not np.array_equal(gpu[k], ref[k]):
            bad = np.argwhere(gpu[k] != ref[k])
            first = tuple(bad[0])
            raise AssertionError("%s: %s differs at %d places, first at %s: gpu %s oracle %s" % (
                what, k, len(bad), first, gpu[k][first], ref[k][first]))


def assert_dynamic_automata_equal(batch, ob, slots, max_len):
    """Slot by slot: the device's dynamic automaton equals the oracle's, state for state."""
    for b in slots:
        D = ob.dynamic(b)
        link, length, endpos, deg = D.tables()
        d = batch.dump(b, 2 * max_len + 2, 3 * max_len + 2)
        assert d["n_tokens"] == ob.seq_len(b)
        assert d["n_states"] == D.n_states, (b, d["n_states"], D.n_states)
        assert d["n_edges"] == D.n_transitions
        # the newest state's record is complete on both sides; compare all tables
        assert np.array_equal(d["length"], length) and np.array_equal(d["link"], link)
        assert np.array_equal(d["min_endpos"], endpos) and np.array_equal(d["deg"], deg)
        got = set(zip(d["edge_src"].tolist(), d["edge_tok"].tolist(), d["edge_tgt"].tolist()))
        exp = {(s, t, u) for s in range(D.n_states) for t, u in D.edges(s).items()}
        assert got == exp
