"""GPU: greedy verification, auxiliary selection and the closed decoding loop against the oracle."""
import random

import numpy as np
import pytest

import oracle
import workloads as W
from oracle import accept

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    import torch
    assert torch.cuda.is_available()
    import paper_2411_10666_b200 as pkg
    pkg.lib()
    return pkg


def _t(a, dev="cuda"):
    import torch
    return torch.from_numpy(np.ascontiguousarray(np.asarray(a, dtype=np.int32))).to(dev)


def test_accept_and_select_random(P):
    import torch
    rng = np.random.default_rng(7)
    for B, L, stride in [(1, 1, 1), (5, 4, 5), (37, 32, 33), (64, 40, 16), (300, 128, 129)]:
        target = rng.integers(0, 4, size=(B, L + 1), dtype=np.int32)
        draft = target[:, :L].copy()
        flip = rng.random((B, L)) < 0.08
        draft[flip] = (draft[flip] + 1) % 4
        dlen = rng.integers(0, L + 1, size=B, dtype=np.int32)
        cap = rng.integers(0, L + 3, size=B, dtype=np.int32)
        for use_cap in (False, True):
            nt, cnt, acc = accept.accept_greedy(draft, dlen, target, cap if use_cap else None, stride)
            g_nt = torch.empty((B, stride), dtype=torch.int32, device="cuda")
            g_cnt = torch.empty(B, dtype=torch.int32, device="cuda"); g_acc = torch.empty_like(g_cnt)
            P.binding.sam_accept_greedy(_t(draft), _t(dlen), _t(target), _t(cap) if use_cap else None, g_nt, g_cnt, g_acc)
            assert np.array_equal(g_nt.cpu().numpy(), nt) and np.array_equal(g_cnt.cpu().numpy(), cnt)
            assert np.array_equal(g_acc.cpu().numpy(), acc)
        src = rng.integers(0, 3, size=B, dtype=np.int32)
        aux = rng.integers(0, 9, size=(B, L), dtype=np.int32); alen = rng.integers(0, L + 1, size=B, dtype=np.int32)
        dd = np.where(np.arange(L)[None, :] < dlen[:, None], draft, -1).astype(np.int32)
        e_d, e_l, e_s = accept.select_auxiliary(dd, dlen, src, aux, alen)
        g_d, g_l, g_s = _t(dd), _t(dlen), _t(src)
        P.binding.sam_select_auxiliary(g_d, g_l, g_s, _t(aux), _t(alen))
        assert np.array_equal(g_d.cpu().numpy(), e_d) and np.array_equal(g_l.cpu().numpy(), e_l)
        assert np.array_equal(g_s.cpu().numpy(), e_s)


@pytest.mark.parametrize("key,N,B,pl,gl,min_match", [("tiny", 30000, 4, 64, 300, 1), ("c2", 300000, 16, 256, 400, 1),
                                                      ("c4", 100000, 24, 600, 300, 3)])
def test_closed_loop_matches_oracle(P, key, N, B, pl, gl, min_match):
    """draft -> verify against the true continuation -> accept -> update, entirely on the device,
    step for step equal to the same loop run by the oracle."""
    import torch
    spec = W.scaled(W.SPECS[key], N, B, pl, gl)
    w = W.make(spec)
    L, total, stride = spec.draft_len, pl + gl, spec.draft_len + 1
    S = oracle.Sam(w.corpus)
    ob = oracle.Batch(S, w.corpus, B, spec.vocab, total, 0, min_match)
    log, pos_ref = accept.decode_loop(ob, w.seqs, pl, L, stride)

    st = P.StaticSam.build(w.corpus, spec.vocab)
    batch = P.Batch(st, B, total, max_draft_len=L, min_match=min_match)
    dev = batch.device
    seqs = _t(w.seqs, dev).long()
    out = batch.step(_t(w.prompts, dev), torch.full((B,), pl, dtype=torch.int32, device=dev), L)
    pos = torch.full((B,), pl, dtype=torch.int64, device=dev)
    nt = torch.empty((B, stride), dtype=torch.int32, device=dev)
    cnt = torch.empty(B, dtype=torch.int32, device=dev); acc = torch.empty_like(cnt)
    ar = torch.arange(L + 1, device=dev)[None, :]
    for step, ref in enumerate(log):
        target = torch.gather(seqs, 1, torch.clamp(pos[:, None] + ar, max=total - 1)).int().contiguous()
        cap = (total - pos).int().contiguous()
        P.binding.sam_accept_greedy(out.draft_tokens, out.draft_len, target, cap, nt, cnt, acc)
        got = out.cpu()
        for k in ("draft_tokens", "draft_len", "match_len", "source", "state", "status"):
            assert np.array_equal(got[k], ref[k]), (step, k)
        assert np.array_equal(cnt.cpu().numpy(), ref["counts"]) and np.array_equal(acc.cpu().numpy(), ref["accepted"])
        out = batch.step(nt, cnt, L, out)                     # no host round trip between verify and update
        pos += cnt.long()
    assert np.array_equal(pos.cpu().numpy(), pos_ref) and (pos_ref == total).all()
    mean_accept = np.mean([r["counts"][r["counts"] > 0].mean() for r in log if (r["counts"] > 0).any()])
    assert mean_accept > 1.05                                 # retrieval drafts do get accepted


def test_fused_verify_and_step_matches_the_two_call_loop(P):
    """sam_step_verified (verification folded into the step kernel) against the oracle's loop."""
    import torch
    spec = W.scaled(W.SPECS["c2"], 200000, 12, 200, 300)
    w = W.make(spec)
    B, pl, L = spec.batch, spec.prompt_len, spec.draft_len
    total = pl + spec.gen_len
    S = oracle.Sam(w.corpus)
    ob = oracle.Batch(S, w.corpus, B, spec.vocab, total)
    log, pos_ref = accept.decode_loop(ob, w.seqs, pl, L, L + 1)

    st = P.StaticSam.build(w.corpus, spec.vocab)
    batch = P.Batch(st, B, total, max_draft_len=L)
    dev = batch.device
    seqs = _t(w.seqs, dev).long()
    outs = [P.StepOutputs(B, L, dev), P.StepOutputs(B, L, dev)]       # the previous draft and the new one alternate
    cur = 0
    batch.step(_t(w.prompts, dev), torch.full((B,), pl, dtype=torch.int32, device=dev), L, outs[cur])
    pos = torch.full((B,), pl, dtype=torch.int64, device=dev)
    cnt = torch.empty(B, dtype=torch.int32, device=dev); acc = torch.empty_like(cnt)
    ar = torch.arange(L + 1, device=dev)[None, :]
    for step, ref in enumerate(log):
        prev, new = outs[cur], outs[1 - cur]
        got = prev.cpu()
        for k in ("draft_tokens", "draft_len", "match_len", "source", "state", "status"):
            assert np.array_equal(got[k], ref[k]), (step, k)
        target = torch.gather(seqs, 1, torch.clamp(pos[:, None] + ar, max=total - 1)).int().contiguous()
        cap = (total - pos).int().contiguous()
        P.binding.sam_step_verified(batch.handle, target, prev.draft_tokens, prev.draft_len, cap, L,
                                    *new.tensors(), counts_out=cnt, accepted_out=acc)
        assert np.array_equal(cnt.cpu().numpy(), ref["counts"]) and np.array_equal(acc.cpu().numpy(), ref["accepted"])
        pos += cnt.long()
        cur = 1 - cur
    assert np.array_equal(pos.cpu().numpy(), pos_ref)
    with pytest.raises(P.SamError):                                  # the previous draft may not be the output buffer
        P.binding.sam_step_verified(batch.handle, target, new.draft_tokens, new.draft_len, cap, L, *new.tensors())


def _large_loop_case(batch):
    spec = W.scaled(W.SPECS["c5"], 150_000, batch, 40, 60)
    w = W.make(spec)
    return spec, w


# 1600 slots: the step kernel preceded by the slot-ordering kernel; 8300 slots: the split step
@pytest.mark.parametrize("n_slots", [1600, 8300])
def test_two_call_loop_above_the_slot_ordering_threshold(P, n_slots):
    """The closed loop with a batch large enough for the slot-ordering kernel (two launches per step):
    the counts each step reads were written by the kernel just before it on the stream
    (sam_accept_greedy), which is the case the ordering kernel must tolerate.  Step for step equal to
    the oracle's loop."""
    import torch
    spec, w = _large_loop_case(n_slots)
    B, pl, L = spec.batch, spec.prompt_len, spec.draft_len
    total, stride = pl + spec.gen_len, L + 1
    S = oracle.Sam(w.corpus)
    ob = oracle.Batch(S, w.corpus, B, spec.vocab, total)
    log, pos_ref = accept.decode_loop(ob, w.seqs, pl, L, stride)

    st = P.StaticSam.build(w.corpus, spec.vocab)
    batch = P.Batch(st, B, total, max_draft_len=L)
    assert batch.launches_per_step() == 2
    dev = batch.device
    seqs = _t(w.seqs, dev).long()
    out = batch.step(_t(w.prompts, dev), torch.full((B,), pl, dtype=torch.int32, device=dev), L)
    pos = torch.full((B,), pl, dtype=torch.int64, device=dev)
    nt = torch.empty((B, stride), dtype=torch.int32, device=dev)
    cnt = torch.empty(B, dtype=torch.int32, device=dev); acc = torch.empty_like(cnt)
    ar = torch.arange(L + 1, device=dev)[None, :]
    kept = []
    for step in range(len(log)):                              # no host read inside the loop
        target = torch.gather(seqs, 1, torch.clamp(pos[:, None] + ar, max=total - 1)).int().contiguous()
        cap = (total - pos).int().contiguous()
        P.binding.sam_accept_greedy(out.draft_tokens, out.draft_len, target, cap, nt, cnt, acc)
        kept.append({k: getattr(out, k).clone() for k in ("draft_tokens", "draft_len", "match_len", "source", "state", "status")})
        kept[-1]["counts"] = cnt.clone(); kept[-1]["accepted"] = acc.clone()
        out = batch.step(nt, cnt, L, out)
        pos += cnt.long()
    torch.cuda.synchronize()
    for step, ref in enumerate(log):
        for k, v in kept[step].items():
            assert np.array_equal(v.cpu().numpy(), ref[k]), (step, k)
    assert np.array_equal(pos.cpu().numpy(), pos_ref) and (pos_ref == total).all()


@pytest.mark.parametrize("n_slots", [1600, 8300])
def test_counts_written_by_the_fused_step_feed_a_plain_step(P, n_slots):
    """sam_step_verified writes counts_out; the very next call on the stream is a sam_step that takes
    that array as its counts (feeding as many tokens of the continuation again).  With 1600 slots the
    plain step sorts its slots by those counts first.  Every output equals the oracle fed the same way."""
    import torch
    spec, w = _large_loop_case(n_slots)
    B, pl, L = spec.batch, spec.prompt_len, spec.draft_len
    total = pl + spec.gen_len
    S = oracle.Sam(w.corpus)
    ob = oracle.Batch(S, w.corpus, B, spec.vocab, total)
    st = P.StaticSam.build(w.corpus, spec.vocab)
    batch = P.Batch(st, B, total, max_draft_len=L)
    dev = batch.device
    seqs = _t(w.seqs, dev).long()
    outs = [P.StepOutputs(B, L, dev) for _ in range(3)]
    batch.step(_t(w.prompts, dev), torch.full((B,), pl, dtype=torch.int32, device=dev), L, outs[0])
    r_out = ob.step(w.prompts, np.full(B, pl, dtype=np.int32), L)
    pos = torch.full((B,), pl, dtype=torch.int64, device=dev)
    r_pos = np.full(B, pl, dtype=np.int64)
    cnt = torch.empty(B, dtype=torch.int32, device=dev); acc = torch.empty_like(cnt)
    ar = torch.arange(L + 1, device=dev)[None, :]
    prev = outs[0]
    for it in range(12):
        mid, new = outs[(2 * it + 1) % 3], outs[(2 * it + 2) % 3]
        # device: verify + update, then a plain step whose counts are the array the first kernel wrote
        target = torch.gather(seqs, 1, torch.clamp(pos[:, None] + ar, max=total - 1)).int().contiguous()
        cap = ((total - pos) // 2).int().contiguous()
        P.binding.sam_step_verified(batch.handle, target, prev.draft_tokens, prev.draft_len, cap, L,
                                    *mid.tensors(), counts_out=cnt, accepted_out=acc)
        again = torch.gather(seqs, 1, torch.clamp(pos[:, None] + cnt.long()[:, None] + ar, max=total - 1)).int().contiguous()
        batch.step(again, cnt, L, new)
        pos += 2 * cnt.long()
        # oracle, the same two updates
        idx = np.minimum(r_pos[:, None] + np.arange(L + 1)[None, :], total - 1)
        r_nt, r_cnt, r_acc = accept.accept_greedy(r_out.draft_tokens, r_out.draft_len,
                                                  np.take_along_axis(w.seqs, idx, axis=1), (total - r_pos) // 2, L + 1)
        r_mid = ob.step(r_nt, r_cnt, L)
        idx2 = np.minimum(r_pos[:, None] + r_cnt[:, None] + np.arange(L + 1)[None, :], total - 1)
        r_new = ob.step(np.ascontiguousarray(np.take_along_axis(w.seqs, idx2, axis=1)), r_cnt, L)
        r_pos += 2 * r_cnt
        assert np.array_equal(cnt.cpu().numpy(), r_cnt) and np.array_equal(acc.cpu().numpy(), r_acc), it
        gm, gn = mid.cpu(), new.cpu()
        for k in ("draft_tokens", "draft_len", "match_len", "source", "state", "status"):
            assert np.array_equal(gm[k], getattr(r_mid, k)), (it, "verified", k)
            assert np.array_equal(gn[k], getattr(r_new, k)), (it, "plain", k)
        prev, r_out = new, r_new
    assert np.array_equal(pos.cpu().numpy(), r_pos) and (r_pos > pl).all()
