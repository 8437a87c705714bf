"""Greedy verification and auxiliary-draft selection, plainly — TEST INFRASTRUCTURE.

accept_greedy follows Section 2.2 of the paper: the target model evaluates the draft
x_draft = (x_{t+1} .. x_{t+n}) in one pass; the accepted tokens x_accept = (x_{t+1} .. x_{t+m}) are
the draft tokens that agree with what the target itself produces, followed by the target's own
next token.  With target[j] = the target's token for the position after the first j draft tokens,
the number of confirmed draft tokens is a = max{ j <= n : draft[i] == target[i] for all i < j } and
x_accept = target[0 .. a], so m = a + 1 (clipped to the row width and to an optional cap).

select_auxiliary follows Section 3.4: the auxiliary drafter has a fixed virtual match length
l_threshold; the automaton's draft is kept only if its match is at least that long (the batch's
min_match), otherwise the auxiliary draft is used.
"""
from __future__ import annotations

import numpy as np


def accept_greedy(draft, draft_len, target, max_new=None, stride=None):
    """draft [B, L], draft_len [B], target [B, L+1] -> (new_tokens [B, stride], counts [B], accepted [B])."""
    draft = np.asarray(draft); target = np.asarray(target)
    B, L = draft.shape
    stride = L + 1 if stride is None else stride
    new_tokens = np.full((B, stride), -1, dtype=np.int32)
    counts = np.zeros(B, dtype=np.int32)
    accepted = np.zeros(B, dtype=np.int32)
    for b in range(B):
        n = int(min(max(draft_len[b], 0), L))
        a = 0
        while a < n and draft[b, a] == target[b, a]:
            a += 1
        m = min(a + 1, stride)
        if max_new is not None:
            m = min(m, max(int(max_new[b]), 0))
        new_tokens[b, :m] = target[b, :m]
        counts[b] = m
        accepted[b] = min(a, m)
    return new_tokens, counts, accepted


def select_auxiliary(draft, draft_len, source, aux, aux_len):
    """In place on copies: where source == 0 and aux_len > 0 the auxiliary draft replaces the row."""
    draft = np.array(draft, dtype=np.int32); draft_len = np.array(draft_len, dtype=np.int32)
    source = np.array(source, dtype=np.int32)
    B, L = draft.shape
    for b in range(B):
        al = int(min(max(aux_len[b], 0), L))
        if source[b] == 0 and al > 0:
            draft[b, :] = -1
            draft[b, :al] = aux[b, :al]
            draft_len[b] = al
            source[b] = 3
    return draft, draft_len, source


def decode_loop(batch, seqs, prompt_len, L, stride, max_steps=100000):
    """Closed loop with the sequences' own continuation standing in for the target model:
    prefill, then draft -> verify -> accept -> update until every sequence is complete.
    `batch` is an oracle.Batch.  Returns a list of per-step dicts (outputs of the step that produced
    the draft, then counts / accepted of its verification) and the positions reached."""
    seqs = np.asarray(seqs, dtype=np.int32)
    B, total = seqs.shape
    out = batch.step(np.ascontiguousarray(seqs[:, :prompt_len]), np.full(B, prompt_len, dtype=np.int32), L)
    pos = np.full(B, prompt_len, dtype=np.int64)
    log = []
    for _ in range(max_steps):
        if (pos >= total).all():
            break
        idx = np.minimum(pos[:, None] + np.arange(L + 1)[None, :], total - 1)
        target = np.take_along_axis(seqs, idx, axis=1)
        new_tokens, counts, accepted = accept_greedy(out.draft_tokens, out.draft_len, target, total - pos, stride)
        log.append(dict(draft_tokens=out.draft_tokens.copy(), draft_len=out.draft_len.copy(), match_len=out.match_len.copy(),
                        source=out.source.copy(), state=out.state.copy(), status=out.status.copy(),
                        counts=counts.copy(), accepted=accepted.copy()))
        out = batch.step(new_tokens, counts, L)
        pos += counts
    return log, pos
