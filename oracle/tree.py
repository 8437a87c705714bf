"""Tree drafts from the static automaton (Appendix A.2, Algorithm 5) — TEST INFRASTRUCTURE.

prim_tree follows Algorithm 5: a priority queue ordered by probability starts with
(1.0, s, start token); while the queue is not empty and the draft has fewer than MAX_SIZE nodes, the
most probable entry is popped and appended, and its top-k successors are pushed with probability
p * topk_prob, topk_prob = freq(successor) / freq(state).

Readings where the paper is silent: probabilities are IEEE float32, the quotient rounded first and
then the product; among equal probabilities the entry pushed earlier is popped first; successors
are pushed in top-k order (freq descending, token ascending); the output also records each node's
parent (the tree a verification mask needs), which the paper's list of tokens leaves implicit.
"""
from __future__ import annotations

import numpy as np


def prim_tree(sam, freq, s: int, start_token: int, max_size: int, k: int):
    """Returns (tokens, parents, probs) lists of at most max_size nodes; node 0 is the start token."""
    f32 = np.float32
    queue = [(f32(1.0), int(s), int(start_token), -1)]       # (p, state, token, parent), in push order
    alive = [True]
    tokens, parents, probs = [], [], []
    while any(alive) and len(tokens) != max_size:
        best = -1
        for i, (p, _, _, _) in enumerate(queue):
            if alive[i] and (best < 0 or p > queue[best][0]):   # strict: the earlier push wins ties
                best = i
        p, state, tok, parent = queue[best]
        alive[best] = False
        node = len(tokens)
        tokens.append(tok); parents.append(parent); probs.append(p)
        fs = f32(freq[state])
        for t_n, s_n in sam.topk(freq, state, k):
            p_n = f32(freq[s_n]) / fs
            queue.append((f32(p * p_n), s_n, t_n, node))
            alive.append(True)
    return tokens, parents, probs
