"""Plain definition of the draft-retrieval results by exhaustive search — TEST INFRASTRUCTURE.

No automaton here.  For a sequence x_1..x_k and a reference text T (1-based positions, as in the
paper's Algorithm 3):

  static  (Section 3.2): l1 = the largest l such that the last l tokens of x occur in T;
                         e1 = the smallest end position of such an occurrence
                              (Section 3.1: min_endpos is the earliest position).
  dynamic (Section 3.3): the matcher is advanced on the automaton of x_1..x_{k-1}, i.e. before
                         x_k is added, so l2 = the largest l such that the last l tokens of x occur
                         in x ending at some position j <= k-1; e2 = the smallest such j.
  choice  (Section 3.2): static iff l1 > l2 + l_bias.
  draft   (Section 3.2): d = T[p+1 : p+n] with p the chosen end position, clipped at the text end.

A match of length 0 has end position 0 (the root's min_endpos, Appendix A.1).
Cost is O(len(T) * l) per query: for tiny inputs only.
"""
from __future__ import annotations


def common_suffix(a, ja: int, b, jb: int) -> int:
    """Length of the longest common suffix of a[0:ja] and b[0:jb]."""
    l = 0
    while l < ja and l < jb and a[ja - 1 - l] == b[jb - 1 - l]:
        l += 1
    return l


def longest_suffix_match(text, n_text: int, x, k: int, max_end: int):
    """(l, e): longest suffix of x[0:k] occurring in text[0:n_text] with 1-based end position
    e <= max_end, and the smallest such e.  (0, 0) when nothing matches."""
    best_l, best_e = 0, 0
    for j in range(1, min(n_text, max_end) + 1):
        l = common_suffix(text, j, x, k)
        if l > best_l:
            best_l, best_e = l, j
    return best_l, best_e


def retrieve(corpus, x, k: int, L: int, l_bias: int = 0, min_match: int = 1):
    """Everything one decoding step reports for the sequence x[0:k].

    Returns dict(l1, e1, l2, e2, source, draft) with source 0 none / 1 static / 2 dynamic."""
    n_corpus = 0 if corpus is None else len(corpus)
    l1, e1 = longest_suffix_match(corpus, n_corpus, x, k, n_corpus) if n_corpus else (0, 0)
    l2, e2 = longest_suffix_match(x, k, x, k, k - 1)
    use_static = l1 > l2 + l_bias
    l_sel = l1 if use_static else l2
    source, draft = 0, []
    if l_sel >= max(1, min_match):
        source = 1 if use_static else 2
        text, n_text, p = (corpus, n_corpus, e1) if use_static else (x, k, e2)
        draft = [int(v) for v in text[p:min(p + L, n_text)]]
    return dict(l1=l1, e1=e1, l2=l2, e2=e2, source=source, draft=draft)


def distinct_substrings(x) -> int:
    """Number of distinct non-empty substrings of x."""
    seen = set()
    n = len(x)
    for i in range(n):
        for j in range(i + 1, n + 1):
            seen.add(tuple(x[i:j]))
    return len(seen)


def endpos_classes(x) -> dict:
    """Map frozenset(end positions, 1-based) -> (longest substring length, earliest end position).

    The states of the suffix automaton of x other than the root are exactly these classes
    (Section 2.1: a node stands for all substrings with the same set of ending positions)."""
    n = len(x)
    ends = {}
    for i in range(n):
        for j in range(i + 1, n + 1):
            ends.setdefault(tuple(x[i:j]), set()).add(j)
    classes = {}
    for sub, e in ends.items():
        key = frozenset(e)
        cur = classes.get(key)
        if cur is None or len(sub) > cur[0]:
            classes[key] = (len(sub), min(e))
    return classes
