"""CPU model of the step kernel's "repeat run" (csrc/step.cu, dyn_repeat_run) against plain Expand.

The kernel extends several tokens of a repeated passage at once: it guesses the states q_k that
Algorithm 3 would clone one after the other, checks the guess against their records, writes all new
states and every link[q_k] first, and only then runs the redirect walks, each from a record read
before any of those writes.  That this order gives the automaton Algorithm 3 gives is an argument
about suffix automata, not about CUDA, so it is checked here on the CPU: the same scheme written
over dictionaries, against a literal Expand, on random texts over tiny vocabularies (where repeats
overlap themselves and periodic stretches are common).  The model is test code of its own: it
shares nothing with the oracle or the library.
"""
import random


class Sam:
    def __init__(self):
        self.len = [0]; self.link = [-1]; self.mep = [0]; self.next = [dict()]
        self.last = 0; self.n = 0; self.text = []; self.pstate = []

    def new(self, ln, link, mep, nx):
        self.len.append(ln); self.link.append(link); self.mep.append(mep); self.next.append(nx)
        return len(self.len) - 1

    def expand(self, t):
        """Algorithm 3, literally."""
        self.n += 1
        c = self.new(self.n, -1, self.n, {})
        p = self.last
        while p != -1 and t not in self.next[p]:
            self.next[p][t] = c; p = self.link[p]
        if p == -1:
            self.link[c] = 0
        else:
            q = self.next[p][t]
            if self.len[p] + 1 == self.len[q]:
                self.link[c] = q
            else:
                cl = self.new(self.len[p] + 1, self.link[q], self.mep[q], dict(self.next[q]))
                while p != -1 and self.next[p].get(t) == q:
                    self.next[p][t] = cl; p = self.link[p]
                self.link[q] = cl; self.link[c] = cl
        self.last = c
        self.text.append(t); self.pstate.append(c)

    def match(self):
        s = self.link[self.last]
        return (s, self.len[s]) if s > 0 else (0, 0)


def try_run(S, toks, deg_limit=2):
    """The kernel's scheme; returns the number of tokens it took (0: not applicable)."""
    s2, l0 = S.match()
    if s2 == 0 or len(toks) < 2:
        return 0
    nx = S.next[s2]
    if not 1 <= len(nx) <= deg_limit or toks[0] not in nx:
        return 0
    q0 = nx[toks[0]]
    if S.len[s2] + 1 == S.len[q0]:
        return 0                                             # solid: no clone
    e, ntok = S.mep[s2], S.n
    rmax = min(len(toks), ntok - e, 32)
    r = 0
    while r < rmax and S.text[e + r] == toks[r]:
        r += 1
    if r < 2:
        return 0
    # the guess: prefix states after e, or ids two apart from q0
    ps = [S.pstate[e + k] if S.pstate[e] == q0 else q0 + 2 * k for k in range(r)]
    rec = []
    for k in range(r):                                       # second read: the records, before any write
        if ps[k] >= len(S.len) or ps[k] == S.last:
            r = k
            break
        q = ps[k]
        rec.append((S.len[q], S.link[q], S.mep[q], dict(S.next[q])))
    for k in range(r):
        ln, _, mp, nxq = rec[k]
        if not (len(nxq) <= deg_limit and mp == e + 1 + k and ln > l0 + k + 1):
            r = k
            break
    for k in range(r - 1):
        nxq = rec[k][3]
        if not (toks[k + 1] in nxq and nxq[toks[k + 1]] == ps[k + 1]):
            r = k + 1
            break
    if r < 2:
        return 0
    u = [S.link[s2]] + [rec[k - 1][1] for k in range(1, r)]  # where each walk starts
    for k in range(r):                                       # a walk's first record must not be a q_k
        if u[k] > 0:
            kk = S.mep[u[k]] - e - 1
            if 0 <= kk < r and ps[kk] == u[k]:
                r = k
                break
    if r < 2:
        return 0
    first = [dict(S.next[x]) if x > 0 else None for x in u[:r]]   # third read, still before any write
    n0, last = len(S.len), S.last
    for k in range(r):                                       # new states, side by side
        S.new(ntok + k + 1, -1, ntok + k + 1, {})
        S.new(l0 + 1 + k, rec[k][1], rec[k][2], dict(rec[k][3]))
    for k in range(r):
        ck = n0 + 2 * k; cl = ck + 1
        prev = last if k == 0 else ck - 2
        S.next[prev][toks[k]] = ck
        S.link[prev] = s2 if k == 0 else cl - 2
        if k < r - 1:
            S.next[cl][toks[k + 1]] = cl + 2
        S.link[ps[k]] = cl
        S.text.append(toks[k]); S.pstate.append(ck)
    S.next[s2][toks[0]] = n0 + 1
    for k in range(r):                                       # the walks, one after the other
        pp, q, cl, t = u[k], ps[k], n0 + 2 * k + 1, toks[k]
        at_first = True
        while pp != -1:
            nxp = first[k] if (at_first and pp > 0) else S.next[pp]
            at_first = False
            if nxp.get(t) != q:
                break
            S.next[pp][t] = cl; pp = S.link[pp]
    S.last = n0 + 2 * (r - 1); S.link[S.last] = S.last + 1; S.n = ntok + r
    return r


def same(A, B):
    return A.len == B.len and A.link == B.link and A.mep == B.mep and A.next == B.next and A.last == B.last


def test_repeat_run_scheme_equals_expand():
    rng = random.Random(20241110)
    runs = tokens_in_runs = 0
    for trial in range(1500):
        vocab = rng.choice([2, 3, 5])
        n = rng.choice([20, 60, 150])
        x = []
        while len(x) < n:
            if x and rng.random() < 0.4:
                s = rng.randrange(len(x))
                for i in range(rng.randint(2, 30)):
                    x.append(x[s + i])                       # may run into what it has just appended
            else:
                x.append(rng.randrange(vocab))
        x = x[:n]
        A, B = Sam(), Sam()
        i = 0
        while i < n:
            m = min(rng.randint(1, 40), n - i)
            toks, j = x[i:i + m], 0
            while j < m:
                r = try_run(B, toks[j:])
                if r:
                    runs += 1; tokens_in_runs += r
                    for t in toks[j:j + r]:
                        A.expand(t)
                    j += r
                else:
                    A.expand(toks[j]); B.expand(toks[j]); j += 1
                assert same(A, B), (trial, i + j, r, x[:i + j])
            i += m
    assert runs > 1000 and tokens_in_runs > 3 * runs          # the scheme was exercised, with long runs too
