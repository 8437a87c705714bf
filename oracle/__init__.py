"""CPU oracle for batched suffix-automaton draft retrieval — TEST INFRASTRUCTURE.

`sam_oracle.c` is the algorithm exactly as the paper states it (Algorithms 1 and 3, Sections 3.2
and 3.3); `bruteforce.py` is the plain definition of the same results by exhaustive search.  This
package may be imported by the tests, by the smoke check and by the benchmark's CPU-baseline leg
only.  It imports nothing from the CUDA package and the CUDA package imports nothing from here.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sam_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None

_i32p = ctypes.POINTER(ctypes.c_int32)
_i64p = ctypes.POINTER(ctypes.c_int64)


def build(force: bool = False) -> str:
    """Compile sam_oracle.c (plain C, OpenMP only for the over-sequences loop)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    lib.osam_new.restype = vp
    lib.osam_new.argtypes = [i64]
    lib.osam_free.argtypes = [vp]
    lib.osam_expand.argtypes = [vp, i32]
    lib.osam_build.restype = vp
    lib.osam_build.argtypes = [_i32p, i64]
    lib.osam_transfer.argtypes = [vp, i32, _i32p, _i32p, _i64p]
    for name in ("osam_n_states", "osam_n_transitions"):
        getattr(lib, name).restype = i64
        getattr(lib, name).argtypes = [vp]
    lib.osam_last.restype = i32
    lib.osam_last.argtypes = [vp]
    lib.osam_err.restype = ctypes.c_int
    lib.osam_err.argtypes = [vp]
    for name in ("osam_link", "osam_length", "osam_min_endpos", "osam_deg"):
        getattr(lib, name).restype = i32
        getattr(lib, name).argtypes = [vp, i32]
    lib.osam_next.restype = i32
    lib.osam_next.argtypes = [vp, i32, i32]
    lib.osam_edges.argtypes = [vp, i32, _i32p, _i32p]
    lib.osam_tables.argtypes = [vp, _i32p, _i32p, _i32p, _i32p]
    lib.osam_counters.argtypes = [vp, _i64p]
    lib.osam_freq.argtypes = [vp, _i64p]
    lib.osam_topk.restype = i32
    lib.osam_topk.argtypes = [vp, _i64p, i32, i32, _i32p, _i32p]
    lib.obatch_new.restype = vp
    lib.obatch_new.argtypes = [vp, _i32p, i64, i32, i32, i32, i32, i32, i32]
    lib.obatch_free.argtypes = [vp]
    lib.obatch_reset.argtypes = [vp, i32]
    lib.obatch_step.restype = ctypes.c_int
    lib.obatch_step.argtypes = [vp, _i32p, i32, _i32p, i32, _i32p, _i32p, _i32p, _i32p, _i32p, _i32p, i32]
    lib.obatch_run.restype = ctypes.c_int
    lib.obatch_run.argtypes = [vp, _i32p, i32, _i32p, i32, i32, _i32p, _i32p, _i32p, _i32p, _i32p, _i32p, i32]
    lib.obatch_dyn.restype = vp
    lib.obatch_dyn.argtypes = [vp, i32]
    lib.obatch_len.restype = i32
    lib.obatch_len.argtypes = [vp, i32]
    lib.obatch_counters.argtypes = [vp, _i64p]
    _lib = lib
    return lib


def _p32(a: np.ndarray):
    assert a.dtype == np.int32 and a.flags["C_CONTIGUOUS"], (a.dtype, a.flags)
    return a.ctypes.data_as(_i32p)


class Sam:
    """One suffix automaton (Algorithm 3), states numbered in creation order."""

    def __init__(self, tokens=None, _handle=None, _owned=True):
        lib = _load()
        self._lib = lib
        self._owned = _owned
        if _handle is not None:
            self._h = _handle
        elif tokens is None:
            self._h = lib.osam_new(0)
        else:
            toks = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
            self._h = lib.osam_build(_p32(toks), toks.shape[0])          # Build-SAM
        if not self._h:
            raise MemoryError("oracle automaton allocation failed")

    def close(self):
        if self._h and self._owned:
            self._lib.osam_free(self._h)
        self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def expand(self, t: int):
        self._lib.osam_expand(self._h, int(t))                            # Expand

    def transfer(self, t: int, s: int, l: int):
        """Transfer (Algorithm 1): returns (s, l, link_moves, next_moves)."""
        cs, cl = ctypes.c_int32(s), ctypes.c_int32(l)
        mv = (ctypes.c_int64 * 2)(0, 0)
        self._lib.osam_transfer(self._h, int(t), ctypes.byref(cs), ctypes.byref(cl), mv)
        return cs.value, cl.value, mv[0], mv[1]

    @property
    def n_states(self) -> int:
        return self._lib.osam_n_states(self._h)

    @property
    def n_transitions(self) -> int:
        return self._lib.osam_n_transitions(self._h)

    @property
    def last(self) -> int:
        return self._lib.osam_last(self._h)

    @property
    def err(self) -> int:
        return self._lib.osam_err(self._h)

    def link(self, s):
        return self._lib.osam_link(self._h, s)

    def length(self, s):
        return self._lib.osam_length(self._h, s)

    def min_endpos(self, s):
        return self._lib.osam_min_endpos(self._h, s)

    def next(self, s, t):
        return self._lib.osam_next(self._h, s, t)

    def edges(self, s) -> dict:
        d = self._lib.osam_deg(self._h, s)
        toks = np.empty(max(d, 1), dtype=np.int32)
        tgts = np.empty(max(d, 1), dtype=np.int32)
        self._lib.osam_edges(self._h, s, _p32(toks), _p32(tgts))
        return {int(toks[i]): int(tgts[i]) for i in range(d)}

    def tables(self):
        """(link, length, min_endpos, deg) as int32 arrays of n_states entries."""
        n = self.n_states
        out = [np.empty(n, dtype=np.int32) for _ in range(4)]
        self._lib.osam_tables(self._h, *[_p32(a) for a in out])
        return tuple(out)

    def counters(self) -> dict:
        c = (ctypes.c_int64 * 4)()
        self._lib.osam_counters(self._h, c)
        return dict(walk_inserts=c[0], clones=c[1], copied_edges=c[2], redirects=c[3])

    def freq(self) -> np.ndarray:
        """freq of every state (Appendix A.1/A.2): occurrences of its substrings in the text."""
        f = np.zeros(self.n_states, dtype=np.int64)
        self._lib.osam_freq(self._h, f.ctypes.data_as(_i64p))
        return f

    def topk(self, freq: np.ndarray, s: int, k: int):
        """Top-k successors of s by freq: list of (token, target)."""
        toks = np.empty(max(k, 1), dtype=np.int32)
        tgts = np.empty(max(k, 1), dtype=np.int32)
        n = self._lib.osam_topk(self._h, freq.ctypes.data_as(_i64p), int(s), int(k), _p32(toks), _p32(tgts))
        return [(int(toks[i]), int(tgts[i])) for i in range(n)]


class StepOut:
    __slots__ = ("draft_tokens", "draft_len", "match_len", "source", "state", "status")

    def __init__(self, batch, L):
        self.draft_tokens = np.empty((batch, L), dtype=np.int32)
        self.draft_len = np.empty(batch, dtype=np.int32)
        self.match_len = np.empty((batch, 2), dtype=np.int32)
        self.source = np.empty(batch, dtype=np.int32)
        self.state = np.empty((batch, 2), dtype=np.int32)
        self.status = np.empty(batch, dtype=np.int32)

    def ptrs(self):
        return [_p32(getattr(self, k)) for k in self.__slots__]


class Batch:
    """B decoding sequences over one shared static automaton (Sections 3.2, 3.3)."""

    def __init__(self, static: Sam | None, corpus, batch: int, vocab: int, max_seq_len: int,
                 l_bias: int = 0, min_match: int = 1, stop_token: int = -1):
        lib = _load()
        self._lib = lib
        self._static = static
        self._corpus = None if corpus is None else np.ascontiguousarray(np.asarray(corpus, dtype=np.int32))
        self.batch = batch
        cp = _p32(self._corpus) if self._corpus is not None else ctypes.cast(None, _i32p)
        cn = 0 if self._corpus is None else self._corpus.shape[0]
        self._h = lib.obatch_new(static._h if static is not None else None, cp, cn,
                                 batch, vocab, max_seq_len, l_bias, min_match, stop_token)

    def close(self):
        if self._h:
            self._lib.obatch_free(self._h)
        self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self, slot: int):
        self._lib.obatch_reset(self._h, int(slot))

    def step(self, new_tokens, counts, L: int, threads: int = 1) -> StepOut:
        nt = np.ascontiguousarray(np.asarray(new_tokens, dtype=np.int32)).reshape(self.batch, -1)
        ct = np.ascontiguousarray(np.asarray(counts, dtype=np.int32))
        out = StepOut(self.batch, L)
        err = self._lib.obatch_step(self._h, _p32(nt), nt.shape[1], _p32(ct), L, *out.ptrs(), threads)
        if err:
            raise AssertionError("oracle self-check failed (err %d)" % err)
        return out

    def run(self, new_tokens, counts, L: int, threads: int = 1) -> StepOut:
        """All steps of new_tokens [S, B, K] / counts [S, B] in one call; outputs of the last step."""
        nt = np.ascontiguousarray(np.asarray(new_tokens, dtype=np.int32))
        ct = np.ascontiguousarray(np.asarray(counts, dtype=np.int32))
        assert nt.ndim == 3 and nt.shape[1] == self.batch and ct.shape == nt.shape[:2]
        out = StepOut(self.batch, L)
        err = self._lib.obatch_run(self._h, _p32(nt), nt.shape[2], _p32(ct), nt.shape[0], L, *out.ptrs(), threads)
        if err:
            raise AssertionError("oracle self-check failed (err %d)" % err)
        return out

    def dynamic(self, b: int) -> Sam:
        return Sam(_handle=self._lib.obatch_dyn(self._h, b), _owned=False)

    def seq_len(self, b: int) -> int:
        return self._lib.obatch_len(self._h, b)

    def counters(self) -> dict:
        c = (ctypes.c_int64 * 13)()
        self._lib.obatch_counters(self._h, c)
        keys = ("static_link_moves", "static_next_moves", "dynamic_link_moves", "dynamic_next_moves",
                "tokens", "draft_tokens", "seq_steps", "walk_inserts", "clones", "copied_edges",
                "redirects", "dyn_states", "dyn_transitions")
        return {k: int(c[i]) for i, k in enumerate(keys)}
