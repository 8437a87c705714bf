"""Seeded synthetic workloads for batched suffix-automaton draft retrieval.

Only inputs are made here (corpus, prompts, generated tokens, accepted-token counts per
decoding step); nothing in this package knows what a suffix automaton is.  The arrays it
returns feed the CPU oracle and the CUDA library alike.

The five named workloads follow the shapes of a speculative-decoding deployment: Zipf-skewed
token ids, verbatim repeated spans (what makes retrieval hit), prompt-copy-heavy generation,
1..16 accepted tokens per step, draft lengths 16..40.  They are synthetic stand-ins; no item of
any public benchmark or corpus is reproduced.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field, replace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "samgen.c")
_LIB = os.path.join(_HERE, "libsamgen.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile samgen.c into libsamgen.so next to it (gcc, a second or two)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32p = ctypes.POINTER(ctypes.c_int32)
        lib.samgen_model_new.restype = ctypes.c_void_p
        lib.samgen_model_new.argtypes = [ctypes.c_int32, ctypes.c_double, ctypes.c_int32, ctypes.c_uint64]
        lib.samgen_model_free.argtypes = [ctypes.c_void_p]
        lib.samgen_corpus.argtypes = [ctypes.c_void_p, i32p, ctypes.c_int64, ctypes.c_double,
                                      ctypes.c_int32, ctypes.c_int32, ctypes.c_uint64]
        lib.samgen_join_documents.restype = ctypes.c_int64
        lib.samgen_join_documents.argtypes = [i32p, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                              ctypes.c_int32, ctypes.c_uint64]
        lib.samgen_sequences.argtypes = [ctypes.c_void_p, i32p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                         i32p, ctypes.c_int64, ctypes.c_double, ctypes.c_double,
                                         ctypes.c_double, ctypes.c_double, ctypes.c_int32,
                                         ctypes.c_int32, ctypes.c_int32, ctypes.c_uint64]
        lib.samgen_schedule.restype = ctypes.c_int32
        lib.samgen_schedule.argtypes = [i32p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                        ctypes.c_int32, ctypes.c_int32, ctypes.c_double, ctypes.c_uint64]
        lib.samgen_pack_steps.argtypes = [i32p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                          i32p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, i32p]
        _lib = lib
    return _lib


def _p(a: np.ndarray):
    assert a.dtype == np.int32 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


@dataclass(frozen=True)
class Spec:
    """Recipe of one workload.  Fractions are expected shares of positions covered by copies."""
    name: str
    corpus_len: int
    vocab: int
    zipf_s: float
    markov: bool
    corpus_copy_frac: float
    span_lo: int
    span_hi: int
    batch: int
    prompt_len: int
    gen_len: int
    prompt_copy_frac: float        # copies inside the prompt
    prompt_p_corpus: float         # share of the prompt's copies that read the corpus (rest: own text)
    gen_copy_frac: float           # copies inside the generated part
    gen_p_corpus: float            # share of those that read the corpus (rest: own text)
    gen_own_prompt_only: bool      # own-text copies of the generated part read the prompt only
    accept_kind: str               # "uniform" or "geometric"
    accept_max: int
    accept_p: float
    draft_len: int
    unrelated_corpus: bool = False  # corpus drawn with another permutation: no useful static hits
    seed: int = 0
    doc_lo: int = 0                # > 0: the corpus is documents of U[doc_lo, doc_hi] tokens joined by `eos`
    doc_hi: int = 0
    eos: int = -1                  # the separator's token id (also the drafts' stop token)


# The five recipes, smallest first; seeds are 0x5A4D0000 + position.
SPECS = {
    "tiny": Spec("tiny", 100_000, 32000, 1.1, False, 0.30, 8, 64, 4, 256, 512,
                 0.40, 0.5, 0.40, 0.5, False, "uniform", 4, 0.0, 16, seed=0x5A4D0000),
    "c2": Spec("c2", 10_000_000, 32000, 1.1, True, 0.25, 8, 128, 64, 1024, 2048,
               0.35, 0.5, 0.35, 0.5, False, "geometric", 8, 0.4, 32, seed=0x5A4D0001),
    "c3": Spec("c3", 100_000_000, 128256, 1.05, False, 0.20, 16, 256, 256, 2048, 4096,
               0.30, 0.5, 0.30, 0.5, False, "geometric", 8, 0.35, 32, seed=0x5A4D0002),
    "c4": Spec("c4", 1_000_000, 32000, 1.1, False, 0.0, 8, 64, 1024, 4096, 2048,
               0.0, 0.0, 0.60, 0.0, True, "geometric", 12, 0.25, 40, unrelated_corpus=True,
               seed=0x5A4D0003),
    "c5": Spec("c5", 200_000_000, 128256, 1.05, True, 0.25, 8, 256, 4096, 2048, 2048,
               0.40, 0.5, 0.40, 0.5, True, "geometric", 16, 0.3, 32, seed=0x5A4D0004),
}

# A sixth recipe, not one of the five benchmark configurations: c2's shape over a corpus that is many
# documents joined by an end-of-sequence token (id vocab - 1), the way a retrieval corpus is put
# together from separate texts.  Run with the stop token set to `eos`, so that no draft crosses a
# document boundary.
DOCS = Spec("docs", 4_000_000, 32000, 1.1, True, 0.25, 8, 128, 64, 1024, 2048,
            0.35, 0.5, 0.35, 0.5, False, "geometric", 8, 0.4, 32, seed=0x5A4D0005,
            doc_lo=40, doc_hi=1200, eos=31999)


def scaled(spec: Spec, corpus_len=None, batch=None, prompt_len=None, gen_len=None, seed=None) -> Spec:
    """A smaller (or differently seeded) instance of the same recipe."""
    kw = {}
    if corpus_len is not None:
        kw["corpus_len"] = int(corpus_len)
    if batch is not None:
        kw["batch"] = int(batch)
    if prompt_len is not None:
        kw["prompt_len"] = int(prompt_len)
    if gen_len is not None:
        kw["gen_len"] = int(gen_len)
    if seed is not None:
        kw["seed"] = int(seed)
    return replace(spec, **kw)


@dataclass
class Workload:
    spec: Spec
    corpus: np.ndarray        # int32 [N]
    seqs: np.ndarray          # int32 [B, P+G] full text of every sequence
    counts: np.ndarray        # int32 [S, B] accepted tokens per generation step (0 = finished)
    new_tokens: np.ndarray    # int32 [S, B, K] tokens of each step, -1 padded
    meta: dict = field(default_factory=dict)

    @property
    def prompts(self) -> np.ndarray:
        return np.ascontiguousarray(self.seqs[:, : self.spec.prompt_len])

    @property
    def n_steps(self) -> int:
        return int(self.counts.shape[0])

    @property
    def seq_steps(self) -> int:
        """Sequence-steps of the generation phase: non-empty (step, sequence) pairs."""
        return int((self.counts > 0).sum())


def make_corpus(spec: Spec) -> np.ndarray:
    lib = _load()
    seed = spec.seed ^ (0xC0FFEE if spec.unrelated_corpus else 0)
    model = lib.samgen_model_new(spec.vocab, spec.zipf_s, int(spec.markov), seed)
    try:
        corpus = np.empty(spec.corpus_len, dtype=np.int32)
        lib.samgen_corpus(model, _p(corpus), spec.corpus_len, spec.corpus_copy_frac,
                          spec.span_lo, spec.span_hi, seed)
        if spec.doc_lo > 0:
            lib.samgen_join_documents(_p(corpus), spec.corpus_len, spec.vocab, spec.eos, spec.doc_lo, spec.doc_hi, seed)
    finally:
        lib.samgen_model_free(model)
    return corpus


def make_sequences(spec: Spec, corpus: np.ndarray, rank: int = 0, world: int = 1):
    """Sequences, counts and per-step token rows for the slice of the batch that `rank` owns.

    The batch is split into `world` contiguous shards; each sequence is drawn from its own
    random stream keyed by its global index, so a shard's content does not depend on `world`."""
    lib = _load()
    lo_b, hi_b = shard_bounds(spec.batch, rank, world)
    model = lib.samgen_model_new(spec.vocab, spec.zipf_s, int(spec.markov), spec.seed)
    try:
        full = np.empty((spec.batch, spec.prompt_len + spec.gen_len), dtype=np.int32)
        # streams are keyed by row index, so generate all rows of the (small) batch and slice
        lib.samgen_sequences(model, _p(full), spec.batch, spec.prompt_len, spec.gen_len,
                             _p(corpus), corpus.shape[0],
                             spec.prompt_copy_frac, spec.prompt_p_corpus,
                             spec.gen_copy_frac, spec.gen_p_corpus, int(spec.gen_own_prompt_only),
                             spec.span_lo, spec.span_hi, spec.seed)
    finally:
        lib.samgen_model_free(model)
    max_steps = spec.gen_len + 1
    counts = np.zeros((max_steps, spec.batch), dtype=np.int32)
    kind = 0 if spec.accept_kind == "uniform" else 1
    n_steps = lib.samgen_schedule(_p(counts), max_steps, spec.batch, spec.gen_len, kind,
                                  spec.accept_max, spec.accept_p, spec.seed)
    assert n_steps >= 0
    counts = np.ascontiguousarray(counts[:n_steps])
    new_tokens = np.empty((n_steps, spec.batch, spec.accept_max), dtype=np.int32)
    lib.samgen_pack_steps(_p(full), spec.batch, spec.prompt_len, spec.gen_len, _p(counts),
                          n_steps, spec.accept_max, -1, _p(new_tokens))
    seqs = np.ascontiguousarray(full[lo_b:hi_b])
    counts = np.ascontiguousarray(counts[:, lo_b:hi_b])
    new_tokens = np.ascontiguousarray(new_tokens[:, lo_b:hi_b])
    return seqs, counts, new_tokens


def shard_bounds(batch: int, rank: int, world: int):
    """Contiguous split of `batch` sequences over `world` ranks (first ranks get the remainder)."""
    base, rem = divmod(batch, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def make(spec_or_name, rank: int = 0, world: int = 1, corpus: np.ndarray | None = None) -> Workload:
    spec = SPECS[spec_or_name] if isinstance(spec_or_name, str) else spec_or_name
    if corpus is None:
        corpus = make_corpus(spec)
    seqs, counts, new_tokens = make_sequences(spec, corpus, rank, world)
    return Workload(spec, corpus, seqs, counts, new_tokens,
                    meta={"rank": rank, "world": world, "data": "synthetic"})
