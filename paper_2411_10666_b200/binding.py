"""ctypes binding of libsamdraft.so: the same calls as include/samdraft.h, argument marshalling only.

Every step of the retrieval path runs inside the CUDA library.  PyTorch is used here for device
memory (the batch workspace and the I/O tensors) and for the current stream, nothing else.  If the
library cannot be built or loaded this module raises; there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_double, c_int, c_int32, c_int64, c_size_t, c_void_p

import numpy as np

from . import _build

_lib = None

SAM_OK = 0
ERR_NAMES = {-1: "ARG", -2: "CUDA", -3: "NOMEM", -4: "WORKSPACE", -5: "IO", -6: "FORMAT", -7: "LIMIT", -8: "NO_DEVICE"}
SEQ_OK, SEQ_CAPACITY, SEQ_WALK_LIMIT, SEQ_BAD_TOKEN, SEQ_BAD_COUNT = 0, 1, 2, 3, 4
SRC_NONE, SRC_STATIC, SRC_DYNAMIC, SRC_AUXILIARY = 0, 1, 2, 3


class SamError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        msg = lib().sam_strerror(code).decode()
        extra = ""
        if code == -2:
            extra = " (cudaError %d)" % lib().sam_last_cuda_error()
        super().__init__("%s: %s [%s]%s" % (what, msg, ERR_NAMES.get(code, code), extra))


class BuildOpts(Structure):
    _fields_ = [("hash_load", c_double), ("keep_host_copy", c_int32), ("tree_topk", c_int32)]


class StaticInfo(Structure):
    _fields_ = [("n_tokens", c_int64), ("n_states", c_int64), ("n_transitions", c_int64),
                ("n_hash_edges", c_int64), ("hash_buckets", c_int64), ("hash_max_probe", c_int32),
                ("vocab", c_int32), ("device_bytes", c_size_t), ("build_seconds", c_double),
                ("tree_topk", c_int32), ("reserved", c_int32)]


class BatchOpts(Structure):
    _fields_ = [("batch", c_int32), ("max_seq_len", c_int32), ("max_draft_len", c_int32),
                ("l_bias", c_int32), ("min_match", c_int32), ("vocab", c_int32),
                ("max_host_stride", c_int32), ("slab_bytes", c_int32), ("pool_slabs", c_int64),
                ("stop_token_plus_one", c_int32), ("reserved", c_int32)]


_i32p = POINTER(c_int32)

# name -> (restype, argtypes); every symbol include/samdraft.h declares
SIGNATURES = {
    "sam_build_static": (c_int, [c_void_p, c_int64, c_int32, c_int, POINTER(BuildOpts), POINTER(c_void_p)]),
    "sam_static_save": (c_int, [c_void_p, c_char_p]),
    "sam_static_load": (c_int, [c_char_p, c_int, POINTER(c_void_p)]),
    "sam_static_info": (c_int, [c_void_p, POINTER(StaticInfo)]),
    "sam_static_state": (c_int, [c_void_p, c_int64, _i32p, _i32p, _i32p, _i32p, c_void_p, c_void_p, c_int32]),
    "sam_static_tables": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int64]),
    "sam_build_static_tables": (c_int, [c_void_p, c_int64, c_int32, POINTER(c_int64), POINTER(c_int64), _i32p,
                                        c_void_p, c_void_p, c_void_p, c_void_p, c_int64,
                                        c_void_p, c_void_p, c_void_p, c_int64]),
    "sam_static_destroy": (None, [c_void_p]),
    "sam_batch_workspace_bytes": (c_int, [POINTER(BatchOpts), POINTER(c_size_t)]),
    "sam_batch_create": (c_int, [c_void_p, POINTER(BatchOpts), c_void_p, c_size_t, c_void_p, POINTER(c_void_p)]),
    "sam_batch_reset": (c_int, [c_void_p, c_void_p, c_int32, c_void_p]),
    "sam_step": (c_int, [c_void_p, c_void_p, c_int32, c_void_p, c_int32,
                         c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "sam_run_steps": (c_int, [c_void_p, c_void_p, c_int32, c_void_p, c_int32, c_int32, c_int32,
                              c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "sam_step_host": (c_int, [c_void_p, c_void_p, c_int32, c_void_p, c_int32,
                              c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "sam_batch_dump": (c_int, [c_void_p, c_int32, _i32p, _i32p, _i32p, c_void_p, c_void_p, c_void_p, c_void_p,
                               c_int32, c_void_p, c_void_p, c_void_p, c_int32, c_void_p]),
    "sam_batch_pool_info": (c_int, [c_void_p, POINTER(c_int64), POINTER(c_int64), c_void_p]),
    "sam_batch_launches_per_step": (c_int, [c_void_p]),
    "sam_batch_destroy": (None, [c_void_p]),
    "sam_accept_greedy": (c_int, [c_int32, c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_void_p, c_int32,
                                  c_void_p, c_void_p, c_void_p]),
    "sam_step_verified": (c_int, [c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_void_p, c_int32,
                                  c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "sam_select_auxiliary": (c_int, [c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "sam_tree_draft": (c_int, [c_void_p, c_int32, c_void_p, c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_void_p,
                               c_void_p, c_void_p]),
    "sam_static_freq": (c_int, [c_void_p, c_void_p, c_int64]),
    "sam_retrieve_noalloc": (c_int, [c_void_p, c_int32, c_int32, c_void_p, c_int32, c_void_p, c_int32, c_int32, c_int32,
                                     c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "sam_noalloc_capacity_bytes": (c_size_t, []),
    "sam_probe_random_read": (c_int, [c_void_p, c_size_t, c_int32, c_int32, c_void_p, POINTER(c_double), POINTER(c_double)]),
    "sam_probe_chase": (c_int, [c_void_p, c_size_t, c_int64, c_int32, c_void_p, POINTER(c_double)]),
    "sam_strerror": (c_char_p, [c_int]),
    "sam_last_cuda_error": (c_int, []),
    "sam_version": (c_char_p, []),
    "sam_counters_available": (c_int, []),
    "sam_counters_attach": (c_int, [c_void_p, c_int32]),
}


def lib():
    """The loaded library (built on first use).  Raises if it cannot be built or loaded."""
    global _lib
    if _lib is None:
        path = _build.build()
        L = ctypes.CDLL(path)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)          # AttributeError if the symbol is missing
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def _check(rc: int, what: str):
    if rc != SAM_OK:
        raise SamError(rc, what)


def _np32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _dev_ptr(t, name: str):
    import torch
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.int32 and t.is_contiguous()):
        raise TypeError("%s must be a contiguous int32 CUDA tensor" % name)
    return t.data_ptr()


def _stream_ptr(stream=None):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


# ---------------------------------------------------------------------------------------------
# thin wrappers, one per C call
# ---------------------------------------------------------------------------------------------

def sam_build_static(corpus_host, vocab: int, device: int = 0, hash_load: float = 0.0, tree_topk: int = 0):
    corpus = _np32(corpus_host)
    opts = BuildOpts(hash_load, 0, tree_topk)
    h = c_void_p()
    _check(lib().sam_build_static(corpus.ctypes.data, corpus.shape[0], vocab, device, byref(opts), byref(h)),
           "sam_build_static")
    return h


def sam_static_info(h) -> StaticInfo:
    info = StaticInfo()
    _check(lib().sam_static_info(h, byref(info)), "sam_static_info")
    return info


def sam_static_save(h, path: str):
    _check(lib().sam_static_save(h, path.encode()), "sam_static_save")


def sam_static_load(path: str, device: int = 0):
    h = c_void_p()
    _check(lib().sam_static_load(path.encode(), device, byref(h)), "sam_static_load")
    return h


def sam_static_destroy(h):
    lib().sam_static_destroy(h)


def sam_static_state(h, state: int, max_edges: int = 64):
    ln, lk, ep, ne = c_int32(), c_int32(), c_int32(), c_int32()
    toks = np.empty(max(max_edges, 1), dtype=np.int32)
    tgts = np.empty(max(max_edges, 1), dtype=np.int32)
    _check(lib().sam_static_state(h, state, byref(ln), byref(lk), byref(ep), byref(ne),
                                  toks.ctypes.data, tgts.ctypes.data, max_edges), "sam_static_state")
    k = min(ne.value, max_edges)
    return dict(length=ln.value, link=lk.value, min_endpos=ep.value, deg=ne.value,
                next={int(toks[i]): int(tgts[i]) for i in range(k)})


def sam_static_tables(h):
    n = sam_static_info(h).n_states
    out = [np.empty(n, dtype=np.int32) for _ in range(4)]
    _check(lib().sam_static_tables(h, *[a.ctypes.data for a in out], n), "sam_static_tables")
    return dict(length=out[0], link=out[1], min_endpos=out[2], deg=out[3])


def sam_build_static_tables(corpus_host, vocab: int):
    """Host-only construction decoded into flat tables (no device)."""
    corpus = _np32(corpus_host)
    ns, nt, mp = c_int64(), c_int64(), c_int32()
    _check(lib().sam_build_static_tables(corpus.ctypes.data, corpus.shape[0], vocab, byref(ns), byref(nt), byref(mp),
                                         None, None, None, None, 0, None, None, None, 0), "sam_build_static_tables")
    st = [np.empty(ns.value, dtype=np.int32) for _ in range(4)]
    ed = [np.empty(nt.value, dtype=np.int32) for _ in range(3)]
    _check(lib().sam_build_static_tables(corpus.ctypes.data, corpus.shape[0], vocab, byref(ns), byref(nt), byref(mp),
                                         *[a.ctypes.data for a in st], ns.value,
                                         *[a.ctypes.data for a in ed], nt.value), "sam_build_static_tables")
    return dict(length=st[0], link=st[1], min_endpos=st[2], deg=st[3],
                edge_src=ed[0], edge_tok=ed[1], edge_tgt=ed[2], hash_max_probe=mp.value)


def sam_batch_workspace_bytes(opts: BatchOpts) -> int:
    out = c_size_t()
    _check(lib().sam_batch_workspace_bytes(byref(opts), byref(out)), "sam_batch_workspace_bytes")
    return out.value


def sam_batch_create(static_h, opts: BatchOpts, workspace, stream=None):
    import torch
    assert isinstance(workspace, torch.Tensor) and workspace.is_cuda and workspace.dtype == torch.uint8
    h = c_void_p()
    _check(lib().sam_batch_create(static_h, byref(opts), workspace.data_ptr(), workspace.numel(),
                                  _stream_ptr(stream), byref(h)), "sam_batch_create")
    return h


def sam_batch_reset(h, slots=None, stream=None):
    if slots is None:
        _check(lib().sam_batch_reset(h, None, -1, _stream_ptr(stream)), "sam_batch_reset")
    else:
        s = _np32(slots)
        _check(lib().sam_batch_reset(h, s.ctypes.data, s.shape[0], _stream_ptr(stream)), "sam_batch_reset")


def sam_batch_destroy(h):
    lib().sam_batch_destroy(h)


def sam_step(h, new_tokens, stride, counts, L, draft_tokens, draft_len, match_len, source, state, status, stream=None):
    _check(lib().sam_step(h, _dev_ptr(new_tokens, "new_tokens"), stride, _dev_ptr(counts, "counts"), L,
                          _dev_ptr(draft_tokens, "draft_tokens"), _dev_ptr(draft_len, "draft_len"),
                          _dev_ptr(match_len, "match_len"), _dev_ptr(source, "source"),
                          _dev_ptr(state, "state"), _dev_ptr(status, "status"), _stream_ptr(stream)), "sam_step")


def sam_run_steps(h, new_tokens, stride, counts, n_steps, L, out_per_step,
                  draft_tokens, draft_len, match_len, source, state, status, stream=None):
    _check(lib().sam_run_steps(h, _dev_ptr(new_tokens, "new_tokens"), stride, _dev_ptr(counts, "counts"),
                               n_steps, L, int(out_per_step),
                               _dev_ptr(draft_tokens, "draft_tokens"), _dev_ptr(draft_len, "draft_len"),
                               _dev_ptr(match_len, "match_len"), _dev_ptr(source, "source"),
                               _dev_ptr(state, "state"), _dev_ptr(status, "status"), _stream_ptr(stream)),
           "sam_run_steps")


def _host_ptr(t, name):
    """Host buffer: a numpy int32 array, a CPU (ideally pinned) int32 torch tensor, or a plain int
    that is taken as the buffer's address (for loops that precompute their pointers)."""
    if t is None or isinstance(t, int):
        return t
    import torch
    if isinstance(t, np.ndarray):
        assert t.dtype == np.int32 and t.flags["C_CONTIGUOUS"], name
        return t.ctypes.data
    assert isinstance(t, torch.Tensor) and not t.is_cuda and t.dtype == torch.int32 and t.is_contiguous(), name
    return t.data_ptr()


def sam_step_host(h, new_tokens, stride, counts, L, draft_tokens, draft_len, match_len, source, state, status,
                  stream=None):
    _check(lib().sam_step_host(h, _host_ptr(new_tokens, "new_tokens"), stride, _host_ptr(counts, "counts"), L,
                               _host_ptr(draft_tokens, "draft_tokens"), _host_ptr(draft_len, "draft_len"),
                               _host_ptr(match_len, "match_len"), _host_ptr(source, "source"),
                               _host_ptr(state, "state"), _host_ptr(status, "status"), _stream_ptr(stream)),
           "sam_step_host")


def sam_step_host_prepared(h, stride, L, draft_tokens, draft_len, match_len, source, state, status, stream=None):
    """The same call as sam_step_host for a loop that makes it every step: whatever does not change
    from step to step (the output arrays, stride, L, the stream) is converted once, and the returned
    function takes the step's new_tokens and counts (arrays, or plain addresses)."""
    fn = lib().sam_step_host
    fixed = [c_void_p(_host_ptr(x, n)) for x, n in ((draft_tokens, "draft_tokens"), (draft_len, "draft_len"),
                                                     (match_len, "match_len"), (source, "source"), (state, "state"),
                                                     (status, "status"))]
    sp, hh = c_void_p(_stream_ptr(stream)), c_void_p(h) if isinstance(h, int) else h

    def call(new_tokens, counts):
        rc = fn(hh, _host_ptr(new_tokens, "new_tokens"), stride, _host_ptr(counts, "counts"), L, *fixed, sp)
        if rc != SAM_OK:
            raise SamError(rc, "sam_step_host")
    return call


def sam_batch_dump(h, slot: int, max_states: int, max_edges: int, stream=None):
    nt, ns, ne = c_int32(), c_int32(), c_int32()
    st = [np.zeros(max(max_states, 1), dtype=np.int32) for _ in range(4)]
    ed = [np.zeros(max(max_edges, 1), dtype=np.int32) for _ in range(3)]
    _check(lib().sam_batch_dump(h, slot, byref(nt), byref(ns), byref(ne), *[a.ctypes.data for a in st], max_states,
                                *[a.ctypes.data for a in ed], max_edges, _stream_ptr(stream)), "sam_batch_dump")
    s, e = min(ns.value, max_states), min(ne.value, max_edges)
    return dict(n_tokens=nt.value, n_states=ns.value, n_edges=ne.value,
                length=st[0][:s], link=st[1][:s], min_endpos=st[2][:s], deg=st[3][:s],
                edge_src=ed[0][:e], edge_tok=ed[1][:e], edge_tgt=ed[2][:e])


def sam_batch_pool_info(h, stream=None):
    tot, free = c_int64(), c_int64()
    _check(lib().sam_batch_pool_info(h, byref(tot), byref(free), _stream_ptr(stream)), "sam_batch_pool_info")
    return tot.value, free.value


def sam_accept_greedy(draft_tokens, draft_len, target_tokens, max_new, new_tokens, counts, accepted=None, stream=None):
    B, L = draft_tokens.shape
    _check(lib().sam_accept_greedy(B, _dev_ptr(draft_tokens, "draft_tokens"), _dev_ptr(draft_len, "draft_len"), L,
                                   _dev_ptr(target_tokens, "target_tokens"), _dev_ptr(max_new, "max_new"),
                                   _dev_ptr(new_tokens, "new_tokens"), new_tokens.shape[1], _dev_ptr(counts, "counts"),
                                   _dev_ptr(accepted, "accepted"), _stream_ptr(stream)), "sam_accept_greedy")


def sam_step_verified(h, target_tokens, prev_draft_tokens, prev_draft_len, max_new, L,
                      draft_tokens, draft_len, match_len, source, state, status, counts_out=None, accepted_out=None,
                      stream=None):
    _check(lib().sam_step_verified(h, _dev_ptr(target_tokens, "target_tokens"), prev_draft_tokens.shape[1],
                                   _dev_ptr(prev_draft_tokens, "prev_draft_tokens"), _dev_ptr(prev_draft_len, "prev_draft_len"),
                                   _dev_ptr(max_new, "max_new"), L,
                                   _dev_ptr(draft_tokens, "draft_tokens"), _dev_ptr(draft_len, "draft_len"),
                                   _dev_ptr(match_len, "match_len"), _dev_ptr(source, "source"),
                                   _dev_ptr(state, "state"), _dev_ptr(status, "status"),
                                   _dev_ptr(counts_out, "counts_out"), _dev_ptr(accepted_out, "accepted_out"),
                                   _stream_ptr(stream)), "sam_step_verified")


def sam_select_auxiliary(draft_tokens, draft_len, source, aux_tokens, aux_len, stream=None):
    B, L = draft_tokens.shape
    _check(lib().sam_select_auxiliary(B, L, _dev_ptr(draft_tokens, "draft_tokens"), _dev_ptr(draft_len, "draft_len"),
                                      _dev_ptr(source, "source"), _dev_ptr(aux_tokens, "aux_tokens"),
                                      _dev_ptr(aux_len, "aux_len"), _stream_ptr(stream)), "sam_select_auxiliary")


def sam_tree_draft(static_h, states, start_tokens, max_size: int, k: int, tree_tokens, tree_parents, tree_probs,
                   tree_size, stream=None):
    import torch
    pp = None
    if tree_probs is not None:
        assert tree_probs.is_cuda and tree_probs.dtype == torch.float32 and tree_probs.is_contiguous()
        pp = tree_probs.data_ptr()
    _check(lib().sam_tree_draft(static_h, states.shape[0], _dev_ptr(states, "states"),
                                _dev_ptr(start_tokens, "start_tokens"), max_size, k,
                                _dev_ptr(tree_tokens, "tree_tokens"), _dev_ptr(tree_parents, "tree_parents"), pp,
                                _dev_ptr(tree_size, "tree_size"), _stream_ptr(stream)), "sam_tree_draft")


def sam_static_freq(h):
    n = sam_static_info(h).n_states
    out = np.empty(n, dtype=np.uint32)
    _check(lib().sam_static_freq(h, out.ctypes.data, n), "sam_static_freq")
    return out


def sam_retrieve_noalloc(static_h, vocab, tokens, counts, L, l_bias, min_match,
                         draft_tokens, draft_len, match_len, source, state, status, stream=None):
    """One-shot retrieval over the library's built-in scratch array; allocates nothing."""
    _check(lib().sam_retrieve_noalloc(static_h, vocab, tokens.shape[0], _dev_ptr(tokens, "tokens"), tokens.shape[1],
                                      _dev_ptr(counts, "counts"), L, l_bias, min_match,
                                      _dev_ptr(draft_tokens, "draft_tokens"), _dev_ptr(draft_len, "draft_len"),
                                      _dev_ptr(match_len, "match_len"), _dev_ptr(source, "source"),
                                      _dev_ptr(state, "state"), _dev_ptr(status, "status"), _stream_ptr(stream)),
           "sam_retrieve_noalloc")


COUNTER_NAMES = ("static_rounds", "static_link_moves", "static_next_moves", "dynamic_rounds", "walk_inserts",
                 "clones", "copied_edges", "redirects", "tokens", "seq_steps")
N_COUNTERS = 12


def sam_counters_available() -> bool:
    return bool(lib().sam_counters_available())


def sam_counters_attach(counters, slots: int = 0):
    """counters: a zeroed torch uint64/int64 device tensor [slots, N_COUNTERS], or None to detach."""
    if counters is None:
        _check(lib().sam_counters_attach(None, 0), "sam_counters_attach")
    else:
        assert counters.is_cuda and counters.is_contiguous() and counters.element_size() == 8
        assert counters.numel() >= slots * N_COUNTERS
        _check(lib().sam_counters_attach(counters.data_ptr(), slots), "sam_counters_attach")


def sam_probe_random_read(buf, granule: int, iters: int = 5, stream=None):
    g, r = c_double(), c_double()
    _check(lib().sam_probe_random_read(buf.data_ptr(), buf.numel() * buf.element_size(), granule, iters,
                                       _stream_ptr(stream), byref(g), byref(r)), "sam_probe_random_read")
    return g.value, r.value


def sam_probe_chase(buf, hops: int, chains: int = 1, stream=None):
    ns = c_double()
    _check(lib().sam_probe_chase(buf.data_ptr(), buf.numel() * buf.element_size(), hops, chains,
                                 _stream_ptr(stream), byref(ns)), "sam_probe_chase")
    return ns.value


# ---------------------------------------------------------------------------------------------
# small owner objects (lifetime + torch memory), still no arithmetic
# ---------------------------------------------------------------------------------------------

def _on_ram_disk(path: str) -> bool:
    """True if `path` lies on a memory-backed filesystem (an image written there would use up RAM)."""
    try:
        real, best, kind = os.path.realpath(path), "", ""
        for line in open("/proc/mounts"):
            f = line.split()
            if len(f) >= 3 and (real == f[1] or real.startswith(f[1].rstrip("/") + "/")) and len(f[1]) >= len(best):
                best, kind = f[1], f[2]
        return kind in ("tmpfs", "ramfs")
    except OSError:
        return False


class StaticSam:
    """A static automaton on a device.  `StaticSam.build(corpus, vocab)` or `StaticSam.load(path)`."""

    def __init__(self, handle, device: int):
        self.handle, self.device = handle, device

    @classmethod
    def build(cls, corpus, vocab: int, device: int = 0, hash_load: float = 0.0, tree_topk: int = 0):
        return cls(sam_build_static(corpus, vocab, device, hash_load, tree_topk), device)

    @classmethod
    def load(cls, path: str, device: int = 0):
        return cls(sam_static_load(path, device), device)

    def save(self, path: str):
        sam_static_save(self.handle, path)

    @classmethod
    def cached(cls, corpus, vocab: int, cache_dir: str, device: int = 0, tree_topk: int = 0):
        """The automaton of `corpus` from a saved image under `cache_dir` when there is one, else built
        and, room on the disk permitting, saved there.  The file name is a digest of the corpus bytes,
        the vocabulary, the top-k setting and the library version, so a stale image is never picked up;
        an image that fails its checksum is rebuilt.  Returns (automaton, "loaded" | "built")."""
        import hashlib
        import shutil
        c = _np32(corpus)
        h = hashlib.blake2b(digest_size=12)
        h.update(memoryview(c).cast("B"))
        h.update(("|%d|%d|%s" % (vocab, tree_topk, lib().sam_version().decode())).encode())
        path = os.path.join(cache_dir, "static-%s.samimg" % h.hexdigest())
        if os.path.exists(path):
            try:
                return cls.load(path, device), "loaded"
            except SamError:
                pass
        st = cls.build(c, vocab, device, 0.0, tree_topk)
        try:
            os.makedirs(cache_dir, exist_ok=True)
            need = int(st.info.device_bytes * 1.1) + (2 << 30)
            if not _on_ram_disk(cache_dir) and shutil.disk_usage(cache_dir).free > need:
                tmp = path + ".tmp%d" % os.getpid()
                st.save(tmp)
                os.replace(tmp, path)
        except (OSError, SamError):
            pass                                        # a cache that cannot be written is not an error
        return st, "built"

    @property
    def info(self) -> StaticInfo:
        return sam_static_info(self.handle)

    def close(self):
        if self.handle:
            sam_static_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class StepOutputs:
    """Device tensors a step writes."""

    def __init__(self, batch: int, L: int, device, steps: int | None = None):
        import torch
        lead = () if steps is None else (steps,)
        mk = lambda *shape: torch.empty(lead + shape, dtype=torch.int32, device=device)
        self.draft_tokens = mk(batch, L)
        self.draft_len = mk(batch)
        self.match_len = mk(batch, 2)
        self.source = mk(batch)
        self.state = mk(batch, 2)
        self.status = mk(batch)

    def tensors(self):
        return (self.draft_tokens, self.draft_len, self.match_len, self.source, self.state, self.status)

    def cpu(self):
        return {k: getattr(self, k).cpu().numpy() for k in
                ("draft_tokens", "draft_len", "match_len", "source", "state", "status")}


class Batch:
    """B sequence slots over an optional static automaton; owns the workspace tensor."""

    def __init__(self, static: StaticSam | None, batch: int, max_seq_len: int, max_draft_len: int = 32,
                 l_bias: int = 0, min_match: int = 1, vocab: int = 0, max_host_stride: int = 0,
                 slab_bytes: int = 0, pool_slabs: int = 0, device: int | None = None, stop_token: int = -1):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("samdraft needs a CUDA device; there is no CPU path")
        self.static = static
        dev = static.device if static is not None else (0 if device is None else device)
        self.device = torch.device("cuda", dev)
        self.opts = BatchOpts(batch, max_seq_len, max_draft_len, l_bias, min_match, vocab,
                              max_host_stride, slab_bytes, pool_slabs, stop_token + 1, 0)
        nbytes = sam_batch_workspace_bytes(self.opts)
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            self.handle = sam_batch_create(static.handle if static is not None else None, self.opts, self.workspace)
        self.batch, self.max_draft_len = batch, max_draft_len

    def step(self, new_tokens, counts, L: int, out: StepOutputs | None = None) -> StepOutputs:
        out = out or StepOutputs(self.batch, L, self.device)
        with __import__("torch").cuda.device(self.device):
            sam_step(self.handle, new_tokens, new_tokens.shape[-1], counts, L, *out.tensors())
        return out

    def run_steps(self, new_tokens, counts, L: int, per_step: bool = True, out: StepOutputs | None = None):
        n_steps = new_tokens.shape[0]
        out = out or StepOutputs(self.batch, L, self.device, n_steps if per_step else None)
        with __import__("torch").cuda.device(self.device):
            sam_run_steps(self.handle, new_tokens, new_tokens.shape[-1], counts, n_steps, L, per_step, *out.tensors())
        return out

    def reset(self, slots=None):
        sam_batch_reset(self.handle, slots)

    def dump(self, slot: int, max_states: int, max_edges: int):
        return sam_batch_dump(self.handle, slot, max_states, max_edges)

    def pool_info(self):
        return sam_batch_pool_info(self.handle)

    def launches_per_step(self) -> int:
        n = lib().sam_batch_launches_per_step(self.handle)
        _check(n if n < 0 else SAM_OK, "sam_batch_launches_per_step")
        return n

    def close(self):
        if getattr(self, "handle", None):
            sam_batch_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
