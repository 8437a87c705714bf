#!/usr/bin/env python
"""Benchmark of the batched suffix-automaton draft-retrieval step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload c5]

A "step" is one `sam_step` over the whole batch: every slot feeds its accepted tokens of that
decoding step through the static automaton (Transfer) and its own dynamic automaton
(Transfer + Expand), the source is chosen and the draft is read.  The prompt prefill and W
warm-up steps run untimed; then exactly K consecutive decoding steps of the schedule are timed
with CUDA events.  The K-step region is repeated from an identical state (reset, prefill, warm-up,
L2 flush) until a few seconds have passed so that clock samples exist; the reported value is the
median repeat.  One JSON line is printed by rank 0.

The headline workload is the largest of the five recipes (c5: 4096 sequences over a 200 M-token
corpus).  At one GPU the line also carries `all_workloads`: the same measurement, shorter, for the
other four recipes.  The CPU oracle is timed beside every workload on the same decoding steps; its
automata are built in child processes while the GPU part runs (the builds are single-threaded and
take minutes at 100-200 M tokens), and each child's timed run starts only when the GPU part is over.

Under torchrun each rank owns a contiguous shard of a batch that is N times larger (weak scaling,
the static automaton replicated, no collective on the data path); the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as W  # noqa: E402

METRIC = "sam_sequence_steps_per_sec"
UNIT = "sequence-steps/s"
HEADLINE = "c5"
ORDER = ["tiny", "c2", "c3", "c4", "c5"]

# Algorithmic bytes per sequence-step averaged over a recipe's whole generation phase (from the CPU
# oracle's operation counters, `python -m oracle.count_ops <workload>`).  Used only when the oracle leg
# is switched off; otherwise the bytes come from the oracle's counters over exactly the timed steps.
ALGO_BYTES_WHOLE_PHASE = {"tiny": 750.3, "c2": 857.7, "c3": 935.1, "c4": 1374.8, "c5": 1024.1}

# DRAM traffic of one step launch (dram__bytes_read.sum + dram__bytes_write.sum, one-pass ncu capture that
# leaves the caches as the loop leaves them), per capture: bytes per launch, sequence-steps per launch of
# the captured case, and the digest of the kernel sources the capture was taken on.  A capture whose digest
# is not that of the sources as they stand is not reported.
NCU_TRAFFIC = {
    # workload: (bytes per launch, slots per launch in the capture, source digest, note)
    "c5": (4978176, 4096, "536687ab2bd76708",
           "median of 60 launches, one-pass capture with the caches left as the loop leaves them, taken on the recipe over a "
           "10 M-token corpus (3.80 MB read + 1.17 MB written per launch of 4096 slots) and carried over per slot: the "
           "full-size corpus changes which lines are read, not how many"),
}
KERNEL_SOURCES = ("paper_2411_10666_b200/csrc/step.cu", "paper_2411_10666_b200/csrc/layout.h")


def kernel_digest() -> str:
    h = hashlib.sha256()
    for rel in KERNEL_SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=512)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=HEADLINE, choices=sorted(W.SPECS))
    ap.add_argument("--min-seconds", type=float, default=2.5, help="keep repeating the timed region this long")
    ap.add_argument("--max-repeats", type=int, default=300)
    ap.add_argument("--batch", type=int, default=0,
                    help="run the workload's recipe with this many sequences per GPU instead of its own batch (a scaling probe, not a headline)")
    ap.add_argument("--corpus-tokens", type=int, default=0,
                    help="run the workload's recipe over a corpus of this many tokens (a reduced case for profiler captures, not a headline)")
    ap.add_argument("--prompt-len", type=int, default=0, help="run the workload's recipe with prompts of this many tokens (a reduced case)")
    ap.add_argument("--gen-len", type=int, default=0, help="run the workload's recipe with this many generated tokens (a reduced case)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-probes", action="store_true")
    ap.add_argument("--no-all-workloads", action="store_true", help="measure the named workload only")
    ap.add_argument("--cpu-wait-seconds", type=float, default=900.0,
                    help="how long to wait for an oracle automaton that is still being built")
    ap.add_argument("--cache-dir", default=os.environ.get("SAMDRAFT_CACHE_DIR", ""),
                    help="keep built static automata here between runs (sam_static_save / sam_static_load; the c5 image is "
                         "18 GB); default: the SAMDRAFT_CACHE_DIR environment variable, else no caching")
    ap.add_argument("--tree-draft", action="store_true",
                    help="also time sam_tree_draft (builds the static automaton with top-k successor data)")
    ap.add_argument("--closed-loop", action="store_true",
                    help="also run draft -> verify -> accept -> update on the device with the true continuation as target")
    return ap.parse_args(argv)


def dist_env():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def variant(name: str, batch: int = 0, corpus_tokens: int = 0, prompt_len: int = 0, gen_len: int = 0) -> W.Spec:
    spec = W.SPECS[name]
    return W.scaled(spec, batch=batch or None, corpus_len=corpus_tokens or None, prompt_len=prompt_len or None,
                    gen_len=gen_len or None)


def named_variant(args, name: str) -> W.Spec:
    """The recipe `name` as the command line asks for it: size options apply to the named workload only."""
    if name != args.workload:
        return variant(name)
    return variant(name, args.batch, args.corpus_tokens, args.prompt_len, args.gen_len)


def named_label(args, name: str) -> str:
    if name != args.workload:
        return name
    return workload_label(name, args.batch, args.corpus_tokens, args.prompt_len, args.gen_len)


def config_dict(base: W.Spec, label: str, world: int) -> dict:
    """What names the workload; the same for the GPU arm and the reference arm."""
    return {"workload": label, "batch_per_gpu": base.batch, "global_batch": base.batch * world,
            "prompt_len": base.prompt_len, "gen_len": base.gen_len, "draft_len": base.draft_len,
            "accept_max": base.accept_max, "corpus_tokens": base.corpus_len, "vocab": base.vocab,
            "parallelism": "batch-sharded x%d, static automaton replicated" % world,
            "l2": "GPU arm: L2 flushed (288 MB write) before each timed region and the static store is larger than "
                  "the 126 MB L2 except for the smallest recipes; per-sequence automata stay cache-warm between "
                  "consecutive steps.  CPU arm: caches as the preceding steps leave them"}


def workload_label(name: str, batch: int, corpus_tokens: int, prompt_len: int = 0, gen_len: int = 0) -> str:
    extra = []
    if batch > 0:
        extra.append("%d sequences" % batch)
    if corpus_tokens > 0:
        extra.append("%d corpus tokens" % corpus_tokens)
    if prompt_len > 0:
        extra.append("prompts of %d tokens" % prompt_len)
    if gen_len > 0:
        extra.append("%d generated tokens" % gen_len)
    return name + (" (recipe run with %s)" % ", ".join(extra) if extra else "")


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples of one GPU while the timed regions run."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.proc = None
        try:
            fd, self.path = tempfile.mkstemp(prefix="samclk_", suffix=".csv")
            self.f = os.fdopen(fd, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 8:
                    continue
                try:
                    sm.append(float(f[0]))
                    mx.append(float(f[1]))
                except ValueError:
                    continue
                for n, v in zip(names, f[4:8]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            os.unlink(self.path)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def shard_workload(spec: W.Spec, rank: int, world: int, corpus=None):
    """Weak scaling: the global batch is `world` times the recipe's batch; this rank's shard."""
    big = W.scaled(spec, batch=spec.batch * world)
    if corpus is None:
        corpus = W.make_corpus(big)
    seqs, counts, new_tokens = W.make_sequences(big, corpus, rank, world)
    return big, corpus, seqs, counts, new_tokens


def reduce_max_sum(local_ms: float, local_units: int, world: int):
    """(max over ranks of the time, sum over ranks of the units) — the only cross-rank exchange."""
    if world == 1:
        return local_ms, local_units
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([local_ms], dtype=torch.float64, device=dev)
    u = torch.tensor([local_units], dtype=torch.int64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), int(u.item())


# ---------------------------------------------------------------------------------------------
# the CPU oracle, timed in a child process
# ---------------------------------------------------------------------------------------------

def algorithmic_bytes(c: dict, L: int) -> dict:
    """Bytes the method itself must touch for the steps whose operation counts are `c`: a state is a
    32-byte record; 32 B per Transfer move; per accepted token a new state (32 B), its two link fields
    (8 B) and the text append (4 B); per walk-insert 32 B read + 8 B written; per clone 32 B read + 32 B
    written; per redirect 32 B read + 4 B written; per step the two matched states' records, the drafted
    tokens, the output row (4 L + 28 B) and the input row (4 m + 4 B)."""
    steps, toks = max(c["seq_steps"], 1), c["tokens"]
    static_b = 32 * (c["static_link_moves"] + c["static_next_moves"])
    dyn_b = toks * 44 + c["walk_inserts"] * 40 + c["clones"] * 64 + c["redirects"] * 36
    step_b = c["seq_steps"] * (64 + 4 * L + 28 + 4) + 4 * toks + 4 * c["draft_tokens"]
    return {"static": static_b / steps, "dynamic": dyn_b / steps, "step_io": step_b / steps,
            "total": (static_b + dyn_b + step_b) / steps}


def dependent_accesses(c: dict) -> dict:
    """Accesses per sequence-step that Algorithms 1 and 3 make one after the other (each needs the
    result of the one before): on the static chain every Transfer move, then the matched state's record
    and the draft; on the dynamic chain every link or next move of Transfer / Expand's walk, every clone
    (the record of q) and redirect, then record and draft."""
    steps = max(c["seq_steps"], 1)
    st = (c["static_link_moves"] + c["static_next_moves"]) / steps + 2
    dy = (c["dynamic_link_moves"] + c["dynamic_next_moves"] + c["clones"] + c["redirects"]) / steps + 2
    return {"static_chain": st, "dynamic_chain": dy}


def oracle_leg(base: W.Spec, Wm: int, K: int, threads: int, single_thread_budget_s: float = 8.0, wait_for_go=None, ready=None):
    """Build the oracle's automata for `base`, run prefill and warm-up steps untimed, then time the K
    decoding steps [Wm, Wm + K) on all `threads` cores (OpenMP over sequences, static automaton shared),
    and a bounded share of them on one thread."""
    import oracle
    few = max(1, min(4, threads // 4)) if wait_for_go is not None else threads   # untimed phases keep out of the GPU part's way
    t0 = time.perf_counter()
    corpus = W.make_corpus(base)
    seqs, counts, new_tokens = W.make_sequences(base, corpus)
    t1 = time.perf_counter()
    S = oracle.Sam(corpus)
    build_s = time.perf_counter() - t1
    B, L = seqs.shape[0], base.draft_len
    K = min(K, counts.shape[0] - Wm)
    prompts = np.ascontiguousarray(seqs[:, :base.prompt_len])
    pcount = np.full(B, base.prompt_len, dtype=np.int32)

    def fresh():
        ob = oracle.Batch(S, corpus, B, base.vocab, base.prompt_len + base.gen_len)
        ob.step(prompts, pcount, L, few)
        if Wm > 0:
            ob.run(new_tokens[:Wm], counts[:Wm], L, few)
        return ob

    ob = fresh()
    if ready is not None:
        ready({"build_s": build_s, "inputs_s": t1 - t0})
    if wait_for_go is not None:
        wait_for_go()
    few = threads                                        # the GPU part is over: use every core from here on
    ob.step(np.zeros((B, 1), dtype=np.int32), np.zeros(B, dtype=np.int32), L, threads)   # an empty step: the thread pool exists before the clock starts
    c0 = ob.counters()
    t2 = time.perf_counter()
    ob.run(new_tokens[Wm:Wm + K], counts[Wm:Wm + K], L, threads)
    dt = time.perf_counter() - t2
    c1 = ob.counters()
    ob.close()
    d = {k: c1[k] - c0[k] for k in c1}
    units = d["seq_steps"]
    res = {"value": units / dt, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": dt, "steps": K,
           "sequence_steps": units, "draft_tokens_per_sec": d["draft_tokens"] / dt,
           "oracle_build_seconds": build_s, "counters": d,
           "sample": "the same %d decoding steps x %d sequences (%d sequence-steps) as the GPU arm, OpenMP over "
                     "sequences on %d threads; static build, prefill and warm-up steps untimed" % (K, B, units, threads)}
    # one thread, on as many of the same steps as fit the budget
    per_step_s = dt * threads / max(K, 1)
    K1 = int(max(1, min(K, single_thread_budget_s / max(per_step_s, 1e-9))))
    ob = fresh()
    c0 = ob.counters()
    t3 = time.perf_counter()
    ob.run(new_tokens[Wm:Wm + K1], counts[Wm:Wm + K1], L, 1)
    dt1 = time.perf_counter() - t3
    u1 = ob.counters()["seq_steps"] - c0["seq_steps"]
    ob.close()
    res["single_thread_value"] = u1 / dt1
    res["single_thread_sample"] = "the first %d of those steps" % K1
    return res


def _oracle_child(conn, base, Wm, K, threads):
    try:
        res = oracle_leg(base, Wm, K, threads, ready=lambda info: conn.send(("ready", info)),
                         wait_for_go=lambda: conn.recv())
        conn.send(("done", res))
    except BaseException as ex:                          # the parent reports why there is no baseline
        try:
            conn.send(("error", "%s: %s" % (type(ex).__name__, ex)))
        except Exception:
            pass
    finally:
        conn.close()


class OracleChildren:
    """One child process per workload, started (spawn) before the first CUDA call."""

    def __init__(self, names, args, Wm):
        import multiprocessing as mp
        self.ctx = mp.get_context("spawn")
        self.kids = {}
        self.threads = os.cpu_count() or 1
        for name in names:
            base = named_variant(args, name)
            need_gb = estimate_oracle_gb(base)
            avail = mem_available_gb()
            if avail is not None and avail < need_gb + 24:
                self.kids[name] = ("unavailable", "host has %.0f GB available, the oracle's automaton needs about %.0f GB"
                                   % (avail, need_gb))
                continue
            parent, child = self.ctx.Pipe()
            p = self.ctx.Process(target=_oracle_child, args=(child, base, Wm, args.steps, self.threads),
                                 daemon=True)
            p.start()
            child.close()
            self.kids[name] = (p, parent)

    def wait_ready(self, name, wait_s):
        """Wait until `name`'s child has built its automata and run its untimed steps.  The timed runs start
        only when every child is at this point: a build still going on another core would stretch the
        barriers of a timed run on all cores."""
        kid = self.kids.get(name)
        if kid is None or kid[0] == "unavailable":
            return
        p, conn = kid
        try:
            if not conn.poll(wait_s):
                p.terminate()
                self.kids[name] = ("unavailable", "the oracle's automaton was not built within %d s" % wait_s)
                return
            tag, info = conn.recv()
            if tag != "ready":
                self.kids[name] = ("unavailable", str(info))
        except (EOFError, OSError) as ex:
            self.kids[name] = ("unavailable", "oracle process ended early (%s)" % ex)

    def collect(self, name):
        """Let `name`'s child (which is ready) run its timed part now — nothing else is running — and return its result."""
        kid = self.kids.get(name)
        if kid is None:
            return {"unavailable": "not requested"}
        if kid[0] == "unavailable":
            return {"unavailable": kid[1]}
        p, conn = kid
        try:
            conn.send("go")
            if not conn.poll(600):
                p.terminate()
                return {"unavailable": "the oracle's timed run did not end within 600 s"}
            tag, res = conn.recv()
            p.join(timeout=30)
            return res if tag == "done" else {"unavailable": str(res)}
        except (EOFError, OSError) as ex:
            return {"unavailable": "oracle process ended early (%s)" % ex}

    def close(self):
        for kid in self.kids.values():
            if kid[0] != "unavailable" and kid[0].is_alive():
                kid[0].terminate()


def mem_available_gb():
    try:
        for line in open("/proc/meminfo"):
            if line.startswith("MemAvailable:"):
                return int(line.split()[1]) / 1e6
    except OSError:
        pass
    return None


def estimate_oracle_gb(base: W.Spec) -> float:
    """Host memory of the oracle's static automaton (about 1.3 states and 2.1 transitions per corpus
    token, one small heap block per state) plus the corpus and the sequences' own automata."""
    n = base.corpus_len
    return (n * 1.3 * (29 + 32) + n * 4 * 2 + base.batch * (base.prompt_len + base.gen_len) * 200) / 1e9


# ---------------------------------------------------------------------------------------------
# the GPU arm
# ---------------------------------------------------------------------------------------------

def tree_draft_timing(P, st, batch, prepare, out, flush):
    """Time sam_tree_draft (best-first tree over the top-k successors, Algorithm 5) from the static states
    the batch is in after the warm-up steps; L2 flushed before every call."""
    import torch
    prepare()
    torch.cuda.synchronize()
    B = batch.batch
    dev = batch.device
    states = out.state[:, 0].contiguous()
    starts = torch.zeros(B, dtype=torch.int32, device=dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    res = {"slots_with_a_static_match": int((states > 0).sum().item())}
    for max_size, k in ((16, 2), (40, 4), (70, 4)):
        toks = torch.empty((B, max_size), dtype=torch.int32, device=dev)
        par = torch.empty_like(toks)
        sz = torch.empty(B, dtype=torch.int32, device=dev)
        ts = []
        for _ in range(15):
            flush.zero_()
            torch.cuda.synchronize()
            e0.record()
            P.binding.sam_tree_draft(st.handle, states, starts, max_size, k, toks, par, None, sz)
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3)
        res["max_size_%d_k_%d" % (max_size, k)] = {"us_per_call": statistics.median(ts),
                                                   "mean_tree_size": float(sz.float().mean().item())}
    return res


def closed_loop(P, batch, seqs, spec, L):
    """The whole decoding loop on the device: sam_step drafts, the sequences' own continuation plays
    the target model, sam_accept_greedy verifies and produces the next step's input.  Reports the
    mean number of accepted tokens per step (the paper's #MAT) and the time per loop iteration."""
    import torch
    B, total = seqs.shape
    dev = batch.device
    sd = P.binding
    seq_dev = torch.from_numpy(seqs).to(dev).long()
    stride = L + 1
    nt = torch.empty((B, stride), dtype=torch.int32, device=dev)
    cnt = torch.empty(B, dtype=torch.int32, device=dev)
    acc = torch.empty_like(cnt)
    ar = torch.arange(L + 1, device=dev)[None, :]
    batch.reset()
    out = batch.step(seq_dev[:, :spec.prompt_len].int().contiguous(),
                     torch.full((B,), spec.prompt_len, dtype=torch.int32, device=dev), L)
    pos = torch.full((B,), spec.prompt_len, dtype=torch.int64, device=dev)
    steps = seq_steps = accepted_draft = 0
    src_hist = torch.zeros(4, dtype=torch.int64, device=dev)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    while True:
        target = torch.gather(seq_dev, 1, torch.clamp(pos[:, None] + ar, max=total - 1)).int().contiguous()
        cap = (total - pos).int().contiguous()
        sd.sam_accept_greedy(out.draft_tokens, out.draft_len, target, cap, nt, cnt, acc)
        active = cnt > 0
        src_hist += torch.bincount(out.source[active].long(), minlength=4)
        seq_steps += int(active.sum().item())               # one host read per iteration, to know when to stop
        accepted_draft += int(acc.sum().item())
        if not bool(active.any().item()):
            break
        batch.step(nt, cnt, L, out)
        pos += cnt.long()
        steps += 1
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    gen = int((pos - spec.prompt_len).sum().item())
    h = src_hist.tolist()
    # The same loop once more with verification folded into the step (sam_step_verified) and nothing but that
    # call inside the timed region: the loop is deterministic, so the target rows and caps of every iteration are
    # recorded in a first pass and replayed from device memory, one launch per iteration, no host read.
    n_it = min(steps, 256)
    targets = torch.empty((n_it, B, L + 1), dtype=torch.int32, device=dev)
    caps = torch.empty((n_it, B), dtype=torch.int32, device=dev)
    outs = [P.StepOutputs(B, L, dev), P.StepOutputs(B, L, dev)]

    def fused_pass(record):
        batch.reset()
        batch.step(seq_dev[:, :spec.prompt_len].int().contiguous(),
                   torch.full((B,), spec.prompt_len, dtype=torch.int32, device=dev), L, outs[0])
        p2 = torch.full((B,), spec.prompt_len, dtype=torch.int64, device=dev)
        cur = 0
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for it in range(n_it):
            prev, new = outs[cur], outs[1 - cur]
            if record:
                targets[it] = torch.gather(seq_dev, 1, torch.clamp(p2[:, None] + ar, max=total - 1)).int()
                caps[it] = (total - p2).int()
            sd.sam_step_verified(batch.handle, targets[it], prev.draft_tokens, prev.draft_len, caps[it], L,
                                 *new.tensors(), counts_out=cnt, accepted_out=acc)
            if record:
                p2 += cnt.long()
            cur = 1 - cur
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / max(n_it, 1)

    fused_pass(True)
    fused_us = statistics.median(fused_pass(False) for _ in range(5))
    return {"decoding_steps": steps, "sequence_steps": seq_steps, "generated_tokens": gen,
            "us_per_fused_verify_and_step": fused_us,
            "fused_note": "sam_step_verified alone, %d consecutive iterations of the closed loop replayed from recorded target rows, "
                          "CUDA events, no host read inside" % n_it,
            "mean_accepted_tokens_per_step": gen / max(seq_steps, 1),
            "mean_confirmed_draft_tokens_per_step": accepted_draft / max(seq_steps, 1),
            "draft_source_share": {"none": h[0] / max(seq_steps, 1), "static": h[1] / max(seq_steps, 1),
                                   "dynamic": h[2] / max(seq_steps, 1)},
            "us_per_loop_iteration": dt * 1e6 / max(steps, 1),
            "note": "target = the sequence's own continuation (synthetic); torch gathers the target rows"}


def peak_stream():
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        return float(peaks["hbm_gbs"]), "measured stream copy"
    except Exception:
        return 6650.0, "fallback stream copy"


def measure_gpu(P, args, name, rank, world, local_rank, full):
    """One workload on this rank's GPU.  `full`: the headline treatment (graph replay, probes, clock samples)."""
    import torch
    sd = P.binding
    base = named_variant(args, name)
    label = named_label(args, name)
    t0 = time.perf_counter()
    spec, corpus, seqs, counts, new_tokens = shard_workload(base, rank, world)
    inputs_s = time.perf_counter() - t0
    B, L = seqs.shape[0], spec.draft_len
    msl = spec.prompt_len + spec.gen_len
    Wm = args.warmup
    K = min(args.steps, counts.shape[0] - Wm)
    assert K >= 1 and Wm >= 3, "need at least 3 warm-up steps and 1 timed step"

    t0 = time.perf_counter()
    topk = 4 if (args.tree_draft and full) else 0
    if args.cache_dir and rank == 0:
        st, static_source = P.StaticSam.cached(corpus, spec.vocab, args.cache_dir, device=local_rank, tree_topk=topk)
    else:
        st, static_source = P.StaticSam.build(corpus, spec.vocab, device=local_rank, tree_topk=topk), "built"
    build_s = time.perf_counter() - t0
    info = st.info
    batch = P.Batch(st, B, msl, max_draft_len=L, max_host_stride=spec.accept_max)
    dev = batch.device
    prompts = torch.from_numpy(np.ascontiguousarray(seqs[:, :spec.prompt_len])).to(dev)
    pcount = torch.full((B,), spec.prompt_len, dtype=torch.int32, device=dev)
    nt_dev = torch.from_numpy(new_tokens[:Wm + K]).to(dev)
    ct_dev = torch.from_numpy(counts[:Wm + K]).to(dev)
    out = P.StepOutputs(B, L, dev)
    flush = torch.empty(288 << 20, dtype=torch.uint8, device=dev)      # larger than the 126 MB L2

    def prepare():
        batch.reset()
        batch.step(prompts, pcount, L, out)
        batch.run_steps(nt_dev[:Wm], ct_dev[:Wm], L, per_step=False, out=out)
        flush.zero_()

    units = int((counts[Wm:Wm + K] > 0).sum())
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    # prefill throughput, reported separately (not part of the headline)
    batch.reset()
    torch.cuda.synchronize()
    e0.record()
    batch.step(prompts, pcount, L, out)
    e1.record()
    torch.cuda.synchronize()
    prefill_ms = e0.elapsed_time(e1)

    sampler = None
    if full and rank == 0:
        gpu_id = str(torch.cuda.current_device())
        try:                                              # the physical GPU, whatever CUDA_VISIBLE_DEVICES says
            gpu_id = "GPU-" + str(torch.cuda.get_device_properties(torch.cuda.current_device()).uuid)
        except Exception:
            pass
        sampler = ClockSampler(gpu_id)
    min_seconds = args.min_seconds if full else min(args.min_seconds, 1.0)
    times = []
    t_start = time.perf_counter()
    while True:
        prepare()
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
        e0.record()
        batch.run_steps(nt_dev[Wm:Wm + K], ct_dev[Wm:Wm + K], L, per_step=False, out=out)
        e1.record()
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
        times.append(e0.elapsed_time(e1))
        elapsed = time.perf_counter() - t_start
        stop = len(times) >= 3 and (elapsed >= min_seconds or len(times) >= args.max_repeats)
        if world > 1:                                                   # all ranks stop together
            flag = torch.tensor([1 if stop else 0], device=dev)
            torch.distributed.all_reduce(flag, op=torch.distributed.ReduceOp.MAX)
            stop = bool(flag.item())
        if stop:
            break
    status_ok = bool((out.status == 0).all().item())

    # the same K launches captured once in a CUDA graph and replayed (reported beside the headline,
    # which stays the plain stream launches)
    graph_ms = None
    if world == 1 and full:
        try:
            side = torch.cuda.Stream()
            prepare()
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(graph, stream=side):
                    batch.run_steps(nt_dev[Wm:Wm + K], ct_dev[Wm:Wm + K], L, per_step=False, out=out)
            gt = []
            for _ in range(7):
                prepare()
                torch.cuda.synchronize()
                e0.record()
                graph.replay()
                e1.record()
                torch.cuda.synchronize()
                gt.append(e0.elapsed_time(e1))
            graph_ms = statistics.median(gt)
            del graph
        except Exception:                                         # capture unsupported: no figure
            graph_ms = None

    # end to end through the host-array call: pinned inputs, H2D + step + D2H + sync every step
    nt_pin = torch.from_numpy(new_tokens[:Wm + K]).pin_memory()
    ct_pin = torch.from_numpy(counts[:Wm + K]).pin_memory()
    mk = lambda *s: torch.empty(s, dtype=torch.int32).pin_memory()
    ho = [mk(B, L), mk(B), mk(B, 2), mk(B), mk(B, 2), mk(B)]
    ho_ptr = [t.data_ptr() for t in ho]                     # addresses are passed as plain ints
    nt_base, nt_step = nt_pin.data_ptr(), B * spec.accept_max * 4
    ct_base, ct_step = ct_pin.data_ptr(), B * 4
    host_step = sd.sam_step_host_prepared(batch.handle, spec.accept_max, L, *ho_ptr)   # sam_step_host, arguments bound once
    e2e_times = []
    for _ in range(3):
        prepare()
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
        t1 = time.perf_counter()
        for s in range(Wm, Wm + K):                     # step s reads its own rows of the pinned arrays
            host_step(nt_base + s * nt_step, ct_base + s * ct_step)
        torch.cuda.synchronize()
        e2e_times.append((time.perf_counter() - t1) * 1e3)
    clocks = sampler.stop() if sampler else None

    # draft tokens per second: count drafted tokens of every timed step once (untimed pass)
    prepare()
    per = batch.run_steps(nt_dev[Wm:Wm + K], ct_dev[Wm:Wm + K], L, per_step=True)
    active = ct_dev[Wm:Wm + K] > 0
    draft_tokens = int((per.draft_len * active).sum().item())
    accepted_tokens = int(counts[Wm:Wm + K].sum())
    torch.cuda.synchronize()
    del per

    ms_local = statistics.median(times)
    ms, units_all = reduce_max_sum(ms_local, units, world)
    e2e_ms, _ = reduce_max_sum(statistics.median(e2e_times), units, world)
    _, drafts_all = reduce_max_sum(0.0, draft_tokens, world)

    launch_us = ms_local * 1e3 / K
    res = {
        "label": label, "base": base, "K": K, "Wm": Wm, "B": B, "L": L, "world": world,
        "value": units_all / (ms * 1e-3), "ms_per_step": ms / K, "launch_us": launch_us,
        "units_local": units, "units_all": units_all,
        "draft_tokens_per_sec": drafts_all / (ms * 1e-3),
        "accepted_tokens_per_sec": accepted_tokens * world / (ms * 1e-3),
        "best_ms_per_step": min(times) / K, "repeats": len(times),
        "prefill_tokens_per_sec": B * spec.prompt_len / (prefill_ms * 1e-3),
        "static": {"states": int(info.n_states), "transitions": int(info.n_transitions), "device_bytes": int(info.device_bytes),
                   "seconds": build_s, "source": static_source, "inputs_seconds": inputs_s},
        "status_all_ok": status_ok,
        "e2e": {"value": units_all / (e2e_ms * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": B * spec.accept_max * 4 + B * 4, "d2h_bytes_per_step": B * (L + 7) * 4,
                "ms_per_step": e2e_ms / K, "api": "sam_step_host"},
        "gpu_launches": K * batch.launches_per_step(), "launches_per_step": batch.launches_per_step(),
        "graph_replay": None if graph_ms is None else {"ms_per_step": graph_ms / K, "value": units / (graph_ms * 1e-3),
                                                       "note": "the K sam_step launches captured in one CUDA graph"},
        "clocks": clocks,
    }

    if full and rank == 0 and not args.no_probes:
        # the random-access denominators, measured now on a buffer the size of the static store
        fp = min(max(int(info.device_bytes), 256 << 20), 8 << 30)
        buf = torch.empty(fp, dtype=torch.uint8, device=dev)
        rnd = {}
        for g in (32, 64, 128):
            gbps, mreq = sd.sam_probe_random_read(buf, g, iters=3)
            rnd[str(g)] = {"GB/s": round(gbps, 1), "Mreq/s": round(mreq, 1)}
        chains = min(2 * B, 65536)
        ns1 = sd.sam_probe_chase(buf, 20000, chains=1)
        nsc = sd.sam_probe_chase(buf, 20000, chains=chains)
        del buf
        res["probes"] = {"random_read": rnd, "footprint_bytes": fp,
                         "dependent_load_ns": {"1_chain": round(ns1, 1), "%d_chains" % chains: round(nsc, 1)},
                         "chains": chains}
    if full and args.tree_draft:
        res["tree_draft"] = tree_draft_timing(P, st, batch, prepare, out, flush)
    if full and args.closed_loop:
        res["closed_loop"] = closed_loop(P, batch, seqs, spec, L)

    batch.close()
    st.close()
    del batch, st, flush, nt_dev, ct_dev, prompts, out, nt_pin, ct_pin, ho
    torch.cuda.empty_cache()
    return res


def device_counters(args, name):
    """Operation counts of the timed steps from the library built with the counters (a child process:
    the package loads one build of the library per process).  None if that fails."""
    cmd = [sys.executable, os.path.join(ROOT, "bench_counters.py"), "--workload", name, "--warmup", str(args.warmup),
           "--steps", str(args.steps)]
    if name == args.workload:
        for flag, v in (("--batch", args.batch), ("--corpus-tokens", args.corpus_tokens), ("--prompt-len", args.prompt_len),
                        ("--gen-len", args.gen_len)):
            if v:
                cmd += [flag, str(v)]
    try:
        out = subprocess.run(cmd, capture_output=True, text=True, timeout=900)
        lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
        return json.loads(lines[-1]) if out.returncode == 0 and lines else None
    except Exception:
        return None


def roofline_block(res, cpu, probes, dev_counters=None):
    """The roofline object of one workload: algorithmic bytes per launch over the launch time against
    the stream-copy peak, the random-read rate and the dependent-access bound beside it."""
    name = res["base"].name
    L = res["L"]
    counters = cpu.get("counters") if cpu else None
    if counters and res["world"] == 1:
        ab = algorithmic_bytes(counters, L)
        algo_b, algo_src = ab["total"], "CPU oracle's operation counters over exactly the timed steps"
    else:
        ab = None
        algo_b, algo_src = ALGO_BYTES_WHOLE_PHASE[name], "CPU oracle's operation counters averaged over the recipe's whole generation phase"
    per_launch = res["units_local"] / res["K"]
    achieved = algo_b * per_launch / (res["launch_us"] * 1e-6) / 1e9
    peak, peak_src = peak_stream()
    digest = kernel_digest()
    cap = NCU_TRAFFIC.get(res["label"])
    traffic, traffic_src = None, "no ncu capture of this workload with the kernel sources as they stand (digest %s)" % digest
    if cap is not None:
        if cap[2] == digest:
            traffic = cap[0] * (per_launch / cap[1]) if cap[1] else cap[0]
            traffic_src = cap[3]
        else:
            traffic_src = "ncu capture is of kernel sources %s, they are now %s: not reported" % (cap[2], digest)
    r = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
         "traffic": traffic, "traffic_source": traffic_src, "peak_source": peak_src,
         "kernel": "sam_step_split_kernel" if res["B"] >= 8192 else "sam_step_kernel", "launch_us": res["launch_us"],
         "algorithmic_bytes_per_sequence_step": algo_b, "algorithmic_bytes_source": algo_src,
         "sequence_steps_per_launch": per_launch}
    if ab:
        r["algorithmic_bytes_split"] = {k: round(v, 1) for k, v in ab.items()}
    if probes:
        r["random_read"] = probes["random_read"]
        r["frac_of_random_32B"] = achieved / probes["random_read"]["32"]["GB/s"]
        r["dependent_load_ns"] = probes["dependent_load_ns"]
        if counters:
            # the dependent-access bound: a sequence's two chains run side by side, each makes its
            # accesses one after the other, so a sequence-step takes at least (accesses of the longer
            # chain) x (latency of a dependent load at this concurrency)
            d = dependent_accesses(counters)
            t_dep = probes["dependent_load_ns"]["%d_chains" % probes["chains"]] * 1e-9
            dmax = max(d.values())
            bound = res["B"] / (dmax * t_dep)
            r["concurrency_bound"] = {"value": bound, "unit": UNIT,
                                      "formula": "B / (d x t_dep): B sequences in flight, d dependent accesses of the longer chain per sequence-step, t_dep at 2B chains",
                                      "dependent_accesses_per_sequence_step": {k: round(v, 2) for k, v in d.items()},
                                      "note": "d counts the accesses Algorithms 1 and 3 make one after the other; the kernel reads guessed states side by side where it can, so it may exceed this figure"}
            r["frac_of_concurrency_bound"] = (res["units_local"] / (res["launch_us"] * 1e-6 * res["K"])) / bound
        if dev_counters:
            # the same bound with the rounds of dependent reads the kernels themselves made (counters build):
            # what the read-ahead, the runs and the prefix states leave of the algorithms' chains
            ps = dev_counters["per_sequence_step"]
            t_dep = probes["dependent_load_ns"]["%d_chains" % probes["chains"]] * 1e-9
            dk = max(ps["static_rounds"], ps["dynamic_rounds"])
            kb = res["B"] / (dk * t_dep)
            r["latency_bound"] = {"value": kb, "unit": UNIT,
                                  "formula": "B / (d x t_dep), d = rounds of dependent reads of the longer chain per sequence-step, counted by the kernels (library built with -DSAM_COUNTERS)",
                                  "rounds_per_sequence_step": {"static_chain": round(ps["static_rounds"], 2), "dynamic_chain": round(ps["dynamic_rounds"], 2)},
                                  "t_dep_ns": probes["dependent_load_ns"]["%d_chains" % probes["chains"]]}
            r["frac_of_latency_bound"] = (res["units_local"] / (res["launch_us"] * 1e-6 * res["K"])) / kb
    return r


def main_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return 0
    base = named_variant(args, args.workload)
    label = named_label(args, args.workload)
    threads = os.cpu_count() or 1
    res = oracle_leg(base, args.warmup, args.steps, threads)
    K = res["steps"]
    value = res["value"]
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": K, "warmup": args.warmup, "ms_per_step": res["seconds"] * 1e3 / K, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": config_dict(base, label, world),
        "draft_tokens_per_sec": res["draft_tokens_per_sec"],
        "cpu_baseline": {k: res[k] for k in ("value", "unit", "cores", "kind", "sample", "single_thread_value",
                                             "single_thread_sample", "oracle_build_seconds")},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def main_ours(args):
    rank, world, local_rank = dist_env()
    one = world == 1
    names = [args.workload]
    if one and not args.no_all_workloads and not (args.batch or args.corpus_tokens or args.prompt_len or args.gen_len):
        names += [n for n in ORDER if n != args.workload]
    kids = None
    if one and not args.no_cpu_baseline:
        kids = OracleChildren(names, args, args.warmup)       # spawned before the first CUDA call

    import torch
    if not torch.cuda.is_available():
        if kids:
            kids.close()
        raise SystemExit("bench.py needs a CUDA device: the retrieval path has no CPU implementation")
    torch.cuda.set_device(local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group(backend="nccl", device_id=torch.device("cuda", local_rank))
    import paper_2411_10666_b200 as P
    P.lib()

    t_all = time.perf_counter()
    results = {}
    for n in names:
        results[n] = measure_gpu(P, args, n, rank, world, local_rank, full=(n == args.workload))
    gpu_part_s = time.perf_counter() - t_all
    dev_counters = None
    if one and rank == 0 and not args.no_probes:
        dev_counters = device_counters(args, args.workload)      # (the oracle's automata are still being built meanwhile)
    if rank != 0:
        if world > 1:
            torch.distributed.destroy_process_group()
        return 0

    # the oracle's timed runs, one after the other, once every automaton is built
    cpu = {}
    if kids:
        t_wait = time.perf_counter()
        for n in names:
            kids.wait_ready(n, max(30.0, args.cpu_wait_seconds - (time.perf_counter() - t_wait)))
        for n in names:
            cpu[n] = kids.collect(n)
        kids.close()

    head = results[args.workload]
    probes = head.get("probes")
    head_cpu = cpu.get(args.workload)
    line = {
        "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": head["K"], "warmup": head["Wm"],
        "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int32", "data": "synthetic",
        "config": config_dict(head["base"], head["label"], world),
        "timing": {"repeats": head["repeats"], "how": "median of repeats, CUDA events, max over ranks",
                   "gpu_part_seconds": gpu_part_s},
        "draft_tokens_per_sec": head["draft_tokens_per_sec"],
        "accepted_tokens_per_sec": head["accepted_tokens_per_sec"],
        "best_ms_per_step": head["best_ms_per_step"],
        "prefill_tokens_per_sec": head["prefill_tokens_per_sec"],
        "static": head["static"], "static_build_seconds": head["static"]["seconds"],
        "status_all_ok": head["status_all_ok"],
        "e2e": head["e2e"], "gpu_launches": head["gpu_launches"], "graph_replay": head["graph_replay"],
        "clocks": head["clocks"],
        "roofline": roofline_block(head, head_cpu if head_cpu and "value" in head_cpu else None, probes, dev_counters),
    }
    if dev_counters:
        line["kernel_counters"] = {"per_sequence_step": {k: round(v, 3) for k, v in dev_counters["per_sequence_step"].items()},
                                   "steps": dev_counters["steps"], "how": "python bench_counters.py (library built with -DSAM_COUNTERS)"}
    for k in ("tree_draft", "closed_loop"):
        if k in head:
            line[k] = head[k]
    if head_cpu is not None:
        line["cpu_baseline"] = ({k: v for k, v in head_cpu.items() if k != "counters"} if "value" in head_cpu
                                else {"value": None, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
                                      "sample": "none", "unavailable": head_cpu.get("unavailable")})
    if len(names) > 1:
        allw = {}
        for n in ORDER:
            r = results[n]
            c = cpu.get(n)
            ok = bool(c) and "value" in c
            rf = roofline_block(r, c if ok else None, probes if n == args.workload else None)
            allw[n] = {"value": r["value"], "unit": UNIT, "us_per_step": r["ms_per_step"] * 1e3, "batch": r["B"],
                       "steps": r["K"], "repeats": r["repeats"], "launches_per_step": r["launches_per_step"],
                       "draft_tokens_per_sec": r["draft_tokens_per_sec"], "e2e_value": r["e2e"]["value"],
                       "static_bytes": r["static"]["device_bytes"], "status_all_ok": r["status_all_ok"],
                       "algorithmic_bytes_per_sequence_step": rf["algorithmic_bytes_per_sequence_step"],
                       "achieved_GBps": rf["achieved"], "frac_of_stream_copy": rf["frac"],
                       "cpu_oracle_value": c["value"] if ok else None,
                       "cpu_oracle_cores": c["cores"] if ok else None,
                       "cpu_oracle_note": None if ok else (c or {}).get("unavailable", "not run")}
            if probes:
                allw[n]["frac_of_random_32B"] = rf["achieved"] / probes["random_read"]["32"]["GB/s"]
        line["all_workloads"] = allw
        line["all_workloads_note"] = ("the four other recipes measured the same way with a shorter timed region; the random-read "
                                      "rate in their fractions is the one measured over the headline workload's footprint")
    print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()
    return 0


if __name__ == "__main__":
    a = parse_args()
    sys.exit(main_reference(a) if a.impl == "reference" else main_ours(a))
