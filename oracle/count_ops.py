"""Operation counters of the CPU oracle on a workload's generation phase, and the algorithmic
bytes per sequence-step that follow from them.  TEST INFRASTRUCTURE (calls only oracle/ and the
input generator).

    python -m oracle.count_ops c2 [c4 ...]

Byte model (what the method itself must touch, independent of any layout tuning beyond "a state
is a 32-byte record"):
  static  : 32 B per Transfer move (each link or next move lands on one state record)
  dynamic : per accepted token 32 B (new state) + 8 B (its two link fields) + 4 B (text append);
            per walk-insert 32 B read + 8 B transition written; per clone 32 B read + 32 B written;
            per redirect 32 B read + 4 B written
  per step: 2 x 32 B (the two matched states' records for min_endpos), 4 B per drafted token read,
            the output row (4 L + 28 B) and the input row (4 m + 4 B)
"""
from __future__ import annotations

import json
import sys
import time

import numpy as np

import oracle
import workloads as W


def count(name: str, threads: int = 8) -> dict:
    spec = W.SPECS[name]
    w = W.make(spec)
    t0 = time.time()
    S = oracle.Sam(w.corpus)
    build_s = time.time() - t0
    B, L = spec.batch, spec.draft_len
    ob = oracle.Batch(S, w.corpus, B, spec.vocab, spec.prompt_len + spec.gen_len)
    ob.step(w.prompts, np.full(B, spec.prompt_len, dtype=np.int32), L, threads)
    c0 = ob.counters()
    drafted = 0
    for s in range(w.n_steps):
        out = ob.step(w.new_tokens[s], w.counts[s], L, threads)
        drafted += int(out.draft_len[w.counts[s] > 0].sum())
    c1 = ob.counters()
    d = {k: c1[k] - c0[k] for k in c1}
    steps, toks = d["seq_steps"], d["tokens"]
    static_b = 32 * (d["static_link_moves"] + d["static_next_moves"])
    dyn_b = toks * (32 + 8 + 4) + d["walk_inserts"] * 40 + d["clones"] * 64 + d["redirects"] * 36
    step_b = steps * (64 + 4 * L + 28 + 4) + 4 * toks + 4 * drafted
    total = static_b + dyn_b + step_b
    return {
        "workload": name, "seq_steps": steps, "tokens": toks, "tokens_per_seq_step": toks / steps,
        "drafted_tokens_per_seq_step": drafted / steps,
        "per_token": {k: d[k] / toks for k in ("static_link_moves", "static_next_moves", "dynamic_link_moves",
                                                "dynamic_next_moves", "walk_inserts", "clones", "copied_edges",
                                                "redirects")},
        "bytes_per_seq_step": {"static": static_b / steps, "dynamic": dyn_b / steps, "step_io": step_b / steps,
                               "total": total / steps},
        "static_states": S.n_states, "static_transitions": S.n_transitions, "oracle_build_s": build_s,
        "dyn_states_per_token": c1["dyn_states"] / c1["tokens"],
        "dyn_transitions_per_token": c1["dyn_transitions"] / c1["tokens"],
    }


if __name__ == "__main__":
    for n in sys.argv[1:] or ["tiny"]:
        print(json.dumps(count(n)), flush=True)
