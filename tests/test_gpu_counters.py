"""GPU: the operation counters of the step kernels (library built with -DSAM_COUNTERS) against the
CPU oracle's.  What both sides can count — the link and next moves of Transfer on the static
automaton (Algorithm 1), and of Expand the transitions added on the suffix-link walk, the clones,
the transitions a clone copies and the redirected transitions (Algorithm 3) — must agree exactly,
whichever way the kernels went about it (one Expand at a time, runs of new tokens, runs of cloning
tokens, matches followed through prefix states, the split step with its per-lane static chains)."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest

import oracle
import workloads as W

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SAME = ("static_link_moves", "static_next_moves", "walk_inserts", "clones", "copied_edges", "redirects", "tokens", "seq_steps")


def _device_counts(args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench_counters.py"), "--from-reset"] + args,
                         capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-3000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    return json.loads(lines[-1])


@pytest.mark.parametrize("name,corpus,batch,pl,gl", [("c2", 300_000, 24, 300, 500), ("c4", 100_000, 32, 900, 400),
                                                     ("c5", 200_000, 1700, 60, 90), ("c5", 200_000, 8300, 60, 60)])
def test_counts_equal_the_oracles(name, corpus, batch, pl, gl):
    got = _device_counts(["--workload", name, "--corpus-tokens", str(corpus), "--batch", str(batch),
                          "--prompt-len", str(pl), "--gen-len", str(gl)])
    assert got["status_all_ok"] and got["launches_per_step"] == (2 if batch >= 1536 else 1)
    spec = W.scaled(W.SPECS[name], corpus, batch, pl, gl)
    w = W.make(spec)
    S = oracle.Sam(w.corpus)
    ob = oracle.Batch(S, w.corpus, batch, spec.vocab, pl + gl)
    ob.step(w.prompts, np.full(batch, pl, dtype=np.int32), spec.draft_len, 8)
    ob.run(w.new_tokens, w.counts, spec.draft_len, 8)
    ref = ob.counters()
    for k in SAME:
        assert got["counters"][k] == ref[k], (k, got["counters"][k], ref[k])
    # the rounds of dependent reads are the kernels' own figure: at least the control words and the draft
    c = got["counters"]
    assert c["static_rounds"] >= c["seq_steps"] and c["dynamic_rounds"] >= 2 * c["seq_steps"]
