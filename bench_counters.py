#!/usr/bin/env python
"""Operation counts of the step kernels on a workload, from the library built with -DSAM_COUNTERS.

    python bench_counters.py --workload c5 [--warmup 8 --steps 512] [--batch N] [--corpus-tokens N] [--from-reset]

Runs the workload's prompt prefill and decoding steps through `sam_step` with the counters attached and
prints one JSON line: per counter the sum over all slots for the decoding steps [warmup, warmup + steps)
(or, with --from-reset, for everything since the empty batch: prefill and all steps), and the means per
sequence-step that `bench.py` turns into the dependent-access bound.  The counters build is a second
compilation of the same sources; this script re-runs itself with SAMDRAFT_VARIANT=counters so that the
package loads it.  It needs a CUDA device.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c5")
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--steps", type=int, default=512)
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--corpus-tokens", type=int, default=0)
    ap.add_argument("--prompt-len", type=int, default=0)
    ap.add_argument("--gen-len", type=int, default=0)
    ap.add_argument("--from-reset", action="store_true", help="count the prefill and every decoding step")
    return ap.parse_args(argv)


def main():
    args = parse_args()
    if os.environ.get("SAMDRAFT_VARIANT") != "counters":
        env = dict(os.environ, SAMDRAFT_VARIANT="counters")
        return subprocess.call([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env)
    import numpy as np
    import torch
    import workloads as W
    import paper_2411_10666_b200 as P
    sd = P.binding
    P.lib()
    assert sd.sam_counters_available(), "the library was not built with -DSAM_COUNTERS"
    base = W.DOCS if args.workload == "docs" else W.SPECS[args.workload]
    spec = W.scaled(base, corpus_len=args.corpus_tokens or None, batch=args.batch or None,
                    prompt_len=args.prompt_len or None, gen_len=args.gen_len or None)
    corpus = W.make_corpus(spec)
    seqs, counts, new_tokens = W.make_sequences(spec, corpus)
    B, L = seqs.shape[0], spec.draft_len
    n_steps = counts.shape[0]
    lo = 0 if args.from_reset else min(args.warmup, n_steps)
    hi = n_steps if args.from_reset else min(lo + args.steps, n_steps)
    st = P.StaticSam.build(corpus, spec.vocab)
    batch = P.Batch(st, B, spec.prompt_len + spec.gen_len, max_draft_len=L)
    dev = batch.device
    out = P.StepOutputs(B, L, dev)
    cnt = torch.zeros((B, sd.N_COUNTERS), dtype=torch.int64, device=dev)
    nt = torch.from_numpy(new_tokens[:hi]).to(dev)
    ct = torch.from_numpy(counts[:hi]).to(dev)
    torch.cuda.synchronize()
    if args.from_reset:
        sd.sam_counters_attach(cnt, B)
    batch.step(torch.from_numpy(np.ascontiguousarray(seqs[:, :spec.prompt_len])).to(dev),
               torch.full((B,), spec.prompt_len, dtype=torch.int32, device=dev), L, out)
    if lo > 0:
        batch.run_steps(nt[:lo], ct[:lo], L, per_step=False, out=out)
    torch.cuda.synchronize()
    if not args.from_reset:
        sd.sam_counters_attach(cnt, B)
    if hi > lo:
        batch.run_steps(nt[lo:hi], ct[lo:hi], L, per_step=False, out=out)
    torch.cuda.synchronize()
    sd.sam_counters_attach(None)
    ok = bool((out.status == 0).all().item())
    tot = cnt.sum(dim=0).tolist()
    res = {k: int(tot[i]) for i, k in enumerate(sd.COUNTER_NAMES)}
    steps = max(res["seq_steps"], 1)
    line = {"workload": spec.name, "batch": B, "corpus_tokens": spec.corpus_len, "steps": [lo, hi], "from_reset": args.from_reset,
            "launches_per_step": batch.launches_per_step(), "status_all_ok": ok, "counters": res,
            "per_sequence_step": {k: res[k] / steps for k in res}}
    print(json.dumps(line))
    return 0


if __name__ == "__main__":
    sys.exit(main())
