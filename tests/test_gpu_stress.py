"""GPU: randomized parity stress, off by default (set SAMDRAFT_STRESS_SECONDS to run it that long).

Seed after seed, a reduced instance of one of the five workload recipes and a random text over a tiny
vocabulary are run through the CUDA library and through the CPU oracle; every output of every step
and the dynamic automata, state for state, must be equal.  Every fifth seed also runs a batch of more than
8192 short sequences (the split step) with random l_bias / min_match / stop token and some slots sitting steps out."""
import os
import random
import time

import numpy as np
import pytest

import workloads as W
from _parity import assert_dynamic_automata_equal, assert_same, gpu_run, oracle_run
from test_gpu_parity import _rand_text, _steps_from_text

pytestmark = pytest.mark.gpu

SECONDS = float(os.environ.get("SAMDRAFT_STRESS_SECONDS", "0") or 0)
CASES = {"c2": (300_000, 16, 400, 700), "c3": (400_000, 24, 500, 800), "c4": (150_000, 32, 1200, 700),
         "c5": (400_000, 64, 500, 500), "tiny": (60_000, 4, 256, 512)}


@pytest.mark.skipif(SECONDS <= 0, reason="set SAMDRAFT_STRESS_SECONDS=<seconds> to run the randomized stress")
def test_randomized_parity_stress():
    import paper_2411_10666_b200 as P
    P.lib()
    t0, seed, done = time.time(), int(os.environ.get("SAMDRAFT_STRESS_SEED", "1000")), 0
    while time.time() - t0 < SECONDS:
        seed += 1
        key = list(CASES)[seed % len(CASES)]
        N, B, pl, gl = CASES[key]
        spec = W.scaled(W.SPECS[key], N, B, pl, gl, seed=seed)
        w = W.make(spec)
        L, msl = spec.draft_len, spec.prompt_len + spec.gen_len
        st = P.StaticSam.build(w.corpus, spec.vocab)
        ref, ob, _ = oracle_run(w.corpus, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl, threads=8)
        got, batch = gpu_run(P, st, spec.vocab, w.prompts, w.new_tokens, w.counts, L, msl)
        assert_same(got, ref, "%s seed %d" % (key, seed))
        assert (got["status"] == 0).all()
        assert_dynamic_automata_equal(batch, ob, range(min(B, 6)), msl)
        batch.close()
        rng = random.Random(seed)
        vocab = rng.choice([2, 3, 4, 7, 30]); n = rng.choice([300, 900, 2000]); kmax = rng.choice([1, 5, 16, 40])
        x = _rand_text(rng, n, vocab, rng.choice([0.2, 0.4, 0.7]))
        nt, ct = _steps_from_text(x, rng, kmax)
        corpus = np.array(_rand_text(rng, rng.choice([50, 800]), vocab, 0.3), dtype=np.int32)
        st = P.StaticSam.build(corpus, vocab)
        empty = np.zeros((1, 0), np.int32)
        ref, ob, _ = oracle_run(corpus, vocab, empty, nt, ct, 8, n)
        got, batch = gpu_run(P, st, vocab, empty, nt, ct, 8, n)
        assert_same(got, ref, "small text, seed %d" % seed)
        assert_dynamic_automata_equal(batch, ob, [0], n)
        batch.close()
        if seed % 5 == 0:                                   # the split step: more than 8192 slots, short sequences
            key = rng.choice(["c5", "c2", "c4"])
            B = rng.choice([8200, 8333, 9000])
            spec = W.scaled(W.SPECS[key], rng.choice([50_000, 200_000]), B, rng.choice([20, 90, 150]), rng.choice([40, 80]), seed=seed)
            w = W.make(spec)
            L, msl = rng.choice([4, 32, 40]), spec.prompt_len + spec.gen_len
            counts = w.counts.copy()
            counts[rng.randrange(counts.shape[0]), ::rng.choice([3, 11])] = 0
            l_bias, min_match, stop = rng.choice([(0, 1, -1), (1, 2, 5), (5, 5, -1), (0, 0, 17)])
            st = P.StaticSam.build(w.corpus, spec.vocab)
            ref, ob, _ = oracle_run(w.corpus, spec.vocab, w.prompts, w.new_tokens, counts, L, msl, l_bias, min_match,
                                    threads=8, stop_token=stop)
            got, batch = gpu_run(P, st, spec.vocab, w.prompts, w.new_tokens, counts, L, msl, l_bias, min_match, stop_token=stop)
            assert batch.launches_per_step() == 2
            assert_same(got, ref, "split step, %s seed %d" % (key, seed))
            assert_dynamic_automata_equal(batch, ob, [0, B // 2, B - 1], msl)
            batch.close()
        done += 1
    print("stress: %d seeds in %.0f s" % (done, time.time() - t0))
    assert done >= 1
