"""Host-side checks of the benchmark and of the workload recipes (no GPU)."""
import json
import os
import subprocess
import sys

import numpy as np

import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "40", "--warmup", "3"], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["impl"] == "reference" and j["metric"] == "sam_sequence_steps_per_sec" and j["unit"] == "sequence-steps/s"
    assert j["steps"] == 40 and j["warmup"] == 3 and j["value"] > 0 and j["higher_is_better"] is True
    assert j["cpu_baseline"]["kind"] == "oracle" and j["cpu_baseline"]["cores"] >= 1
    assert j["e2e"]["h2d_bytes_per_step"] == 0 and j["e2e"]["d2h_bytes_per_step"] == 0
    assert j["config"]["workload"] == "tiny"


def test_reference_arm_other_ranks_do_nothing():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--gpus", "2"], capture_output=True, text=True, timeout=120, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_recipes_have_the_stated_shape():
    for name, spec in W.SPECS.items():
        small = W.scaled(spec, corpus_len=min(spec.corpus_len, 200_000), batch=min(spec.batch, 8))
        w = W.make(small)
        assert w.corpus.shape == (small.corpus_len,) and w.corpus.dtype == np.int32
        assert w.corpus.min() >= 0 and w.corpus.max() < spec.vocab
        assert w.seqs.shape == (small.batch, spec.prompt_len + spec.gen_len)
        assert w.seqs.min() >= 0 and w.seqs.max() < spec.vocab
        c = w.counts
        assert (c.sum(axis=0) == spec.gen_len).all() and c.max() <= spec.accept_max and c.min() >= 0
        # the packed step rows are exactly the generated part, in order
        for b in range(small.batch):
            toks = np.concatenate([w.new_tokens[s, b, :c[s, b]] for s in range(w.n_steps)])
            assert np.array_equal(toks, w.seqs[b, spec.prompt_len:])
        assert (w.new_tokens[np.arange(spec.accept_max)[None, None, :] >= c[:, :, None]] == -1).all()
        mean_m = c[c > 0].mean()
        expect = {"tiny": 2.5, "c2": 2.46, "c3": 2.77, "c4": 3.87, "c5": 3.32}[name]
        assert abs(mean_m - expect) < 0.35, (name, mean_m)
    # seeds: same recipe twice gives the same arrays; another seed differs
    a = W.make(W.scaled(W.SPECS["tiny"], corpus_len=5000))
    b = W.make(W.scaled(W.SPECS["tiny"], corpus_len=5000))
    c2 = W.make(W.scaled(W.SPECS["tiny"], corpus_len=5000, seed=7))
    assert np.array_equal(a.corpus, b.corpus) and np.array_equal(a.seqs, b.seqs)
    assert not np.array_equal(a.corpus, c2.corpus)


def test_multi_document_recipe_joins_documents_with_the_separator():
    """The sixth recipe: separators stand at document ends only, documents have the stated lengths, and
    the CPU oracle run with the separator as stop token never drafts across a document boundary."""
    import oracle
    spec = W.scaled(W.DOCS, corpus_len=200_000, batch=6, prompt_len=150, gen_len=250)
    w = W.make(spec)
    ends = np.flatnonzero(w.corpus == spec.eos)
    assert ends[-1] == spec.corpus_len - 1
    lens = np.diff(np.concatenate([[-1], ends]))
    assert lens[:-1].min() >= spec.doc_lo and lens.max() <= spec.doc_hi
    S = oracle.Sam(w.corpus)
    L, B = spec.draft_len, spec.batch
    ob = oracle.Batch(S, w.corpus, B, spec.vocab, spec.prompt_len + spec.gen_len, stop_token=spec.eos)
    free = oracle.Batch(S, w.corpus, B, spec.vocab, spec.prompt_len + spec.gen_len)
    outs = [ob.step(w.prompts, np.full(B, spec.prompt_len, dtype=np.int32), L)]
    plain = [free.step(w.prompts, np.full(B, spec.prompt_len, dtype=np.int32), L)]
    for s in range(w.n_steps):
        outs.append(ob.step(w.new_tokens[s], w.counts[s], L))
        plain.append(free.step(w.new_tokens[s], w.counts[s], L))
    cut = 0
    for o, q in zip(outs, plain):
        assert not (o.draft_tokens == spec.eos).any()
        assert np.array_equal(o.match_len, q.match_len) and np.array_equal(o.source, q.source)
        for b in range(B):
            d, full = o.draft_tokens[b, :o.draft_len[b]], q.draft_tokens[b, :q.draft_len[b]]
            hit = np.flatnonzero(full == spec.eos)
            assert np.array_equal(d, full[:hit[0]] if len(hit) else full)     # the plain slice, cut at the separator
            cut += len(hit) > 0
    assert cut > 0


def test_byte_model_and_workload_naming_of_the_benchmark():
    """The benchmark's algorithmic-byte model on hand-made counters, and the `config` object, which must be the
    same for the GPU arm and the reference arm (both build it with the one function)."""
    sys.path.insert(0, ROOT)
    import bench
    c = dict(seq_steps=10, tokens=30, static_link_moves=5, static_next_moves=25, dynamic_link_moves=7, dynamic_next_moves=20,
             walk_inserts=60, clones=4, copied_edges=5, redirects=6, draft_tokens=200)
    b = bench.algorithmic_bytes(c, 32)
    assert b["static"] == 32 * 30 / 10
    assert b["dynamic"] == (30 * 44 + 60 * 40 + 4 * 64 + 6 * 36) / 10
    assert b["step_io"] == (10 * (64 + 4 * 32 + 28 + 4) + 4 * 30 + 4 * 200) / 10
    assert abs(b["total"] - (b["static"] + b["dynamic"] + b["step_io"])) < 1e-9
    d = bench.dependent_accesses(c)
    assert d == {"static_chain": 30 / 10 + 2, "dynamic_chain": (7 + 20 + 4 + 6) / 10 + 2}
    a = bench.parse_args(["--workload", "c4", "--batch", "77", "--impl", "reference"])
    spec = bench.named_variant(a, "c4")
    assert spec.batch == 77 and bench.named_variant(a, "c2").batch == W.SPECS["c2"].batch
    cfg = bench.config_dict(spec, bench.named_label(a, "c4"), 2)
    assert cfg["workload"] == "c4 (recipe run with 77 sequences)" and cfg["global_batch"] == 154 and cfg["batch_per_gpu"] == 77
    assert set(cfg) >= {"workload", "batch_per_gpu", "global_batch", "prompt_len", "gen_len", "draft_len", "corpus_tokens", "vocab", "l2"}
    assert len(bench.kernel_digest()) == 16
