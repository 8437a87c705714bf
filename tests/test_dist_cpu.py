"""World-size-2 run of the benchmark's multi-rank plumbing on CPU (gloo): batch sharding with no
data-path collective, and the max-time / sum-units reduction."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import workloads as W


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import oracle
    base = W.scaled(W.SPECS["tiny"], corpus_len=20000, batch=3, prompt_len=32, gen_len=64)
    spec, corpus, seqs, counts, new_tokens = bench.shard_workload(base, rank, world)
    # each rank runs its shard on its own (here: the oracle stands in for the device)
    S = oracle.Sam(corpus)
    ob = oracle.Batch(S, corpus, seqs.shape[0], spec.vocab, spec.prompt_len + spec.gen_len)
    ob.step(np.ascontiguousarray(seqs[:, :spec.prompt_len]), np.full(seqs.shape[0], spec.prompt_len, dtype=np.int32), 8)
    out = ob.run(new_tokens, counts, 8)
    units = int((counts > 0).sum())
    ms, total = bench.reduce_max_sum(10.0 + rank, units, world)
    q.put((rank, seqs, counts, out.match_len.copy(), units, ms, total))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_the_batch_and_reduce():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted([q.get(timeout=240) for _ in range(world)], key=lambda t: t[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # the union of the shards is the single-process batch of world x 3 sequences, in order
    base = W.scaled(W.SPECS["tiny"], corpus_len=20000, batch=3 * world, prompt_len=32, gen_len=64)
    w = W.make(base)
    assert np.array_equal(np.concatenate([g[1] for g in got]), w.seqs)
    assert np.array_equal(np.concatenate([g[2] for g in got], axis=1), w.counts)
    units = [g[4] for g in got]
    for g in got:
        assert g[5] == 11.0 and g[6] == sum(units)          # max time, summed units on every rank
    # and a rank's results do not depend on the other rank's sequences
    import oracle
    S = oracle.Sam(w.corpus)
    ob = oracle.Batch(S, w.corpus, base.batch, base.vocab, base.prompt_len + base.gen_len)
    ob.step(w.prompts, np.full(base.batch, base.prompt_len, dtype=np.int32), 8)
    ref = ob.run(w.new_tokens, w.counts, 8)
    assert np.array_equal(np.concatenate([g[3] for g in got]), ref.match_len)


def test_shard_bounds_cover_everything():
    for batch in (1, 7, 64, 4096):
        for world in (1, 2, 3, 8):
            b = [W.shard_bounds(batch, r, world) for r in range(world)]
            assert b[0][0] == 0 and b[-1][1] == batch
            assert all(b[i][1] == b[i + 1][0] for i in range(world - 1))
            sizes = [hi - lo for lo, hi in b]
            assert max(sizes) - min(sizes) <= 1
