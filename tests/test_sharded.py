"""Document-sharded runs: the orchestration (paper_1412_1576_b200/sharded.py) on two gloo ranks on
CPU with the oracle as the engine, and -- on a GPU -- with two library contexts in one process.
Either way a sharded run must produce exactly the assignments of one context holding every document."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import ldaref  # noqa: E402
from paper_1412_1576_b200 import sharded, synth  # noqa: E402

SEED, SWEEPS, STEPS = 31, 3, 2


def _corpus():
    return synth.generate(V=300, K=24, D=90, length=("poisson", 40.0), zipf_s=1.0, alpha=0.2, beta=0.05, seed=4)


def _single_oracle(c):
    o = ldaref.Oracle(c.V, c.K, c.alpha, c.beta)
    o.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
    o.init(SEED)
    o.sweep(SWEEPS, STEPS)
    return o


def _gloo_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    c = _corpus()
    w, off = c.word_ids.numpy(), c.doc_offsets.numpy()
    d0, d1 = sharded.shard_documents(off, world, rank)
    run = sharded.ShardedSweep(ldaref.Oracle(c.V, c.K, c.alpha, c.beta), np.zeros(c.V * c.K, np.int32))
    run.load(w, off, d0, d1, sharded.term_frequencies(w, c.V))
    run.init(SEED)
    run.sweep(SWEEPS, STEPS)
    word, doc = run.loglik_parts()
    docs = torch.tensor([doc], dtype=torch.float64)
    dist.all_reduce(docs)
    out[rank] = (d0, d1, run.engine.get_assignments().copy(), run.engine.get_nk().copy(), word, float(docs[0]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_equal_one_context():
    world = 2
    port = 29500 + (os.getpid() % 2000) + 7
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_gloo_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    c = _corpus()
    one = _single_oracle(c)
    off = c.doc_offsets.numpy()
    assert res[0][0] == 0 and res[0][1] == res[1][0] and res[1][1] == off.size - 1 and 0 < res[0][1] < off.size - 1
    z = np.concatenate([res[0][2], res[1][2]])
    assert np.array_equal(z, one.get_assignments())
    for r in range(world):
        assert np.array_equal(res[r][3], one.get_nk())          # every shard ends with the summed n_k
        total, word, doc = one.loglik()
        assert res[r][4] == pytest.approx(word, rel=1e-12) and res[r][5] == pytest.approx(doc, rel=1e-12)


def test_shard_cuts_cover_the_documents_and_balance_tokens():
    off = np.concatenate([[0], np.cumsum(np.random.default_rng(0).integers(0, 50, size=1000))])
    for world in (1, 2, 3, 8):
        cuts = [sharded.shard_documents(off, world, r) for r in range(world)]
        assert cuts[0][0] == 0 and cuts[-1][1] == 1000 and all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
        tokens = [off[b] - off[a] for a, b in cuts]
        assert max(tokens) - min(tokens) <= 2 * 50


@pytest.mark.gpu
def test_two_library_shards_in_one_process_equal_one_context_and_the_oracle():
    """Both shards on the one GPU, one after the other (no kernel waits for another): the collective is a
    plain sum of the two matrices here; what the library does around it is what runs with NCCL."""
    from paper_1412_1576_b200 import binding
    for c in (_corpus(), synth.make("small", seed=0)):
        w, off = c.word_ids.numpy(), c.doc_offsets.numpy()
        tf = sharded.term_frequencies(w, c.V)
        world = 2
        mats = [torch.zeros(c.V * c.K, dtype=torch.int32, device="cuda") for _ in range(world)]
        runs = []
        for r in range(world):
            run = sharded.ShardedSweep(binding.LightLDA(c.V, c.K, c.alpha, c.beta), mats[r], all_reduce=None)
            run.load(w, off, *sharded.shard_documents(off, world, r), tf)
            runs.append(run)

        def exchange_all():
            for run in runs:
                run.engine.word_counts_to_dense(run.matrix)
            total = mats[0] + mats[1]
            for run in runs:
                run.matrix.copy_(total)
                run.engine.word_counts_from_dense(run.matrix)
        for run in runs:
            run.engine.init(SEED)
        exchange_all()
        for _ in range(SWEEPS):
            for run in runs:
                run.engine.sweep(1, STEPS)
            exchange_all()
        z = np.concatenate([run.engine.get_assignments() for run in runs])
        one = binding.LightLDA(c.V, c.K, c.alpha, c.beta)
        one.load_corpus(w, off)
        one.init(SEED)
        one.sweep(SWEEPS, STEPS)
        assert np.array_equal(z, one.get_assignments())
        o = ldaref.Oracle(c.V, c.K, c.alpha, c.beta)
        o.load_corpus(w, off)
        o.init(SEED)
        o.sweep(SWEEPS, STEPS)
        assert np.array_equal(z, o.get_assignments())
        for run in runs:
            assert np.array_equal(run.engine.get_nk(), o.get_nk())
            a, b = run.engine.get_csr(binding.LDA_NWK), o.get_csr(ldaref.NWK)
            for x, y in zip(a, b):
                assert np.array_equal(x, y)
        word, doc = zip(*[run.loglik_parts() for run in runs])
        t, lw, ld = o.loglik()
        assert word[0] == pytest.approx(lw, rel=1e-10) and sum(doc) == pytest.approx(ld, rel=1e-10)
        # a matrix that does not fit the term frequencies is refused
        bad = torch.ones(c.V * c.K, dtype=torch.int32, device="cuda")
        with pytest.raises(binding.LdaError) as e:
            runs[0].engine.word_counts_from_dense(bad)
        assert e.value.status == binding.LDA_ERANGE
