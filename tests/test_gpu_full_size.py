"""CUDA path against the CPU oracle at the sizes and shapes of the benchmark configurations.

The oracle is too slow to sweep 738 M tokens, so at full size it is loaded with the whole corpus
(same counts, same tables) and asked for the chains of a random sample of tokens, which depend on
nothing but the sweep-start state; whole oracle sweeps (its token loop shared among the host's
cores, which a CPU test shows to be the serial sweep token for token) run at 99 M tokens.
"""
import os

import numpy as np
import pytest

from oracle import ldaref
from paper_1412_1576_b200 import binding, synth

pytestmark = pytest.mark.gpu

CORES = max(1, len(os.sched_getaffinity(0)))


def _free_gib():
    import gc
    import torch
    gc.collect()
    torch.cuda.empty_cache()       # contexts of earlier tests gave their memory back to torch's pool
    return torch.cuda.mem_get_info()[0] / 2 ** 30


def _host_gib():
    try:
        with open("/proc/meminfo") as f:
            for ln in f:
                if ln.startswith("MemAvailable"):
                    return int(ln.split()[1]) / 2 ** 20
    except OSError:
        pass
    return 0.0


def _gpu_and_oracle(c, seed, options=None):
    """The library loaded from device tensors, the oracle from host copies of the same arrays."""
    import torch
    g = binding.LightLDA(c.V, c.K, c.alpha, c.beta, options=options)
    g.load_corpus(c.word_ids, c.doc_offsets)
    g.init(seed)
    w = c.word_ids.cpu().numpy()
    off = c.doc_offsets.cpu().numpy()
    o = ldaref.Oracle(c.V, c.K, c.alpha, c.beta)
    o.load_corpus(w, off)
    o.init(seed)
    torch.cuda.empty_cache()
    return g, o, w, off


def _doc_rows_brute_force(z, off, docs):
    rows = {}
    for d in docs:
        uk, uc = np.unique(z[off[d]:off[d + 1]], return_counts=True)
        rows[int(d)] = (uk.astype(np.int32), uc.astype(np.int32))
    return rows


def test_large_full_size_sampled_tokens_against_oracle():
    """Config 4 at its full size (738 M tokens, K = 10 000), in the launch configuration bench.py times:
    after one sweep from a common start, 200 000 random tokens must carry exactly the topic the oracle's
    chain gives them; n_k must equal the oracle's before the sweep and the histogram of z after it; and
    the n_kd rows of a sample of documents must equal a brute-force count."""
    import torch
    scale = 1.0
    if _free_gib() < 70 or _host_gib() < 60:
        scale = 0.25      # the largest size this box holds; a smaller one is not worth the name
    if _free_gib() < 20 or _host_gib() < 16:
        pytest.skip("needs 20 GB of device memory and 16 GB of host memory even at a quarter of the documents")
    c = synth.make("large", seed=0, device="cuda", scale=scale)
    N = c.n_tokens
    g, o, w, off = _gpu_and_oracle(c, 1234)
    del c
    torch.cuda.empty_cache()
    assert np.array_equal(g.get_nk(), o.get_nk())
    rng = np.random.default_rng(5)
    toks = np.unique(rng.integers(0, N, size=200_000))
    want = o.sample_tokens(toks, 2)                 # chains of sweep 0 from the common start
    z0 = o.get_assignments()
    g.sweep(1, 2)
    z1 = g.get_assignments()
    assert np.array_equal(z1[toks], want)
    assert float(np.mean(z1[toks] != z0[toks])) > 0.05      # the sample did move
    nk = np.bincount(z1, minlength=g.K)
    assert np.array_equal(g.get_nk(), nk) and int(nk.sum()) == N
    # n_kd of a sample of documents, and n_kw of a sample of words, against brute-force counts of z1
    ro, top, cnt = g.get_csr(binding.LDA_NDK)
    docs = rng.integers(0, off.size - 1, size=200)
    for d, (uk, uc) in _doc_rows_brute_force(z1, off, docs).items():
        assert np.array_equal(top[ro[d]:ro[d + 1]], uk)
        assert np.array_equal(cnt[ro[d]:ro[d + 1]], uc)
    assert int(ro[-1]) == g.stats()["nnz_dk"]
    del ro, top, cnt
    ro, top, cnt = g.get_csr(binding.LDA_NWK)
    order = np.argsort(w, kind="stable")
    woff = np.searchsorted(w[order], np.arange(g.V + 1))
    for wd in rng.integers(0, g.V, size=200):
        uk, uc = np.unique(z1[order[woff[wd]:woff[wd + 1]]], return_counts=True)
        assert np.array_equal(top[ro[wd]:ro[wd + 1]], uk)
        assert np.array_equal(cnt[ro[wd]:ro[wd + 1]], uc)
    # a second sweep, with the configuration's own four steps, from the state both sides now share
    o.set_assignments(z1, 1234, 1)
    want = o.sample_tokens(toks, 4)
    g.sweep(1, 4)
    assert np.array_equal(g.get_assignments()[toks], want)
    st = g.stats()
    assert st["word_proposed"] == 2 * N and st["doc_proposed"] == 2 * N
    assert 0 < st["word_accepted"] < 2 * N and 0 < st["doc_accepted"] < 2 * N


def test_mid_full_size_two_whole_sweeps():
    """Config 3 at its full size (99 M tokens, K = 1000, documents of ~330 tokens): two whole oracle sweeps;
    every token, every count, every alias table and the move counters equal.  The library runs pass 1 in three
    vocabulary slices (one slice's alias tables in memory at a time), which must not show."""
    import torch
    if _free_gib() < 12 or _host_gib() < 12:
        pytest.skip("needs 12 GB of device and of host memory")
    c = synth.make("mid", seed=0, device="cuda")
    g, o, w, off = _gpu_and_oracle(c, 77, options={"alias_slices": 3})
    del c
    torch.cuda.empty_cache()
    for sweep in range(2):
        g.sweep(1, 2)
        o.sweep_threads(1, 2, CORES)
        assert np.array_equal(g.get_assignments(), o.get_assignments()), sweep
        st = g.stats()
        assert (st["word_accepted"], st["doc_accepted"]) == o.moves()
    assert np.array_equal(g.get_nk(), o.get_nk())
    for which in (binding.LDA_NWK, binding.LDA_NDK):
        a, b = g.get_csr(which), o.get_csr(which)
        for x, y in zip(a, b):
            assert np.array_equal(x, y)
    a, b = g.get_tables(), o.get_tables()
    assert a["dense_mass"] == b["dense_mass"]
    for k in ("dn_thr32", "dn_alias", "mix32", "sp_thr32", "sp_alias"):
        assert np.array_equal(a[k], b[k]), k
    for x, y in zip(g.loglik(), o.loglik()):
        assert x == pytest.approx(y, rel=1e-8)       # ~2e8 lgamma terms added in different orders


def test_big_shape_sample_against_oracle():
    """Config 5's shape (V = 1 M, K = 100 000: 32-bit topics, rows too long for shared memory, log-normal
    document lengths) at 1 % of its documents: two sweeps, everything equal."""
    c = synth.make("big", seed=0, scale=0.01)
    g = binding.LightLDA(c.V, c.K, c.alpha, c.beta)
    g.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
    g.init(31)
    o = ldaref.Oracle(c.V, c.K, c.alpha, c.beta)
    o.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
    o.init(31)
    assert np.array_equal(g.get_assignments(), o.get_assignments())
    for sweep in range(2):
        g.sweep(1, 2)
        o.sweep_threads(1, 2, CORES)
        assert np.array_equal(g.get_assignments(), o.get_assignments()), sweep
    assert np.array_equal(g.get_nk(), o.get_nk())
    for which in (binding.LDA_NWK, binding.LDA_NDK):
        a, b = g.get_csr(which), o.get_csr(which)
        for x, y in zip(a, b):
            assert np.array_equal(x, y)
    a, b = g.get_tables(), o.get_tables()
    for k in ("dn_thr32", "dn_alias", "mix32", "sp_thr32", "sp_alias"):
        assert np.array_equal(a[k], b[k]), k
    for x, y in zip(g.loglik(), o.loglik()):
        assert x == pytest.approx(y, rel=1e-9)


def test_big_full_size_invariants_and_sampled_tokens():
    """Config 5 at its full size (~1 G tokens, 105 GB on the device): the counts must be those of the
    library's own assignments, and a sample of tokens must carry the topic the oracle's chain gives them."""
    import torch
    if _free_gib() < 150 or _host_gib() < 100:
        pytest.skip("needs 150 GB of free device memory and 100 GB of host memory")
    c = synth.make("big", seed=0, device="cuda")
    N = c.n_tokens
    g, o, w, off = _gpu_and_oracle(c, 4321)
    del c
    torch.cuda.empty_cache()
    assert np.array_equal(g.get_nk(), o.get_nk())
    rng = np.random.default_rng(6)
    toks = np.unique(rng.integers(0, N, size=100_000))
    want = o.sample_tokens(toks, 2)
    g.sweep(1, 2)
    z1 = g.get_assignments()
    assert np.array_equal(z1[toks], want)
    nk = np.bincount(z1, minlength=g.K)
    assert np.array_equal(g.get_nk(), nk) and int(nk.sum()) == N
    st = g.stats()
    zc = torch.from_numpy(z1).cuda().long()
    key_w = torch.from_numpy(w).cuda().long() * g.K + zc
    assert st["nnz_wk"] == int(torch.unique(key_w).numel())
    del key_w
    doc = torch.repeat_interleave(torch.arange(off.size - 1, device="cuda"), torch.from_numpy(np.diff(off)).cuda())
    key_d = doc * g.K + zc
    del doc, zc
    assert st["nnz_dk"] == int(torch.unique(key_d).numel())


@pytest.mark.parametrize("workload,scale", [("tiny", 1.0), ("mid", 0.05)])
def test_loglik_trajectory_50_sweeps(workload, scale):
    """Free-running 50 sweeps: log-likelihood within 0.5 % of the oracle's at every checked sweep (in fact
    equal to rounding, since every assignment is)."""
    c = synth.make(workload, seed=2, scale=scale)
    g = binding.LightLDA(c.V, c.K, c.alpha, c.beta)
    g.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
    g.init(99)
    o = ldaref.Oracle(c.V, c.K, c.alpha, c.beta)
    o.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
    o.init(99)
    first = None
    for sweep in range(50):
        g.sweep(1, 2)
        o.sweep_threads(1, 2, CORES)
        if sweep % 7 == 0 or sweep == 49:
            a, b = g.loglik()[0], o.loglik()[0]
            first = b if first is None else first
            assert abs(a - b) <= 0.005 * abs(b), (sweep, a, b)
    assert b > first                         # the chain did climb
    assert float(np.mean(g.get_assignments() == o.get_assignments())) >= 0.999
