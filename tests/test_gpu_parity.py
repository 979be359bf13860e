"""CUDA path against the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest

from oracle import ldaref
from paper_1412_1576_b200 import binding, synth

pytestmark = pytest.mark.gpu

SEED = 20260


def _pair(c, seed=SEED, options=None):
    g = binding.LightLDA(c.V, c.K, c.alpha, c.beta, options=options)
    g.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
    g.init(seed)
    o = ldaref.Oracle(c.V, c.K, c.alpha, c.beta)
    o.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
    o.init(seed)
    return g, o


def _assert_same_counts(g, o):
    assert np.array_equal(g.get_nk(), o.get_nk())
    for which in (binding.LDA_NWK, binding.LDA_NDK):
        a, b = g.get_csr(which), o.get_csr(which)
        assert np.array_equal(a[0], b[0])
        assert np.array_equal(a[1], b[1])
        assert np.array_equal(a[2], b[2])


def _assert_same_moves(g, o, n_tokens, word_steps, doc_steps, iters=1):
    """lda_stats' proposal counters of the last sweep call against the oracle's."""
    st = g.stats()
    assert (st["word_proposed"], st["doc_proposed"]) == (iters * n_tokens * word_steps, iters * n_tokens * doc_steps)
    assert (st["word_accepted"], st["doc_accepted"]) == o.moves()


def _assert_same_tables(g, o):
    a, b = g.get_tables(), o.get_tables()
    assert a["dense_mass"] == b["dense_mass"]
    for k in ("dn_thr32", "dn_alias", "mix32", "sp_thr32", "sp_alias"):
        assert np.array_equal(a[k], b[k]), k


def _toy(V, K, D, L, alpha=0.3, beta=0.2, seed=3, length=None):
    return synth.generate(V=V, K=K, D=D, length=length or ("fixed", L), zipf_s=None, alpha=alpha,
                          beta=beta, seed=seed)


def test_init_and_counts_tiny(tiny_corpus):
    g, o = _pair(tiny_corpus)
    assert np.array_equal(g.get_assignments(), o.get_assignments())
    _assert_same_counts(g, o)


def test_tables_bit_equal_tiny(tiny_corpus):
    g, o = _pair(tiny_corpus)
    _assert_same_tables(g, o)
    o.sweep(2, 2)
    g.set_assignments(o.get_assignments(), SEED, 2)
    _assert_same_counts(g, o)
    _assert_same_tables(g, o)


def test_sweeps_bit_equal_tiny(tiny_corpus):
    """fp64 acceptance in the same operation order: every token agrees, every sweep."""
    c = tiny_corpus
    g, o = _pair(tiny_corpus)
    for sweep in range(20):
        g.sweep(1, 2)
        o.sweep(1, 2)
        assert np.array_equal(g.get_assignments(), o.get_assignments()), sweep
        _assert_same_moves(g, o, c.n_tokens, 1, 1)
    _assert_same_counts(g, o)
    lg, lo = g.loglik(), o.loglik()
    for a, b in zip(lg, lo):
        assert a == pytest.approx(b, rel=1e-10)


@pytest.mark.parametrize("mh_steps", [1, 3, 4])
def test_other_step_counts_tiny(tiny_corpus, mh_steps):
    g, o = _pair(tiny_corpus, seed=7)
    g.sweep(3, mh_steps)
    o.sweep(3, mh_steps)
    assert np.array_equal(g.get_assignments(), o.get_assignments())


def test_four_step_cycle_small_config(small_corpus):
    """The cycle with four steps (the step count of the "large" configuration) has kernels of its own:
    tiles of whole documents, hot and tail words."""
    g, o = _pair(small_corpus, seed=9)
    g.sweep(2, 4)
    o.sweep(2, 4)
    assert np.array_equal(g.get_assignments(), o.get_assignments())
    _assert_same_moves(g, o, small_corpus.n_tokens, 2, 2, iters=2)
    _assert_same_counts(g, o)


def test_small_config_sweeps_counts_tables_loglik(small_corpus):
    """~2M tokens: many tiles, ragged tails, dense and sparse words, hot-word histogram path."""
    c = small_corpus
    g, o = _pair(c)
    st = g.stats()
    assert 0 < st["n_dense_words"] < c.V
    _assert_same_counts(g, o)
    _assert_same_tables(g, o)
    for sweep in range(3):
        g.sweep(1, 2)
        o.sweep(1, 2)
        zg, zo = g.get_assignments(), o.get_assignments()
        agree = float(np.mean(zg == zo))
        assert agree >= 0.999, (sweep, agree)
        assert np.array_equal(zg, zo), sweep
    _assert_same_counts(g, o)
    _assert_same_tables(g, o)
    for a, b in zip(g.loglik(), o.loglik()):
        assert a == pytest.approx(b, rel=1e-10)


def test_small_config_loglik_trajectory_50_sweeps(small_corpus):
    """Free-running 50 sweeps: log-likelihood within 0.5 % of the oracle's at every sweep."""
    c = small_corpus
    g, o = _pair(c, seed=99)
    for sweep in range(50):
        g.sweep(1, 2)
        o.sweep(1, 2)
        if sweep % 7 == 0 or sweep == 49:
            a, b = g.loglik()[0], o.loglik()[0]
            assert abs(a - b) <= 0.005 * abs(b), (sweep, a, b)
    assert float(np.mean(g.get_assignments() == o.get_assignments())) >= 0.999


def test_counts_consistent_with_own_assignments(small_corpus):
    """The library's tables equal a brute-force recount of its own z (bit exact)."""
    c = small_corpus
    g = binding.LightLDA(c.V, c.K, c.alpha, c.beta)
    g.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
    g.init(5)
    g.sweep(4, 2)
    z = g.get_assignments()
    w = c.word_ids.numpy().astype(np.int64)
    off = c.doc_offsets.numpy()
    doc = np.repeat(np.arange(off.size - 1), np.diff(off))
    assert np.array_equal(g.get_nk(), np.bincount(z, minlength=c.K))
    for which, seg, rows in ((binding.LDA_NWK, w, c.V), (binding.LDA_NDK, doc, off.size - 1)):
        ro, top, cnt = g.get_csr(which)
        key = seg * c.K + z
        uk, uc = np.unique(key, return_counts=True)
        assert np.array_equal(uk // c.K * 0 + top, uk % c.K)
        assert np.array_equal(cnt, uc)
        assert np.array_equal(ro, np.searchsorted(uk // c.K, np.arange(rows + 1)))


def test_checkpoint_and_warm_start_continue_bit_exactly(small_corpus):
    """Section 6 (fault tolerance by warm start): the assignments are the whole checkpoint.  A fresh
    context given z, the seed and the sweep counter continues exactly like the one that never stopped."""
    c = small_corpus
    a = binding.LightLDA(c.V, c.K, c.alpha, c.beta)
    a.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
    a.init(SEED)
    a.sweep(2, 2)
    z_ckpt = a.get_assignments().copy()
    a.sweep(2, 2)
    b = binding.LightLDA(c.V, c.K, c.alpha, c.beta)
    b.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
    b.set_assignments(z_ckpt, SEED, 2)
    b.sweep(2, 2)
    assert np.array_equal(a.get_assignments(), b.get_assignments())
    assert np.array_equal(a.get_nk(), b.get_nk())
    assert a.loglik() == b.loglik()


def test_sixteen_bit_import_and_export(small_corpus):
    c = small_corpus
    g, o = _pair(c, seed=4)
    g.sweep(1, 2)
    o.sweep(1, 2)
    z16 = g.get_assignments_u16()
    assert z16.dtype == np.uint16 and np.array_equal(z16.astype(np.int32), o.get_assignments())
    h = binding.LightLDA(c.V, c.K, c.alpha, c.beta)
    h.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
    h.set_assignments_u16(z16, 4, 1)
    _assert_same_counts(h, o)
    h.sweep(1, 2)
    o.sweep(1, 2)
    assert np.array_equal(h.get_assignments(), o.get_assignments())
    bad = z16.copy()
    bad[5] = c.K
    with pytest.raises(binding.LdaError) as e:
        h.set_assignments_u16(bad, 4, 1)
    assert e.value.status == binding.LDA_ERANGE
    # 32-bit topic storage has no 16-bit form
    w = binding.LightLDA(8, 70_000, 0.1, 0.1)
    w.load_corpus(np.array([0, 1, 2], np.int32), np.array([0, 3], np.int64))
    w.init(1)
    with pytest.raises(binding.LdaError) as e:
        w.get_assignments_u16()
    assert e.value.status == binding.LDA_ERANGE
    with pytest.raises(binding.LdaError) as e:
        w.set_assignments_u16(np.zeros(3, np.uint16), 1)
    assert e.value.status == binding.LDA_ERANGE


@pytest.mark.parametrize("dense_frac", [0.0, 1.0])
def test_dense_sparse_split_is_invisible(tiny_corpus, dense_frac):
    """Section 5: the hybrid row storage must not change any result."""
    c = tiny_corpus
    g, o = _pair(c, seed=11, options={"dense_frac": dense_frac, "dense_min_tf": 1})
    g.sweep(3, 2)
    o.sweep(3, 2)
    assert np.array_equal(g.get_assignments(), o.get_assignments())
    _assert_same_counts(g, o)
    _assert_same_tables(g, o)


def test_wide_topics_and_long_documents():
    """K > 65536 uses 32-bit topic storage; documents longer than a sort tile use the histogram path."""
    c = synth.generate(V=300, K=70_000, D=40, length=("fixed", 100), zipf_s=1.0, alpha=0.01, beta=0.01,
                       seed=4)
    g, o = _pair(c, seed=3)
    _assert_same_counts(g, o)
    g.sweep(2, 2)
    o.sweep(2, 2)
    assert np.array_equal(g.get_assignments(), o.get_assignments())
    _assert_same_counts(g, o)
    c2 = synth.generate(V=50, K=40, D=6, length=("fixed", 5000), zipf_s=1.0, alpha=0.1, beta=0.01, seed=5)
    g, o = _pair(c2, seed=3)
    _assert_same_counts(g, o)
    _assert_same_tables(g, o)
    g.sweep(2, 4)
    o.sweep(2, 4)
    assert np.array_equal(g.get_assignments(), o.get_assignments())
    _assert_same_counts(g, o)


def test_hot_words_with_unstaged_rows_and_odd_step_counts():
    """K above the shared-memory staging limit with words hot enough to get their own tiles, and
    step counts that end on a word-proposal or exceed one group of four.  Words of 2049 to 12 288 tokens
    are "warm" (sorted row only, staged by the accept pass), those above keep dense rows that the
    accept pass reads in place."""
    for D in (300, 1500):
        c = synth.generate(V=40, K=20_000, D=D, length=("fixed", 400), zipf_s=1.0, alpha=0.05, beta=0.01, seed=8)
        g, o = _pair(c, seed=5)
        tf = np.bincount(c.word_ids.numpy(), minlength=c.V)
        assert g.stats()["n_dense_words"] == int((tf > 12288).sum()) > 0 and int(((tf > 2048) & (tf <= 12288)).sum()) > 0
        # rows of a few hundred to more than ten thousand items: every scratch placement of the alias build
        nnz = np.diff(o.get_csr(ldaref.NWK)[0])
        assert (D > 300 or nnz.min() < 2048) and 4096 < np.sort(nnz)[-3] and nnz.max() > 12288
        _assert_same_tables(g, o)
        for mh_steps in (2, 5, 3):
            g.sweep(1, mh_steps)
            o.sweep(1, mh_steps)
            assert np.array_equal(g.get_assignments(), o.get_assignments()), mh_steps
        _assert_same_counts(g, o)
        _assert_same_tables(g, o)


@pytest.mark.parametrize("mode", [binding.PROPOSALS_WORD, binding.PROPOSALS_DOC])
def test_single_proposal_chains(tiny_corpus, small_corpus, mode):
    """Word-proposal-only and doc-proposal-only chains (Section 4.3, Fig. 11): every token agrees
    with the oracle's chain of the same schedule, at several step counts, on hot and tail words."""
    for c, sweeps in ((tiny_corpus, 3), (small_corpus, 2)):
        g, o = _pair(c, seed=11)
        g.set_proposals(mode)
        o.set_proposals(mode)
        for mh_steps in (2, 1, 5, 4):
            g.sweep(sweeps, mh_steps)
            o.sweep(sweeps, mh_steps)
            assert np.array_equal(g.get_assignments(), o.get_assignments()), mh_steps
            _assert_same_moves(g, o, c.n_tokens, mh_steps if mode == binding.PROPOSALS_WORD else 0,
                               mh_steps if mode == binding.PROPOSALS_DOC else 0, iters=sweeps)
        _assert_same_counts(g, o)
        # back to the cycle on the same context: the exchange buffers are laid out again
        g.set_proposals(binding.PROPOSALS_CYCLE)
        o.set_proposals(0)
        g.sweep(1, 2)
        o.sweep(1, 2)
        assert np.array_equal(g.get_assignments(), o.get_assignments())
        for a, b in zip(g.loglik(), o.loglik()):
            assert a == pytest.approx(b, rel=1e-10)


def test_single_proposal_chains_wide_topics_long_documents_unstaged_rows():
    c = synth.generate(V=300, K=70_000, D=40, length=("fixed", 100), zipf_s=1.0, alpha=0.01, beta=0.01,
                       seed=4)
    c2 = synth.generate(V=50, K=40, D=6, length=("fixed", 5000), zipf_s=1.0, alpha=0.1, beta=0.01, seed=5)
    c3 = synth.generate(V=40, K=20_000, D=300, length=("fixed", 400), zipf_s=1.0, alpha=0.05, beta=0.01, seed=8)
    for c in (c, c2, c3):
        for mode in (binding.PROPOSALS_WORD, binding.PROPOSALS_DOC):
            g, o = _pair(c, seed=3)
            g.set_proposals(mode)
            o.set_proposals(mode)
            g.sweep(2, 3)
            o.sweep(2, 3)
            assert np.array_equal(g.get_assignments(), o.get_assignments()), mode
            _assert_same_counts(g, o)


@pytest.mark.parametrize("block_log2", [10, 14])
def test_block_size_is_invisible(small_corpus, block_log2):
    """The block-major exchange order is a layout choice: any block size gives the same sweep."""
    c = small_corpus
    g, o = _pair(c, seed=3, options={"block_log2": block_log2})
    g.sweep(2, 4)
    o.sweep(2, 4)
    assert np.array_equal(g.get_assignments(), o.get_assignments())
    _assert_same_counts(g, o)
    for a, b in zip(g.loglik(), o.loglik()):
        assert a == pytest.approx(b, rel=1e-10)


@pytest.mark.parametrize("slices", [2, 5])
def test_vocabulary_slices_are_invisible(small_corpus, slices):
    """Pass 1 slice by slice (only one slice's alias tables in memory): same sweeps, same tables, every
    schedule and step count; less device memory."""
    c = small_corpus
    whole = binding.LightLDA(c.V, c.K, c.alpha, c.beta)
    whole.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
    g, o = _pair(c, seed=8, options={"alias_slices": slices})
    assert g.stats()["device_bytes"] < whole.stats()["device_bytes"]
    whole.close()
    _assert_same_tables(g, o)
    for mode, steps in ((binding.PROPOSALS_CYCLE, 2), (binding.PROPOSALS_CYCLE, 4),
                        (binding.PROPOSALS_WORD, 3), (binding.PROPOSALS_DOC, 2)):
        g.set_proposals(mode)
        o.set_proposals(mode)
        g.sweep(2, steps)
        o.sweep(2, steps)
        assert np.array_equal(g.get_assignments(), o.get_assignments()), (mode, steps)
        assert g.stats()["ms_alias_sparse"] < 0.05     # nothing between its two events
    _assert_same_counts(g, o)
    _assert_same_tables(g, o)
    g.sweep(1, 2)           # a sweep after the tables were read slice by slice
    o.sweep(1, 2)
    assert np.array_equal(g.get_assignments(), o.get_assignments())


def test_vocabulary_slices_large_and_big_shapes():
    """Slices on the benchmark shapes: hot words with dense rows and rows of up to K items (large x0.01),
    32-bit topics with warm words (big x0.003); more slices than some of them have words of a class."""
    for name, scale, slices in (("large", 0.01, 4), ("big", 0.003, 7)):
        c = synth.make(name, seed=0, scale=scale)
        g, o = _pair(c, seed=17, options={"alias_slices": slices})
        for sweep in range(2):
            g.sweep(1, 2)
            o.sweep(1, 2)
            assert np.array_equal(g.get_assignments(), o.get_assignments()), (name, sweep)
        assert np.array_equal(g.get_nk(), o.get_nk())
        _assert_same_tables(g, o)


def test_mid_shape_documents_and_lognormal_lengths():
    """Documents of ~330 tokens (a larger document-tile shape than the 90-token configs pick) and a
    heavy-tailed length law whose longest documents get a CTA of their own."""
    c = synth.make("mid", seed=1, scale=0.01)
    g, o = _pair(c, seed=21)
    _assert_same_counts(g, o)
    for sweep in range(2):
        g.sweep(1, 2)
        o.sweep(1, 2)
        assert np.array_equal(g.get_assignments(), o.get_assignments()), sweep
    _assert_same_counts(g, o)
    _assert_same_tables(g, o)
    c = synth.generate(V=2000, K=300, D=1500, length=("lognormal", 100, 1.2), zipf_s=1.0, alpha=0.05, beta=0.01,
                       seed=12)
    g, o = _pair(c, seed=22)
    g.sweep(2, 4)
    o.sweep(2, 4)
    assert np.array_equal(g.get_assignments(), o.get_assignments())
    _assert_same_counts(g, o)
    for a, b in zip(g.loglik(), o.loglik()):
        assert a == pytest.approx(b, rel=1e-10)


def test_large_shape_sample_against_oracle():
    """The benchmark's workload shape (V = 141 000, K = 10 000, Poisson(90) documents, Zipf 1.1) at 1 % of its
    documents: same kernels, tile shapes and hot/tail split as the full run, small enough for the oracle."""
    c = synth.make("large", seed=0, scale=0.01)
    g, o = _pair(c, seed=1234)
    g.sweep(1, 2)
    o.sweep(1, 2)
    assert np.array_equal(g.get_assignments(), o.get_assignments())
    assert np.array_equal(g.get_nk(), o.get_nk())
    g.sweep(1, 4)
    o.sweep(1, 4)
    assert np.array_equal(g.get_assignments(), o.get_assignments())
    # equal counts, so only the order of summation differs: the oracle adds ~1.5e7 lgamma terms one after
    # the other (error up to n * 2^-53 relative to the sum of magnitudes), the library in 592 partial sums
    for a, b in zip(g.loglik(), o.loglik()):
        assert a == pytest.approx(b, rel=1e-9)


def test_exact_conditional_sweep_matches_oracle(tiny_corpus, small_corpus):
    """The yardstick sweep (every token drawn from Eq. 1 under frozen counts, split as Eq. 3, integer
    masses): every token equal to the oracle's, on short and long documents, hot and tail words, and the
    state it leaves is a state the MH sweep continues from on both sides alike."""
    import os
    cores = max(1, len(os.sched_getaffinity(0)))
    long_docs = synth.generate(V=50, K=40, D=6, length=("fixed", 5000), zipf_s=1.0, alpha=0.1, beta=0.01, seed=5)
    mid = synth.make("mid", seed=1, scale=0.01)
    for c in (tiny_corpus, small_corpus, long_docs, mid):
        g, o = _pair(c, seed=17)
        g.sweep(2, 2)
        o.sweep_threads(2, 2, cores)
        for sweep in range(2):
            g.gibbs_sweep(1)
            o.gibbs_sweep(1, cores)
            assert np.array_equal(g.get_assignments(), o.get_assignments()), sweep
        assert g.stats()["sweeps_done"] == o.sweeps_done == 4
        _assert_same_counts(g, o)
        g.sweep(1, 2)
        o.sweep_threads(1, 2, cores)
        assert np.array_equal(g.get_assignments(), o.get_assignments())
        for a, b in zip(g.loglik(), o.loglik()):
            assert a == pytest.approx(b, rel=1e-10)
    # beyond its limits the entry point refuses
    w = binding.LightLDA(8, 20_000, 0.1, 0.1)
    w.load_corpus(np.array([0, 1, 2], np.int32), np.array([0, 3], np.int64))
    w.init(1)
    with pytest.raises(binding.LdaError) as e:
        w.gibbs_sweep(1)
    assert e.value.status == binding.LDA_ERANGE


def test_edge_cases():
    # empty documents, a single token, one topic, absent words
    w = np.array([3, 3, 0, 7, 7, 7], np.int32)
    off = np.array([0, 0, 2, 2, 3, 6, 6], np.int64)
    for K in (1, 2, 5):
        g = binding.LightLDA(9, K, 0.5, 0.1)
        g.load_corpus(w, off)
        g.init(1)
        o = ldaref.Oracle(9, K, 0.5, 0.1)
        o.load_corpus(w, off)
        o.init(1)
        g.sweep(3, 2)
        o.sweep(3, 2)
        assert np.array_equal(g.get_assignments(), o.get_assignments())
        _assert_same_counts(g, o)
        for a, b in zip(g.loglik(), o.loglik()):
            assert a == pytest.approx(b, rel=1e-10, abs=1e-9)
    # empty corpus
    g = binding.LightLDA(4, 3, 0.5, 0.1)
    g.load_corpus(np.zeros(0, np.int32), np.zeros(1, np.int64))
    g.init(0)
    g.sweep(2, 2)
    assert g.get_assignments().size == 0


def test_alias_slices_option_range(tiny_corpus):
    c = tiny_corpus
    for bad in (0, 2.5, 257):
        with pytest.raises(binding.LdaError):
            binding.LightLDA(c.V, c.K, c.alpha, c.beta, options={"alias_slices": bad})
    g, o = _pair(c, seed=2, options={"alias_slices": 256})     # far more slices than words with tables
    g.sweep(2, 2)
    o.sweep(2, 2)
    assert np.array_equal(g.get_assignments(), o.get_assignments())
    _assert_same_tables(g, o)


def test_error_paths():
    g = binding.LightLDA(4, 3, 0.5, 0.1)
    with pytest.raises(binding.LdaError) as e:
        g.sweep(1, 2)
    assert e.value.status == binding.LDA_ESTATE
    with pytest.raises(binding.LdaError) as e:
        g.load_corpus(np.array([0, 9], np.int32), np.array([0, 2], np.int64))
    assert e.value.status == binding.LDA_ERANGE
    with pytest.raises(binding.LdaError) as e:
        g.load_corpus(np.array([0, 1], np.int32), np.array([0, 3], np.int64))
    assert e.value.status == binding.LDA_ERANGE
    g.load_corpus(np.array([0, 1], np.int32), np.array([0, 2], np.int64))
    with pytest.raises(binding.LdaError) as e:
        g.set_assignments(np.array([0, 5], np.int32), 0)
    assert e.value.status == binding.LDA_ERANGE
    g.init(0)
    with pytest.raises(binding.LdaError) as e:
        g.sweep(1, 0)
    assert e.value.status == binding.LDA_EINVAL
    with pytest.raises(binding.LdaError) as e:
        g.set_proposals(3)
    assert e.value.status == binding.LDA_EINVAL
    g.sweep(1, 2)   # the context is still usable after the refused calls


def test_device_resident_load_matches_host_load(tiny_corpus):
    import torch
    c = tiny_corpus
    a = binding.LightLDA(c.V, c.K, c.alpha, c.beta)
    a.load_corpus(c.word_ids.cuda(), c.doc_offsets.cuda())
    a.init(9)
    b = binding.LightLDA(c.V, c.K, c.alpha, c.beta, stream=torch.cuda.current_stream().cuda_stream)
    b.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
    b.init(9)
    a.sweep(2, 2)
    b.sweep(2, 2)
    assert np.array_equal(a.get_assignments(), b.get_assignments())


def test_chunked_transfers_and_async_export(small_corpus):
    """Assignments cross the host link in chunks on the context's copy stream.  The asynchronous export
    delivers what the blocking one does, the log-likelihood may be taken while it runs, and a sweep
    called before lda_wait() is ordered after the copy."""
    import torch
    c = small_corpus
    g, o = _pair(c, seed=41, options={"copy_chunk_log2": 12})      # some 500 chunks with a ragged last one
    g.sweep(1, 2)
    o.sweep(1, 2)
    want = o.get_assignments()
    for dtype in (torch.int32, torch.int16):
        host = torch.full((g.N,), -1, dtype=dtype).pin_memory()
        g.get_assignments_async(host)
        ll = g.loglik()
        g.wait()
        assert np.array_equal(host.numpy().astype(np.int64) & 0xFFFF, want)
        assert ll[0] == pytest.approx(o.loglik()[0], rel=1e-10)
    # a sweep queued right behind the export must not disturb it, nor be disturbed by it
    host = torch.full((g.N,), -1, dtype=torch.int32).pin_memory()
    g.get_assignments_async(host)
    g.sweep(1, 2)
    o.sweep(1, 2)
    g.wait()
    assert np.array_equal(host.numpy(), want)
    assert np.array_equal(g.get_assignments(), o.get_assignments())
    # import through the chunked path, then go on
    z = o.get_assignments()
    g.set_assignments(z, 41, 2)
    o.set_assignments(z, 41, 2)
    g.sweep(1, 2)
    o.sweep(1, 2)
    assert np.array_equal(g.get_assignments(), o.get_assignments())
    _assert_same_counts(g, o)


def test_step_count_down_and_up_again(small_corpus):
    """The exchange buffers are laid out for the largest step count seen; a shorter chain afterwards uses the
    same buffers with its own record size: four steps, two, one, five, two."""
    c = small_corpus
    g, o = _pair(c, seed=23)
    for steps in (4, 2, 1, 5, 2):
        g.sweep(1, steps)
        o.sweep(1, steps)
        assert np.array_equal(g.get_assignments(), o.get_assignments()), steps
    _assert_same_counts(g, o)
