"""Pins for the oracle's proposals, acceptance ratios, chain, counts and
log-likelihood against what the paper's equations fix (CPU only)."""
import math

import numpy as np
import pytest
from scipy import stats

from oracle import ldaref
from paper_1412_1576_b200 import synth

SEED = 1234


def _dense_counts(c, z):
    """Brute-force count tables from assignments (Section 3, Eq. 12)."""
    w = c.word_ids.numpy()
    off = c.doc_offsets.numpy()
    D = off.size - 1
    doc = np.repeat(np.arange(D), np.diff(off))
    n_wk = np.zeros((c.V, c.K), np.int64)
    n_dk = np.zeros((D, c.K), np.int64)
    np.add.at(n_wk, (w, z), 1)
    np.add.at(n_dk, (doc, z), 1)
    return n_wk, n_dk, n_wk.sum(0), doc


def _oracle(c, seed=SEED):
    o = ldaref.Oracle(c.V, c.K, c.alpha, c.beta)
    o.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
    o.init(seed)
    return o


@pytest.fixture(scope="module")
def tiny(tiny_corpus):
    o = _oracle(tiny_corpus)
    o.sweep(3, 2)   # move away from the uniform start so counts are uneven
    z = o.get_assignments().copy()
    return tiny_corpus, o, z, _dense_counts(tiny_corpus, z)


def _toy(V=12, K=4, D=6, L=8, alpha=0.3, beta=0.2, seed=3):
    c = synth.generate(V=V, K=K, D=D, length=("fixed", L), zipf_s=None, alpha=alpha, beta=beta,
                       seed=seed)
    o = _oracle(c, seed=99)
    o.sweep(2, 2)
    z = o.get_assignments().copy()
    return c, o, z, _dense_counts(c, z)


# ---- counts -------------------------------------------------------------------

def test_counts_match_brute_force_and_invariants(tiny):
    c, o, z, (n_wk, n_dk, n_k, doc) = tiny
    assert np.array_equal(o.get_nk(), n_k)
    off, top, cnt = o.get_csr(ldaref.NWK)
    dense = np.zeros_like(n_wk)
    for w in range(c.V):
        seg = slice(off[w], off[w + 1])
        assert np.all(np.diff(top[seg]) > 0)          # ascending, no duplicates
        assert np.all(cnt[seg] > 0)
        dense[w, top[seg]] = cnt[seg]
    assert np.array_equal(dense, n_wk)
    offd, topd, cntd = o.get_csr(ldaref.NDK)
    dense_d = np.zeros_like(n_dk)
    for d in range(n_dk.shape[0]):
        seg = slice(offd[d], offd[d + 1])
        assert np.all(np.diff(topd[seg]) > 0)
        dense_d[d, topd[seg]] = cntd[seg]
    assert np.array_equal(dense_d, n_dk)
    # invariants: sum_k n_dk = n_d ; sum_d n_dk = n_k = sum_w n_wk ; sum_k n_k = N
    assert np.array_equal(dense_d.sum(1), np.diff(c.doc_offsets.numpy()))
    assert np.array_equal(dense_d.sum(0), n_k)
    assert np.array_equal(dense.sum(0), n_k)
    assert n_k.sum() == c.n_tokens


def test_init_is_uniform_and_a_function_of_seed(tiny_corpus):
    a, b, d = _oracle(tiny_corpus, 5), _oracle(tiny_corpus, 5), _oracle(tiny_corpus, 6)
    za, zb, zd = a.get_assignments(), b.get_assignments(), d.get_assignments()
    assert np.array_equal(za, zb) and not np.array_equal(za, zd)
    assert za.min() >= 0 and za.max() < tiny_corpus.K
    p = stats.chisquare(np.bincount(za, minlength=tiny_corpus.K)).pvalue
    assert p > 1e-4


# ---- proposals ------------------------------------------------------------------

def _word_proposal_pmf_from_tables(tb, w, K, row_topics):
    """Exact law of the oracle's word-proposal draw, from its stored tables."""
    def table_pmf(thr32, alias):
        n = len(thr32)
        p = np.zeros(n)
        for b in range(n):
            keep = 1.0 if alias[b] == b else thr32[b] / 2.0 ** 32
            p[b] += keep / n
            if alias[b] != b:
                p[alias[b]] += (1 - keep) / n
        return p
    lo, hi = tb["row_off"][w], tb["row_off"][w + 1]
    mix = tb["mix32"][w] / 2.0 ** 32
    pmf = (1 - mix) * table_pmf(tb["dn_thr32"], tb["dn_alias"])
    if hi > lo:
        ps = table_pmf(tb["sp_thr32"][lo:hi], tb["sp_alias"][lo:hi])
        np.add.at(pmf, row_topics[lo:hi], mix * ps)
    return pmf


def test_word_proposal_tables_give_eq6(tiny):
    c, o, z, (n_wk, n_dk, n_k, doc) = tiny
    tb = o.get_tables()
    _, top, _ = o.get_csr(ldaref.NWK)
    Vb = c.V * c.beta
    words = np.argsort(-n_wk.sum(1))[:25]
    for w in words:
        q = (n_wk[w] + c.beta) / (n_k + Vb)          # Eq. 6
        q = q / q.sum()
        pmf = _word_proposal_pmf_from_tables(tb, w, c.K, top)
        assert abs(pmf.sum() - 1) < 1e-9
        assert np.max(np.abs(pmf - q)) < 1e-7


def test_word_proposal_draws_chi_square(tiny):
    c, o, z, (n_wk, n_dk, n_k, doc) = tiny
    rng = np.random.default_rng(11)
    Vb = c.V * c.beta
    n_draw = 100_000
    for w in np.argsort(-n_wk.sum(1))[[0, 3, 40]]:
        q = (n_wk[w] + c.beta) / (n_k + Vb)
        q = q / q.sum()
        r = rng.integers(0, 2 ** 32, (n_draw, 3))
        h = np.zeros(c.K)
        for a, b, cc in r:
            h[o.word_proposal(int(w), int(a), int(b), int(cc))] += 1
        keep = q * n_draw >= 5
        obs = np.append(h[keep], h[~keep].sum())
        exp = np.append(q[keep], q[~keep].sum()) * n_draw
        if exp[-1] == 0:
            obs, exp = obs[:-1], exp[:-1]
        assert stats.chisquare(obs, exp).pvalue > 1e-4


def test_doc_proposal_draws_chi_square(tiny):
    c, o, z, (n_wk, n_dk, n_k, doc) = tiny
    rng = np.random.default_rng(12)
    n_draw = 100_000
    for d in (0, 17, 133):
        q = (n_dk[d] + c.alpha) / (n_dk[d].sum() + c.K * c.alpha)   # Eq. 9
        r = rng.integers(0, 2 ** 32, (n_draw, 2))
        h = np.zeros(c.K)
        for a, b in r:
            h[o.doc_proposal(d, int(a), int(b))] += 1
        assert stats.chisquare(h, q * n_draw).pvalue > 1e-4


def test_doc_proposal_branches():
    """r0 chooses the term: low values copy z_dj, high values draw a uniform topic."""
    c, o, z, (n_wk, n_dk, n_k, doc) = _toy()
    off = c.doc_offsets.numpy()
    d, n_d = 2, int(off[3] - off[2])
    for r1 in (0, 2 ** 31, 2 ** 32 - 1):
        j = (r1 * n_d) >> 32
        assert o.doc_proposal(d, 0, r1) == z[off[d] + j]
        assert o.doc_proposal(d, 2 ** 32 - 1, r1) == (r1 * c.K) >> 32
    # branch boundary: copy iff u*(n_d + K*alpha) < n_d
    edge = n_d / (n_d + c.K * c.alpha)
    r_lo, r_hi = int(edge * 2 ** 32) - 2, int(edge * 2 ** 32) + 2
    assert o.doc_proposal(d, r_lo, 0) == z[off[d]]
    assert o.doc_proposal(d, r_hi, 0) == 0


# ---- acceptance ratios ------------------------------------------------------------

def _target(c, n_wk, n_dk, n_k, w, d, z0):
    """Eq. 4 with the token's own count removed at z0."""
    e = np.zeros(c.K)
    e[z0] = 1
    return (n_dk[d] - e + c.alpha) * (n_wk[w] - e + c.beta) / (n_k - e + c.V * c.beta)


def test_acceptance_ratios_equal_p_q_quotients(tiny):
    c, o, z, (n_wk, n_dk, n_k, doc) = tiny
    rng = np.random.default_rng(13)
    wid = c.word_ids.numpy()
    Vb = c.V * c.beta
    for i in rng.integers(0, c.n_tokens, 300):
        w, d, z0 = wid[i], doc[i], z[i]
        p = _target(c, n_wk, n_dk, n_k, w, d, z0)
        qw = (n_wk[w] + c.beta) / (n_k + Vb)        # Eq. 6 (unnormalised)
        qd = n_dk[d] + c.alpha                      # Eq. 9 (unnormalised)
        s, t = rng.integers(0, c.K, 2)
        # the chain only visits states with p(s) > 0; keep s there
        if p[s] <= 0:
            s = z0
        for kind, q in ((0, qw), (1, qd)):
            num, den = o.accept_ratio(int(i), int(s), int(t), kind)
            want = p[t] * q[s] / (p[s] * q[t])      # Eq. 7 / Eq. 10
            assert num / den == pytest.approx(want, rel=1e-11)
            assert num >= 0 and den > 0


# ---- the chain -------------------------------------------------------------------

def _step_matrix(c, o, i, kind, prop_pmf):
    K = c.K
    P = np.zeros((K, K))
    for s in range(K):
        for t in range(K):
            if t == s:
                continue
            num, den = o.accept_ratio(i, s, t, kind)
            # accept iff u*den < num, u = r3/2^32 uniform on a 2^-32 grid
            acc = 1.0 if num >= den else num / den
            P[s, t] = prop_pmf[t] * acc
        P[s, s] = 1 - P[s].sum()
    return P


def test_chain_transition_matrices_leave_eq4_invariant():
    c, o, z, (n_wk, n_dk, n_k, doc) = _toy()
    tb = o.get_tables()
    _, top, _ = o.get_csr(ldaref.NWK)
    wid = c.word_ids.numpy()
    for i in (0, 7, 19, 33, 47):
        w, d, z0 = wid[i], doc[i], z[i]
        p = _target(c, n_wk, n_dk, n_k, w, d, z0)
        assert np.all(p > 0)       # alpha, beta > 0 and counts >= own contribution
        pi = p / p.sum()
        q_word = _word_proposal_pmf_from_tables(tb, w, c.K, top)
        q_doc = (n_dk[d] + c.alpha) / (n_dk[d].sum() + c.K * c.alpha)
        for kind, q in ((0, q_word), (1, q_doc)):
            P = _step_matrix(c, o, i, kind, q)
            assert np.all(P >= -1e-12)
            assert np.max(np.abs(pi @ P - pi)) < 1e-7
            # detailed balance of each MH kernel
            F = pi[:, None] * P
            assert np.max(np.abs(F - F.T)) < 1e-7


def test_chain_histogram_matches_gibbs_conditional():
    """Many replicas of one token's chain (different Philox streams) land on Eq. 4."""
    c, o, z, (n_wk, n_dk, n_k, doc) = _toy(V=10, K=5, D=5, L=10, seed=8)
    wid = c.word_ids.numpy()
    n_rep = 40_000
    for i in (3, 28):
        p = _target(c, n_wk, n_dk, n_k, wid[i], doc[i], z[i])
        pi = p / p.sum()
        h = np.zeros(c.K)
        for rep in range(n_rep):
            h[o.chain(i, 1000 + rep, 24)] += 1
        assert stats.chisquare(h, pi * n_rep).pvalue > 1e-4


def test_chain_with_zero_steps_keeps_state_and_one_step_is_word_proposal(tiny):
    c, o, z, _ = tiny
    wid = c.word_ids.numpy()
    key = [SEED & 0xFFFFFFFF, SEED >> 32]
    for i in (0, 5, 4242):
        assert o.chain(i, 7, 0) == z[i]
        r = ldaref.philox([i, 7, 0, 0], key)
        t = o.word_proposal(int(wid[i]), int(r[0]), int(r[1]), int(r[2]))
        got = o.chain(i, 7, 1)
        if t == z[i]:
            assert got == z[i]
        else:
            num, den = o.accept_ratio(i, int(z[i]), t, 0)
            accept = (int(r[3]) / 2.0 ** 32) * den < num
            assert got == (t if accept else z[i])


def test_single_proposal_chains_still_land_on_eq4():
    """Section 4.3: either proposal alone is a valid MH kernel for Eq. 4 (alpha, beta > 0 give
    both full support); the word-only and doc-only chains of Fig. 11 have the same target."""
    c, o, z, (n_wk, n_dk, n_k, doc) = _toy(V=10, K=5, D=5, L=10, seed=8)
    wid = c.word_ids.numpy()
    n_rep = 20_000
    i = 28
    p = _target(c, n_wk, n_dk, n_k, wid[i], doc[i], z[i])
    pi = p / p.sum()
    hists = {}
    for mode in (1, 2):
        o.set_proposals(mode)
        h = np.zeros(c.K)
        for rep in range(n_rep):
            h[o.chain(i, 5000 + rep, 32)] += 1
        hists[mode] = h
        assert stats.chisquare(h, pi * n_rep).pvalue > 1e-4
    assert not np.array_equal(hists[1], hists[2])     # different kernels, same target
    with pytest.raises(Exception):
        o.set_proposals(3)


def _by_hand(o, i, z0, wid, doc, key, sweep, kinds):
    s = int(z0)
    for m, kind in enumerate(kinds):
        r = ldaref.philox([i, sweep, m, 0], key)
        if kind == 0:
            t = o.word_proposal(int(wid[i]), int(r[0]), int(r[1]), int(r[2]))
        else:
            t = o.doc_proposal(int(doc[i]), int(r[0]), int(r[1]))
        if t == s:
            continue
        num, den = o.accept_ratio(i, s, t, kind)
        if (int(r[3]) / 2.0 ** 32) * den < num:
            s = t
    return s


def test_proposal_modes_pick_the_proposal_of_each_step(tiny):
    """Step m of a chain draws the word-proposal (Eq. 6-8) or the doc-proposal (Eq. 9-11):
    cycle = word on even m, doc on odd m; the two single-proposal modes use one kind on every m."""
    c, o, z, (_, _, _, doc) = tiny
    wid = c.word_ids.numpy()
    key = [SEED & 0xFFFFFFFF, SEED >> 32]
    differ = 0
    try:
        for i in (1, 17, 333, 4242, 5000, 6001):
            want = {}
            for mode, kinds in ((0, (0, 1, 0)), (1, (0, 0, 0)), (2, (1, 1, 1))):
                o.set_proposals(mode)
                want[mode] = _by_hand(o, i, z[i], wid, doc, key, 9, kinds)
                assert o.chain(i, 9, 3) == want[mode]
            differ += len(set(want.values())) > 1
    finally:
        o.set_proposals(0)
    assert differ > 0


def test_sweep_is_frozen_and_order_independent(tiny_corpus):
    """Sampling tokens one by one from the sweep-start state equals the sweep."""
    c = tiny_corpus
    a, b = _oracle(c, 77), _oracle(c, 77)
    a.sweep(2, 2)
    b.sweep(1, 2)
    toks = np.random.default_rng(0).permutation(c.n_tokens)[:3000]
    picked = b.sample_tokens(toks, 2)
    b.sweep(1, 2)
    assert np.array_equal(picked, b.get_assignments()[toks])
    assert np.array_equal(a.get_assignments(), b.get_assignments())
    assert a.sweeps_done == 2


def test_threaded_sweep_is_the_serial_sweep(tiny_corpus, small_corpus):
    """The entry point that shares the token loop among host threads (the benchmark's all-cores leg)
    gives the serial sweep's assignments, counts and move counters, token for token."""
    for c, sweeps in ((tiny_corpus, 3), (small_corpus, 1)):
        a, b = _oracle(c, 5), _oracle(c, 5)
        a.sweep(sweeps, 2)
        sec = b.sweep_threads(sweeps, 2, 4)
        assert sec.shape == (3,) and (sec >= 0).all()
        assert np.array_equal(a.get_assignments(), b.get_assignments())
        assert np.array_equal(a.get_nk(), b.get_nk())
        assert a.moves() == b.moves()
        assert a.loglik() == b.loglik()
        assert a.sweeps_done == b.sweeps_done == sweeps


def test_move_counters_count_the_steps_that_changed_the_state(tiny_corpus):
    """With one step per token a chain moved iff the token's topic changed; with doc-proposals
    only, nothing is booked as a word-proposal move (and the other way round)."""
    c = tiny_corpus
    o = _oracle(c, 8)
    o.sweep(2, 2)
    z0 = o.get_assignments().copy()
    o.sweep(1, 1)                       # the cycle's first step is the word-proposal
    changed = int((o.get_assignments() != z0).sum())
    assert o.moves() == (changed, 0) and changed > 0
    o.set_proposals(2)
    z0 = o.get_assignments().copy()
    o.sweep(1, 1)
    changed = int((o.get_assignments() != z0).sum())
    assert o.moves() == (0, changed) and changed > 0
    # two steps: at least as many moves as changed tokens, at most two per token
    o.set_proposals(0)
    z0 = o.get_assignments().copy()
    o.sweep(1, 2)
    w, d = o.moves()
    changed = int((o.get_assignments() != z0).sum())
    assert changed <= w + d <= 2 * c.n_tokens and w > 0 and d > 0


# ---- exact-conditional yardstick (Eq. 1 / Eq. 3) --------------------------------------------------

def _eq1_conditional(c, z, counts, i):
    """Brute-force p(z_i = k | rest) of Eq. 1 from dense counts, the token's own contribution removed."""
    n_wk, n_dk, n_k, doc = counts
    w, d, s = c.word_ids.numpy()[i], doc[i], z[i]
    own = np.zeros(c.K)
    own[s] = 1.0
    p = (n_dk[d] - own + c.alpha) * (n_wk[w] - own + c.beta) / (n_k - own + c.V * c.beta)
    return p / p.sum()


def test_gibbs_masses_are_eq1_and_the_pick_is_the_inverse_cdf(tiny):
    c, o, z, counts = tiny
    rng = np.random.default_rng(11)
    for i in rng.integers(0, c.n_tokens, size=12):
        dm, pm, _ = o.gibbs_masses(int(i))
        mass = dm.astype(object) + pm.astype(object)          # exact integers
        total = int(mass.sum())
        pmf = np.array([int(m) / total for m in mass])
        assert np.abs(pmf - _eq1_conditional(c, z, counts, i)).max() < 1e-10
        # document-term masses sit on the document's other topics only
        n_dk = counts[1][counts[3][i]].copy()
        n_dk[z[i]] -= 1
        assert np.array_equal(dm > 0, n_dk > 0)
        # inverse CDF in exact integer arithmetic: document-term topics first, then all topics
        order = [(int(m), k) for k, m in enumerate(dm)] + [(int(m), k) for k, m in enumerate(pm)]
        for r0 in [0, 1, 2 ** 31, 2 ** 32 - 1] + [int(x) for x in rng.integers(0, 2 ** 32, size=40)]:
            x, cum, want = (total * r0) >> 32, 0, None
            for m, k in order:
                cum += m
                if cum > x:
                    want = k
                    break
            assert o.gibbs_masses(int(i), r0)[2] == want
        # and its law over uniform random words is the conditional
        draws = np.array([o.gibbs_masses(int(i), int(r))[2] for r in rng.integers(0, 2 ** 32, size=4000)])
        keep = pmf * 4000 >= 5
        obs = np.bincount(draws, minlength=c.K)[keep]
        exp = pmf[keep] * obs.sum() / pmf[keep].sum()
        assert stats.chisquare(obs, exp).pvalue > 1e-4


def test_frozen_gibbs_sweep_draws_every_token_from_the_sweep_start_state(tiny_corpus):
    c = tiny_corpus
    a, b = _oracle(c, 21), _oracle(c, 21)
    a.sweep(2, 2)
    b.sweep(2, 2)
    z0 = a.get_assignments().copy()
    picks = {}
    for i in np.random.default_rng(3).integers(0, c.n_tokens, size=300):
        r = ldaref.philox([int(i), a.sweeps_done, 0, 2], [21, 0])
        picks[int(i)] = a.gibbs_masses(int(i), int(r[0]))[2]
    a.gibbs_sweep(1, 1)
    b.gibbs_sweep(1, 4)                                   # documents shared among threads: same sweep
    z1 = a.get_assignments()
    assert np.array_equal(z1, b.get_assignments()) and a.sweeps_done == 3
    assert all(z1[i] == k for i, k in picks.items())
    assert float(np.mean(z1 != z0)) > 0.2
    n_wk, n_dk, n_k, _ = _dense_counts(c, z1)
    assert np.array_equal(a.get_nk(), n_k)


def test_sequential_gibbs_first_token_follows_eq1():
    """The first token a sequential sweep redraws sees every other token at its old topic: over many
    seeds its new topic is distributed as Eq. 1 says."""
    c, o, z, counts = _toy(V=10, K=5, D=4, L=7)
    p = _eq1_conditional(c, z, counts, 0)
    draws = []
    for seed in range(6000):
        o.set_assignments(z, seed, 0)
        o.gibbs_sweep_sequential(1)
        draws.append(o.get_assignments()[0])
    obs = np.bincount(np.array(draws), minlength=c.K)
    assert stats.chisquare(obs, p * len(draws)).pvalue > 1e-4
    # counts are those of the new assignments
    z1 = o.get_assignments()
    assert np.array_equal(o.get_nk(), np.bincount(z1, minlength=c.K))


def test_yardsticks_order_on_tiny(tiny_corpus):
    """Trend only (the paper prints no number: parity unpinned): after 30 sweeps from the same start the
    sequential Gibbs sampler is ahead of the frozen exact-conditional sweep, which is ahead of (or level
    with) the frozen two-step MH sweep it is the limit of."""
    c = tiny_corpus
    seq, fro, mh = _oracle(c, 3), _oracle(c, 3), _oracle(c, 3)
    seq.gibbs_sweep_sequential(30)
    fro.gibbs_sweep(30, 4)
    mh.sweep(30, 2)
    start = _oracle(c, 3).loglik()[0]
    assert seq.loglik()[0] > fro.loglik()[0] > mh.loglik()[0] - 0.02 * abs(mh.loglik()[0]) and mh.loglik()[0] > start


# ---- log-likelihood -----------------------------------------------------------------

def _sequential_joint(c, z):
    """log p(w, z) by the chain rule of the two Polya urns (independent of the
    closed form): p(z_i | earlier z of the doc) p(w_i | earlier (w, z))."""
    wid = c.word_ids.numpy()
    off = c.doc_offsets.numpy()
    n_wk = np.zeros((c.V, c.K))
    n_k = np.zeros(c.K)
    lw = ld = 0.0
    for d in range(off.size - 1):
        n_dk = np.zeros(c.K)
        for j, i in enumerate(range(off[d], off[d + 1])):
            k, w = z[i], wid[i]
            ld += math.log((n_dk[k] + c.alpha) / (j + c.K * c.alpha))
            lw += math.log((n_wk[w, k] + c.beta) / (n_k[k] + c.V * c.beta))
            n_dk[k] += 1
            n_wk[w, k] += 1
            n_k[k] += 1
    return lw, ld


def test_loglik_equals_sequential_urn_probability(tiny):
    c, o, z, _ = tiny
    total, lw, ld = o.loglik()
    sw, sd = _sequential_joint(c, z)
    assert lw == pytest.approx(sw, rel=1e-10)
    assert ld == pytest.approx(sd, rel=1e-10)
    assert total == pytest.approx(sw + sd, rel=1e-10)


def test_loglik_is_accurate_where_its_large_sums_nearly_cancel():
    """The big-model shape (V = 1e6, K = 1e5): K*lgamma(V*beta) and sum_k lgamma(n_k + V*beta) are
    ~8e9 each and cancel to ~1e7.  The closed form, evaluated with exactly rounded sums (math.fsum
    over scipy's gammaln), pins the oracle's value to 1e-13 of the sum of magnitudes (adding the
    terms one by one onto the large ones misses that by two orders of magnitude)."""
    from scipy.special import gammaln
    c = synth.make("big", seed=3, scale=0.002)
    o = _oracle(c, seed=2)
    o.sweep_threads(1, 2, 4)
    total, lw, ld = o.loglik()
    nk = o.get_nk().astype(np.float64)
    _, _, cw = o.get_csr(ldaref.NWK)
    _, _, cd = o.get_csr(ldaref.NDK)
    nd = np.diff(c.doc_offsets.numpy()).astype(np.float64)
    V, K, D, al, be = c.V, c.K, nd.size, c.alpha, c.beta
    w_terms = [K * math.lgamma(V * be)] + list(gammaln(cw + be) - math.lgamma(be)) + list(-gammaln(nk + V * be))
    d_terms = [D * math.lgamma(K * al)] + list(gammaln(cd + al) - math.lgamma(al)) + list(-gammaln(nd + K * al))
    for got, terms in ((lw, w_terms), (ld, d_terms)):
        assert abs(got - math.fsum(terms)) <= 1e-13 * math.fsum(abs(t) for t in terms)
    assert total == lw + ld


def test_loglik_single_topic_closed_form():
    c = synth.generate(V=30, K=1, D=7, length=("fixed", 9), zipf_s=None, alpha=0.4, beta=0.05,
                       seed=2)
    o = _oracle(c)
    total, lw, ld = o.loglik()
    tf = np.bincount(c.word_ids.numpy(), minlength=c.V)
    N = c.n_tokens
    want_w = math.lgamma(c.V * c.beta) - math.lgamma(N + c.V * c.beta) + sum(
        math.lgamma(n + c.beta) - math.lgamma(c.beta) for n in tf)
    assert lw == pytest.approx(want_w, rel=1e-12)
    assert ld == pytest.approx(0.0, abs=1e-9)     # one topic: p(z) = 1


# ---- behaviour over sweeps (trend only) ------------------------------------------------

def test_loglik_rises_towards_sequential_gibbs_level(tiny_corpus):
    """The paper's claim is qualitative (cycle proposal close to Gibbs per
    iteration); no number is printed, so this checks trend only."""
    c = tiny_corpus
    o = _oracle(c, 3)
    ll0 = o.loglik()[0]
    o.sweep(100, 2)     # frozen counts and two proposals per sweep mix more slowly per sweep
    ll_mh = o.loglik()[0]
    assert ll_mh > ll0 + 0.15 * abs(ll0)
    # sequential collapsed Gibbs (Eq. 1), plain numpy
    rng = np.random.default_rng(0)
    wid = c.word_ids.numpy()
    z = ldaref.Oracle(c.V, c.K, c.alpha, c.beta)
    z.load_corpus(wid, c.doc_offsets.numpy())
    z.init(3)
    zz = z.get_assignments().copy()
    n_wk, n_dk, n_k, doc = _dense_counts(c, zz)
    n_wk, n_dk, n_k = n_wk.astype(float), n_dk.astype(float), n_k.astype(float)
    for _ in range(30):
        for i in range(c.n_tokens):
            w, d, k = wid[i], doc[i], zz[i]
            n_wk[w, k] -= 1; n_dk[d, k] -= 1; n_k[k] -= 1
            p = (n_dk[d] + c.alpha) * (n_wk[w] + c.beta) / (n_k + c.V * c.beta)
            k = rng.choice(c.K, p=p / p.sum())
            zz[i] = k
            n_wk[w, k] += 1; n_dk[d, k] += 1; n_k[k] += 1
    z.set_assignments(zz, 3)
    ll_gibbs = z.loglik()[0]
    assert abs(ll_mh - ll_gibbs) < 0.05 * abs(ll_gibbs)


def test_each_single_proposal_neglects_one_part_of_the_likelihood():
    """Section 4.3 / Fig. 11, qualitative (the paper prints no number): with few MH steps the
    word-proposal alone leaves the document part of the likelihood behind and the doc-proposal
    alone the word part; the cycle is between the two on both parts."""
    cfg = dict(synth.CONFIGS["small"])
    cfg["D"] = 500
    c = synth.generate(seed=0, **cfg)
    parts = {}
    for mode in (0, 1, 2):
        o = ldaref.Oracle(c.V, c.K, c.alpha, c.beta)
        o.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
        o.init(5)
        o.set_proposals(mode)
        o.sweep(40, 2)
        _, parts[mode, "word"], parts[mode, "doc"] = o.loglik()
    assert parts[1, "word"] > parts[0, "word"] > parts[2, "word"]
    assert parts[2, "doc"] > parts[0, "doc"] > parts[1, "doc"]
    # the neglected part is far behind, the other one only a little ahead
    assert parts[0, "word"] - parts[2, "word"] > 5 * (parts[2, "doc"] - parts[0, "doc"])


def test_set_assignments_installs_z_and_its_counts(tiny_corpus):
    """ldaref_set_assignments: the assignments become exactly the given z, every count table becomes the
    brute-force count of z, the Philox position becomes (seed, sweep) -- shown by continuing, draw for draw, a
    context that REACHED that position by sweeping -- and a topic outside [0, K) is refused."""
    c = tiny_corpus
    rng = np.random.default_rng(17)
    z = rng.integers(0, c.K, size=c.n_tokens).astype(np.int32)
    o = _oracle(c, 5)
    o.sweep(2, 2)                                  # some other state first
    o.set_assignments(z, 99, 3)
    assert np.array_equal(o.get_assignments(), z)
    n_wk, n_dk, n_k, _ = _dense_counts(c, z)
    assert np.array_equal(o.get_nk(), n_k)
    for which, dense in ((ldaref.NWK, n_wk), (ldaref.NDK, n_dk)):
        off, top, cnt = o.get_csr(which)
        rebuilt = np.zeros_like(dense)
        for r in range(dense.shape[0]):
            assert np.all(np.diff(top[off[r]:off[r + 1]]) > 0)          # topics ascending, no duplicates
            rebuilt[r, top[off[r]:off[r + 1]]] = cnt[off[r]:off[r + 1]]
        assert np.array_equal(rebuilt, dense) and int(cnt[:off[-1]].min()) >= 1
    # the counter: a context seeded 99 that has done three sweeps stands at sweep 3 of the same streams; handing
    # its assignments, seed and sweep number to another context must continue it draw for draw
    p = _oracle(c, 99)
    p.sweep(3, 2)
    zp = p.get_assignments()
    o.set_assignments(zp, 99, 3)
    o.sweep(1, 2)
    p.sweep(1, 2)
    assert np.array_equal(o.get_assignments(), p.get_assignments())
    q = _oracle(c, 5)
    q.set_assignments(zp, 99, 4)                   # another sweep number: other draws
    q.sweep(1, 2)
    assert not np.array_equal(q.get_assignments(), p.get_assignments())
    bad = z.copy()
    bad[7] = c.K
    with pytest.raises(Exception):
        o.set_assignments(bad, 1, 0)
