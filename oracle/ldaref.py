"""ctypes wrapper around the CPU oracle (``lda_oracle.c``).

TEST INFRASTRUCTURE: only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this.  It compiles the C file with gcc on first use
(``oracle/_build/libldaref.so``) and shares nothing with the CUDA path.
"""

from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lda_oracle.c")
_OUT = os.path.join(_HERE, "_build", "libldaref.so")
_lock = threading.Lock()
_lib = None

NK, NWK, NDK = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle; plain -O2, no FMA contraction, no fast-math."""
    os.makedirs(os.path.dirname(_OUT), exist_ok=True)
    if force or not os.path.exists(_OUT) or os.path.getmtime(_OUT) < os.path.getmtime(_SRC):
        tmp = _OUT + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
                               "-Wall", "-Wextra", "-shared", "-fPIC", _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _OUT)
    return _OUT


def _p(dtype):
    return np.ctypeslib.ndpointer(dtype=dtype, flags="C_CONTIGUOUS")


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = C.CDLL(build())
            vp = C.c_void_p
            L.ldaref_philox4x32_10.argtypes = [_p(np.uint32), _p(np.uint32), _p(np.uint32)]
            L.ldaref_philox4x32_10.restype = None
            L.ldaref_alias_build.argtypes = [C.c_int32, _p(np.uint64), _p(np.uint32), _p(np.int32),
                                             _p(np.uint64), C.POINTER(C.c_uint64),
                                             C.POINTER(C.c_uint64), C.POINTER(C.c_int32)]
            L.ldaref_alias_draw.argtypes = [C.c_int32, _p(np.uint32), _p(np.int32), C.c_uint32,
                                            C.c_uint32]
            L.ldaref_alias_draw.restype = C.c_int32
            L.ldaref_create.argtypes = [C.c_int32, C.c_int32, C.c_double, C.c_double,
                                        C.POINTER(vp)]
            L.ldaref_destroy.argtypes = [vp]
            L.ldaref_destroy.restype = None
            L.ldaref_load_corpus.argtypes = [vp, _p(np.int32), C.c_int64, _p(np.int64), C.c_int64]
            L.ldaref_init.argtypes = [vp, C.c_uint64]
            L.ldaref_set_assignments.argtypes = [vp, _p(np.int32), C.c_uint64, C.c_uint32]
            L.ldaref_build_tables.argtypes = [vp]
            L.ldaref_sweep.argtypes = [vp, C.c_int32, C.c_int32]
            L.ldaref_sweep_threads.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, _p(np.float64)]
            L.ldaref_set_proposals.argtypes = [vp, C.c_int]
            L.ldaref_sample_tokens.argtypes = [vp, _p(np.int64), C.c_int64, C.c_int32,
                                               _p(np.int32)]
            L.ldaref_sweep_prefix.argtypes = [vp, C.c_int64, C.c_int32, _p(np.int32)]
            L.ldaref_chain.argtypes = [vp, C.c_int64, C.c_uint32, C.c_int32,
                                       C.POINTER(C.c_int32)]
            L.ldaref_word_proposal.argtypes = [vp, C.c_int32, C.c_uint32, C.c_uint32, C.c_uint32,
                                               C.POINTER(C.c_int32)]
            L.ldaref_doc_proposal.argtypes = [vp, C.c_int32, C.c_uint32, C.c_uint32,
                                              C.POINTER(C.c_int32)]
            L.ldaref_accept_ratio.argtypes = [vp, C.c_int64, C.c_int32, C.c_int32, C.c_int32,
                                              C.POINTER(C.c_double), C.POINTER(C.c_double)]
            L.ldaref_loglik.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                        C.POINTER(C.c_double)]
            L.ldaref_get_counts.argtypes = [vp, C.c_int, vp, vp, vp, C.c_int64,
                                            C.POINTER(C.c_int64)]
            L.ldaref_get_assignments.argtypes = [vp, _p(np.int32)]
            L.ldaref_get_tables.argtypes = [vp, vp, vp, C.c_int64, vp, vp, vp,
                                            C.POINTER(C.c_uint64)]
            L.ldaref_gibbs_sweep.argtypes = [vp, C.c_int32, C.c_int32]
            L.ldaref_gibbs_sweep_sequential.argtypes = [vp, C.c_int32]
            L.ldaref_gibbs_masses.argtypes = [vp, C.c_int64, _p(np.uint64), _p(np.uint64), C.c_uint32,
                                              C.POINTER(C.c_int32)]
            L.ldaref_set_shard.argtypes = [vp, C.c_int64]
            L.ldaref_word_counts_to_dense.argtypes = [vp, _p(np.int32)]
            L.ldaref_word_counts_from_dense.argtypes = [vp, _p(np.int32)]
            L.ldaref_get_moves.argtypes = [vp, _p(np.int64)]
            L.ldaref_sweeps_done.argtypes = [vp]
            L.ldaref_sweeps_done.restype = C.c_uint32
            _lib = L
    return _lib


class OracleError(RuntimeError):
    pass


def _check(rc: int, what: str):
    if rc != 0:
        raise OracleError(f"{what} failed with status {rc}")


def philox(ctr, key) -> np.ndarray:
    out = np.zeros(4, np.uint32)
    lib().ldaref_philox4x32_10(np.ascontiguousarray(ctr, np.uint32),
                               np.ascontiguousarray(key, np.uint32), out)
    return out


def alias_build(weights):
    """Returns dict(thr32, alias, thr, W, W44, shift) for integer weights."""
    wt = np.ascontiguousarray(weights, np.uint64)
    n = wt.size
    thr32 = np.zeros(n, np.uint32)
    alias = np.zeros(n, np.int32)
    thr = np.zeros(n, np.uint64)
    W, W44, sh = C.c_uint64(), C.c_uint64(), C.c_int32()
    _check(lib().ldaref_alias_build(n, wt, thr32, alias, thr, C.byref(W), C.byref(W44),
                                    C.byref(sh)), "alias_build")
    return dict(thr32=thr32, alias=alias, thr=thr, W=W.value, W44=W44.value, shift=sh.value)


def alias_draw(thr32, alias, r1: int, r2: int) -> int:
    return lib().ldaref_alias_draw(len(thr32), np.ascontiguousarray(thr32, np.uint32),
                                   np.ascontiguousarray(alias, np.int32), r1, r2)


class Oracle:
    """Same call sequence as the CUDA library: create, load_corpus, init, sweep."""

    def __init__(self, V: int, K: int, alpha: float, beta: float):
        self.V, self.K, self.alpha, self.beta = V, K, alpha, beta
        self._h = C.c_void_p()
        _check(lib().ldaref_create(V, K, alpha, beta, C.byref(self._h)), "create")
        self.N = 0
        self.D = 0

    def close(self):
        if self._h:
            lib().ldaref_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def load_corpus(self, word_ids, doc_offsets):
        w = np.ascontiguousarray(word_ids, np.int32)
        o = np.ascontiguousarray(doc_offsets, np.int64)
        self.N, self.D = w.size, o.size - 1
        _check(lib().ldaref_load_corpus(self._h, w, w.size, o, o.size - 1), "load_corpus")

    def init(self, seed: int):
        _check(lib().ldaref_init(self._h, seed), "init")

    def set_assignments(self, z, seed: int, sweep: int = 0):
        _check(lib().ldaref_set_assignments(self._h, np.ascontiguousarray(z, np.int32), seed,
                                            sweep), "set_assignments")

    def set_proposals(self, mode: int):
        """0 = cycle (word, doc, word, ...), 1 = word-proposal only, 2 = doc-proposal only."""
        _check(lib().ldaref_set_proposals(self._h, mode), "set_proposals")

    def sweep(self, iters: int, mh_steps: int):
        _check(lib().ldaref_sweep(self._h, iters, mh_steps), "sweep")

    def sweep_threads(self, iters: int, mh_steps: int, threads: int) -> np.ndarray:
        """The same sweeps with the token loop on `threads` host threads; returns the seconds spent
        in (table build, token loop, count rebuild)."""
        sec = np.zeros(3, np.float64)
        _check(lib().ldaref_sweep_threads(self._h, iters, mh_steps, threads, sec), "sweep_threads")
        return sec

    def sample_tokens(self, tokens, mh_steps: int) -> np.ndarray:
        t = np.ascontiguousarray(tokens, np.int64)
        out = np.zeros(t.size, np.int32)
        _check(lib().ldaref_sample_tokens(self._h, t, t.size, mh_steps, out), "sample_tokens")
        return out

    def sweep_prefix(self, n: int, mh_steps: int) -> np.ndarray:
        out = np.zeros(max(n, 1), np.int32)
        _check(lib().ldaref_sweep_prefix(self._h, n, mh_steps, out), "sweep_prefix")
        return out[:n]

    def chain(self, token: int, sweep: int, steps: int) -> int:
        z = C.c_int32()
        _check(lib().ldaref_chain(self._h, token, sweep, steps, C.byref(z)), "chain")
        return z.value

    def word_proposal(self, w: int, r0: int, r1: int, r2: int) -> int:
        t = C.c_int32()
        _check(lib().ldaref_word_proposal(self._h, w, r0, r1, r2, C.byref(t)), "word_proposal")
        return t.value

    def doc_proposal(self, d: int, r0: int, r1: int) -> int:
        t = C.c_int32()
        _check(lib().ldaref_doc_proposal(self._h, d, r0, r1, C.byref(t)), "doc_proposal")
        return t.value

    def accept_ratio(self, token: int, s: int, t: int, kind: int):
        num, den = C.c_double(), C.c_double()
        _check(lib().ldaref_accept_ratio(self._h, token, s, t, kind, C.byref(num), C.byref(den)),
               "accept_ratio")
        return num.value, den.value

    def loglik(self):
        t, w, d = C.c_double(), C.c_double(), C.c_double()
        _check(lib().ldaref_loglik(self._h, C.byref(t), C.byref(w), C.byref(d)), "loglik")
        return t.value, w.value, d.value

    def get_nk(self) -> np.ndarray:
        out = np.zeros(self.K, np.int32)
        nnz = C.c_int64()
        _check(lib().ldaref_get_counts(self._h, NK, None, None, out.ctypes.data, self.K,
                                       C.byref(nnz)), "get_counts(NK)")
        return out

    def get_csr(self, which: int):
        rows = self.V if which == NWK else self.D
        nnz = C.c_int64()
        _check(lib().ldaref_get_counts(self._h, which, None, None, None, 0, C.byref(nnz)),
               "get_counts(size)")
        off = np.zeros(rows + 1, np.int64)
        top = np.zeros(max(nnz.value, 1), np.int32)
        cnt = np.zeros(max(nnz.value, 1), np.int32)
        _check(lib().ldaref_get_counts(self._h, which, off.ctypes.data, top.ctypes.data,
                                       cnt.ctypes.data, nnz.value, C.byref(nnz)), "get_counts")
        return off, top[:nnz.value], cnt[:nnz.value]

    def get_assignments(self) -> np.ndarray:
        out = np.zeros(max(self.N, 1), np.int32)
        _check(lib().ldaref_get_assignments(self._h, out), "get_assignments")
        return out[:self.N]

    def get_tables(self):
        off, _, _ = self.get_csr(NWK)
        nnz = int(off[-1])
        sp_thr = np.zeros(max(nnz, 1), np.uint32)
        sp_al = np.zeros(max(nnz, 1), np.int32)
        mix = np.zeros(self.V, np.uint32)
        dthr = np.zeros(self.K, np.uint32)
        dal = np.zeros(self.K, np.int32)
        B = C.c_uint64()
        _check(lib().ldaref_get_tables(self._h, sp_thr.ctypes.data, sp_al.ctypes.data, nnz,
                                       mix.ctypes.data, dthr.ctypes.data, dal.ctypes.data,
                                       C.byref(B)), "get_tables")
        return dict(row_off=off, sp_thr32=sp_thr[:nnz], sp_alias=sp_al[:nnz], mix32=mix,
                    dn_thr32=dthr, dn_alias=dal, dense_mass=B.value)

    def gibbs_sweep(self, iters: int, threads: int = 1):
        """Frozen exact-conditional sweeps (the yardstick of the frozen MH sweep)."""
        _check(lib().ldaref_gibbs_sweep(self._h, iters, threads), "gibbs_sweep")

    def gibbs_sweep_sequential(self, iters: int):
        """Textbook collapsed Gibbs sweeps, counts updated token by token."""
        _check(lib().ldaref_gibbs_sweep_sequential(self._h, iters), "gibbs_sweep_sequential")

    def gibbs_masses(self, token: int, r0: int = 0):
        """(document-term masses, smoothing-term masses, topic picked for the random word r0) of the
        frozen exact-conditional draw of one token."""
        dm, pm = np.zeros(self.K, np.uint64), np.zeros(self.K, np.uint64)
        k = C.c_int32()
        _check(lib().ldaref_gibbs_masses(self._h, token, dm, pm, r0, C.byref(k)), "gibbs_masses")
        return dm, pm, k.value

    def set_shard(self, first_token: int, global_term_freq=None):
        """This context holds a run of documents of a larger corpus that starts at token first_token
        (the term frequencies are accepted for symmetry with the library and not needed here)."""
        _check(lib().ldaref_set_shard(self._h, first_token), "set_shard")

    def word_counts_to_dense(self, matrix: np.ndarray):
        assert matrix.dtype == np.int32 and matrix.size == self.V * self.K and matrix.flags.c_contiguous
        _check(lib().ldaref_word_counts_to_dense(self._h, matrix.reshape(-1)), "word_counts_to_dense")

    def word_counts_from_dense(self, matrix: np.ndarray):
        assert matrix.dtype == np.int32 and matrix.size == self.V * self.K and matrix.flags.c_contiguous
        _check(lib().ldaref_word_counts_from_dense(self._h, matrix.reshape(-1)), "word_counts_from_dense")

    def moves(self):
        """(word-proposal steps, doc-proposal steps) of the last sweep call that moved a chain."""
        out = np.zeros(2, np.int64)
        _check(lib().ldaref_get_moves(self._h, out), "get_moves")
        return int(out[0]), int(out[1])

    @property
    def sweeps_done(self) -> int:
        return lib().ldaref_sweeps_done(self._h)
