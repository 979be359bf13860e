"""Thin ctypes binding of the C ABI declared in ``include/lda_b200.h``.

Argument marshalling only: every step of the sweep runs in the library's CUDA
kernels.  The module-level functions carry the C names (``lda_create`` ...);
``LightLDA`` is a small convenience wrapper around one context.  If the shared
library is missing or a call fails, an exception is raised -- there is no
fallback path of any kind.
"""

from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

LDA_OK, LDA_EINVAL, LDA_ERANGE, LDA_ESTATE, LDA_ENOMEM, LDA_ECUDA, LDA_EINTERNAL = 0, -1, -2, -3, -4, -5, -6
LDA_NK, LDA_NWK, LDA_NDK = 0, 1, 2

EXPORTS = [
    "lda_create", "lda_set_stream", "lda_set_allocator", "lda_set_option", "lda_set_proposals", "lda_load_corpus", "lda_load_corpus_device",
    "lda_set_shard", "lda_word_counts_to_dense", "lda_word_counts_from_dense", "lda_init", "lda_set_assignments", "lda_set_assignments_u16", "lda_sweep", "lda_gibbs_sweep", "lda_loglik", "lda_get_counts",
    "lda_get_assignments", "lda_get_assignments_u16", "lda_get_assignments_async", "lda_get_assignments_u16_async", "lda_wait", "lda_get_tables", "lda_get_stats", "lda_last_error", "lda_destroy",
    "lda_dense_table_noalloc",
]


class lda_stats(C.Structure):
    _fields_ = [
        ("n_tokens", C.c_int64), ("n_docs", C.c_int64), ("nnz_wk", C.c_int64), ("nnz_dk", C.c_int64),
        ("n_dense_words", C.c_int64), ("device_bytes", C.c_int64), ("kernel_launches", C.c_int64),
        ("sweeps_done", C.c_int32), ("iters", C.c_int32),
        ("ms_alias_dense", C.c_float), ("ms_alias_sparse", C.c_float), ("ms_sample", C.c_float),
        ("ms_count_wk", C.c_float), ("ms_count_k", C.c_float), ("ms_count_dk", C.c_float),
        ("ms_total", C.c_float), ("ms_propose", C.c_float), ("ms_doc_side", C.c_float),
        ("ms_accept", C.c_float),
        ("word_proposed", C.c_int64), ("word_accepted", C.c_int64),
        ("doc_proposed", C.c_int64), ("doc_accepted", C.c_int64),
    ]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


# lda_alloc_fn / lda_free_fn of the header
ALLOC_FN = C.CFUNCTYPE(C.c_void_p, C.c_size_t, C.c_void_p)
FREE_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p)


class LdaError(RuntimeError):
    def __init__(self, status: int, what: str, msg: str = ""):
        super().__init__(f"{what} failed with status {status}" + (f": {msg}" if msg else ""))
        self.status = status


_lib = None


def library_path() -> str:
    return _build.LIB_PATH


def load_library(path: str | None = None):
    """Open the shared library (no build here: build with ``paper_1412_1576_b200.build``)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or library_path()
    if not os.path.exists(path):
        raise FileNotFoundError(
            f"{path} is missing: build it with `python -m paper_1412_1576_b200.build` "
            "(there is no CPU fallback)")
    L = C.CDLL(path)
    vp, i32, i64, u32, u64, dbl = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32, C.c_uint64, C.c_double
    L.lda_create.argtypes = [i32, i32, dbl, dbl, C.POINTER(vp)]
    L.lda_set_stream.argtypes = [vp, vp]
    L.lda_set_allocator.argtypes = [vp, ALLOC_FN, FREE_FN, vp]
    L.lda_set_option.argtypes = [vp, C.c_char_p, dbl]
    L.lda_set_proposals.argtypes = [vp, C.c_int]
    L.lda_load_corpus.argtypes = [vp, vp, i64, vp, i64]
    L.lda_load_corpus_device.argtypes = [vp, vp, i64, vp, i64]
    L.lda_init.argtypes = [vp, u64]
    L.lda_set_assignments.argtypes = [vp, vp, u64, u32]
    L.lda_set_assignments_u16.argtypes = [vp, vp, u64, u32]
    L.lda_sweep.argtypes = [vp, i32, i32]
    L.lda_gibbs_sweep.argtypes = [vp, i32]
    L.lda_set_shard.argtypes = [vp, i64, vp]
    L.lda_word_counts_to_dense.argtypes = [vp, vp]
    L.lda_word_counts_from_dense.argtypes = [vp, vp]
    L.lda_loglik.argtypes = [vp, C.POINTER(dbl), C.POINTER(dbl), C.POINTER(dbl)]
    L.lda_get_counts.argtypes = [vp, C.c_int, vp, vp, vp, i64, C.POINTER(i64)]
    L.lda_get_assignments.argtypes = [vp, vp]
    L.lda_get_assignments_u16.argtypes = [vp, vp]
    L.lda_get_assignments_async.argtypes = [vp, vp]
    L.lda_get_assignments_u16_async.argtypes = [vp, vp]
    L.lda_wait.argtypes = [vp]
    L.lda_get_tables.argtypes = [vp, vp, vp, i64, vp, vp, vp, C.POINTER(u64)]
    L.lda_get_stats.argtypes = [vp, C.POINTER(lda_stats)]
    L.lda_dense_table_noalloc.argtypes = [vp, i32, i32, dbl, vp, vp, vp, vp, vp]
    L.lda_last_error.argtypes = [vp]
    L.lda_last_error.restype = C.c_char_p
    L.lda_destroy.argtypes = [vp]
    L.lda_destroy.restype = None
    for name in EXPORTS:
        if name not in ("lda_last_error", "lda_destroy"):
            getattr(L, name).restype = C.c_int
    if path == library_path():
        _lib = L
    return L


# --- the C names, marshalling only -----------------------------------------------------------

def lda_create(V, K, alpha, beta):
    h = C.c_void_p()
    rc = load_library().lda_create(V, K, alpha, beta, C.byref(h))
    return rc, h


def lda_set_stream(h, cuda_stream):
    return load_library().lda_set_stream(h, C.c_void_p(cuda_stream))


def lda_set_allocator(h, alloc_fn, free_fn):
    """alloc_fn / free_fn: ALLOC_FN / FREE_FN objects (the caller keeps them alive), or None, None."""
    return load_library().lda_set_allocator(h, alloc_fn or ALLOC_FN(0), free_fn or FREE_FN(0), None)


def torch_caching_allocator(stream: int | None):
    """(ALLOC_FN, FREE_FN) that take the context's device memory from PyTorch's caching allocator,
    on the given stream (a raw cudaStream_t; None = the default stream)."""
    import torch
    device = torch.cuda.current_device()

    def alloc(nbytes, _user):
        try:
            return torch.cuda.caching_allocator_alloc(int(nbytes), device, stream or 0)
        except Exception:          # out of memory: the library reports LDA_ENOMEM
            return None

    def free(ptr, _user):
        try:
            if ptr:
                torch.cuda.caching_allocator_delete(ptr)
        except Exception:          # interpreter shutdown: the process's memory goes with it
            pass
    return ALLOC_FN(alloc), FREE_FN(free)


def lda_set_option(h, key, value):
    return load_library().lda_set_option(h, key.encode(), float(value))


PROPOSALS_CYCLE, PROPOSALS_WORD, PROPOSALS_DOC = 0, 1, 2


def lda_set_proposals(h, mode):
    return load_library().lda_set_proposals(h, int(mode))


def lda_load_corpus(h, word_ids, doc_offsets):
    """word_ids int32[N], doc_offsets int64[D+1]: numpy arrays (host memory)."""
    w = np.ascontiguousarray(word_ids, np.int32)
    o = np.ascontiguousarray(doc_offsets, np.int64)
    return load_library().lda_load_corpus(h, w.ctypes.data, w.size, o.ctypes.data, o.size - 1)


def lda_load_corpus_device(h, word_ids_ptr, n_tokens, doc_offsets_ptr, n_docs):
    """Raw device pointers (e.g. ``tensor.data_ptr()`` of CUDA tensors)."""
    return load_library().lda_load_corpus_device(h, C.c_void_p(word_ids_ptr), n_tokens,
                                                 C.c_void_p(doc_offsets_ptr), n_docs)


def lda_init(h, seed):
    return load_library().lda_init(h, seed)


def lda_set_assignments(h, z, seed, sweep=0):
    z = np.ascontiguousarray(z, np.int32)
    return load_library().lda_set_assignments(h, z.ctypes.data, seed, sweep)


def lda_set_assignments_ptr(h, z_host_ptr, seed, sweep=0):
    return load_library().lda_set_assignments(h, C.c_void_p(z_host_ptr), seed, sweep)


def lda_set_assignments_u16(h, z, seed, sweep=0):
    z = np.ascontiguousarray(z, np.uint16)
    return load_library().lda_set_assignments_u16(h, z.ctypes.data, seed, sweep)


def lda_set_assignments_u16_ptr(h, z_host_ptr, seed, sweep=0):
    return load_library().lda_set_assignments_u16(h, C.c_void_p(z_host_ptr), seed, sweep)


def lda_sweep(h, iters, mh_steps):
    return load_library().lda_sweep(h, iters, mh_steps)


def lda_set_shard(h, first_token, global_term_freq=None):
    tf = None if global_term_freq is None else np.ascontiguousarray(global_term_freq, np.int32)
    return load_library().lda_set_shard(h, int(first_token), None if tf is None else tf.ctypes.data)


def lda_word_counts_to_dense(h, nwk_dev_ptr):
    return load_library().lda_word_counts_to_dense(h, C.c_void_p(nwk_dev_ptr))


def lda_word_counts_from_dense(h, nwk_dev_ptr):
    return load_library().lda_word_counts_from_dense(h, C.c_void_p(nwk_dev_ptr))


def lda_gibbs_sweep(h, iters):
    return load_library().lda_gibbs_sweep(h, iters)


def lda_loglik(h):
    t, w, d = C.c_double(), C.c_double(), C.c_double()
    rc = load_library().lda_loglik(h, C.byref(t), C.byref(w), C.byref(d))
    return rc, (t.value, w.value, d.value)


def lda_get_counts(h, which, row_offsets=None, topics=None, counts=None):
    """Buffers are numpy arrays or None; returns (status, nnz)."""
    nnz = C.c_int64()
    cap = 0
    for a in (topics, counts):
        if a is not None:
            cap = a.size
    p = lambda a: None if a is None else a.ctypes.data
    rc = load_library().lda_get_counts(h, which, p(row_offsets), p(topics), p(counts), cap, C.byref(nnz))
    return rc, nnz.value


def lda_get_assignments(h, z_out):
    return load_library().lda_get_assignments(h, z_out.ctypes.data)


def lda_get_assignments_ptr(h, z_host_ptr):
    return load_library().lda_get_assignments(h, C.c_void_p(z_host_ptr))


def lda_get_assignments_u16(h, z_out):
    return load_library().lda_get_assignments_u16(h, z_out.ctypes.data)


def lda_get_assignments_u16_ptr(h, z_host_ptr):
    return load_library().lda_get_assignments_u16(h, C.c_void_p(z_host_ptr))


def lda_get_assignments_async_ptr(h, z_host_ptr):
    """Queues the export into (pinned) host memory at this address; complete after lda_wait()."""
    return load_library().lda_get_assignments_async(h, C.c_void_p(z_host_ptr))


def lda_get_assignments_u16_async_ptr(h, z_host_ptr):
    return load_library().lda_get_assignments_u16_async(h, C.c_void_p(z_host_ptr))


def lda_wait(h):
    return load_library().lda_wait(h)


def lda_get_tables(h, sp_thr32, sp_alias, mix32, dn_thr32, dn_alias):
    B = C.c_uint64()
    p = lambda a: None if a is None else a.ctypes.data
    cap = 0 if sp_thr32 is None else sp_thr32.size
    rc = load_library().lda_get_tables(h, p(sp_thr32), p(sp_alias), cap, p(mix32), p(dn_thr32),
                                       p(dn_alias), C.byref(B))
    return rc, B.value


def lda_dense_table_noalloc(n_k_ptr, K, V, beta, dn_thr32_ptr, dn_alias_ptr, dense_mass_ptr,
                            status_ptr=None, cuda_stream=None):
    """Dense smoothing table into caller-owned DEVICE buffers (raw pointers); the library
    allocates nothing.  Queued on ``cuda_stream``; returns the launch status only."""
    return load_library().lda_dense_table_noalloc(
        C.c_void_p(n_k_ptr), K, V, beta, C.c_void_p(dn_thr32_ptr), C.c_void_p(dn_alias_ptr),
        C.c_void_p(dense_mass_ptr), C.c_void_p(status_ptr) if status_ptr else None,
        C.c_void_p(cuda_stream) if cuda_stream else None)


def lda_get_stats(h):
    s = lda_stats()
    rc = load_library().lda_get_stats(h, C.byref(s))
    return rc, s


def lda_last_error(h):
    m = load_library().lda_last_error(h)
    return m.decode() if m else ""


def lda_destroy(h):
    load_library().lda_destroy(h)


# --- convenience wrapper ---------------------------------------------------------------------

class LightLDA:
    """One sampler context on the current CUDA device."""

    def __init__(self, V: int, K: int, alpha: float, beta: float, stream: int | None = None,
                 options: dict | None = None, allocator: str = "torch"):
        """allocator: "torch" takes the context's device memory from PyTorch's caching allocator (so it
        shares one pool with the caller's tensors), "cuda" leaves the library on cudaMalloc."""
        self.V, self.K, self.alpha, self.beta = V, K, alpha, beta
        rc, self._h = lda_create(V, K, alpha, beta)
        if rc:
            self._h = None
            raise LdaError(rc, "lda_create")
        self.N = self.D = 0
        if stream is not None:
            self._ck(lda_set_stream(self._h, stream), "lda_set_stream")
        self._allocator = None
        if allocator == "torch":
            self._allocator = torch_caching_allocator(stream)    # kept alive as long as the context
            self._ck(lda_set_allocator(self._h, *self._allocator), "lda_set_allocator")
        elif allocator != "cuda":
            raise ValueError("allocator must be 'torch' or 'cuda'")
        for k, val in (options or {}).items():
            self._ck(lda_set_option(self._h, k, val), f"lda_set_option({k})")

    def _ck(self, rc, what):
        if rc:
            raise LdaError(rc, what, lda_last_error(self._h))

    def close(self):
        if getattr(self, "_h", None):
            lda_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def load_corpus(self, word_ids, doc_offsets):
        """numpy / CPU tensors go through the host entry point, CUDA tensors through the device one."""
        if hasattr(word_ids, "is_cuda") and word_ids.is_cuda:
            import torch
            w = word_ids.contiguous()
            o = doc_offsets.to(device=w.device, dtype=torch.int64).contiguous()
            assert w.dtype == torch.int32
            self.N, self.D = w.numel(), o.numel() - 1
            torch.cuda.current_stream(w.device).synchronize()
            self._ck(lda_load_corpus_device(self._h, w.data_ptr(), self.N, o.data_ptr(), self.D),
                     "lda_load_corpus_device")
        else:
            w = np.ascontiguousarray(np.asarray(word_ids), np.int32)
            o = np.ascontiguousarray(np.asarray(doc_offsets), np.int64)
            self.N, self.D = w.size, o.size - 1
            self._ck(lda_load_corpus(self._h, w, o), "lda_load_corpus")

    def init(self, seed: int):
        self._ck(lda_init(self._h, seed), "lda_init")

    def set_assignments(self, z, seed: int, sweep: int = 0):
        self._ck(lda_set_assignments(self._h, z, seed, sweep), "lda_set_assignments")

    def set_assignments_u16(self, z, seed: int, sweep: int = 0):
        self._ck(lda_set_assignments_u16(self._h, z, seed, sweep), "lda_set_assignments_u16")

    def set_proposals(self, mode: int):
        """PROPOSALS_CYCLE (word, doc, word, ...), PROPOSALS_WORD or PROPOSALS_DOC (Section 4.3)."""
        self._ck(lda_set_proposals(self._h, mode), "lda_set_proposals")

    def sweep(self, iters: int, mh_steps: int):
        self._ck(lda_sweep(self._h, iters, mh_steps), "lda_sweep")

    def set_shard(self, first_token: int, global_term_freq=None):
        self._ck(lda_set_shard(self._h, first_token, global_term_freq), "lda_set_shard")

    def word_counts_to_dense(self, matrix):
        """matrix: CUDA int32 tensor of V*K elements (torch), filled with this context's n_kw."""
        self._ck(lda_word_counts_to_dense(self._h, matrix.data_ptr()), "lda_word_counts_to_dense")

    def word_counts_from_dense(self, matrix):
        self._ck(lda_word_counts_from_dense(self._h, matrix.data_ptr()), "lda_word_counts_from_dense")

    def gibbs_sweep(self, iters: int):
        """Frozen exact-conditional sweeps (yardstick for the MH sweep)."""
        self._ck(lda_gibbs_sweep(self._h, iters), "lda_gibbs_sweep")

    def loglik(self):
        rc, v = lda_loglik(self._h)
        self._ck(rc, "lda_loglik")
        return v

    def get_nk(self) -> np.ndarray:
        out = np.zeros(self.K, np.int32)
        rc, _ = lda_get_counts(self._h, LDA_NK, None, None, out)
        self._ck(rc, "lda_get_counts(NK)")
        return out

    def get_csr(self, which: int):
        rows = self.V if which == LDA_NWK else self.D
        rc, nnz = lda_get_counts(self._h, which)
        self._ck(rc, "lda_get_counts(size)")
        off = np.zeros(rows + 1, np.int64)
        top = np.zeros(max(nnz, 1), np.int32)
        cnt = np.zeros(max(nnz, 1), np.int32)
        rc, nnz = lda_get_counts(self._h, which, off, top, cnt)
        self._ck(rc, "lda_get_counts")
        return off, top[:nnz], cnt[:nnz]

    def get_assignments(self) -> np.ndarray:
        out = np.zeros(max(self.N, 1), np.int32)
        self._ck(lda_get_assignments(self._h, out), "lda_get_assignments")
        return out[:self.N]

    def get_assignments_async(self, host_tensor):
        """Starts copying the assignments into a pinned CPU tensor (int32, or uint16/int16 for 16-bit topics) and
        returns; the tensor is complete after wait().  lda_loglik and lda_get_stats may run meanwhile."""
        narrow = host_tensor.element_size() == 2
        fn = lda_get_assignments_u16_async_ptr if narrow else lda_get_assignments_async_ptr
        assert host_tensor.numel() >= self.N and host_tensor.is_contiguous() and not host_tensor.is_cuda
        self._ck(fn(self._h, host_tensor.data_ptr()), "lda_get_assignments_async")

    def wait(self):
        self._ck(lda_wait(self._h), "lda_wait")

    def get_assignments_u16(self) -> np.ndarray:
        out = np.zeros(max(self.N, 1), np.uint16)
        self._ck(lda_get_assignments_u16(self._h, out), "lda_get_assignments_u16")
        return out[:self.N]

    def get_tables(self):
        rc, nnz = lda_get_counts(self._h, LDA_NWK)
        self._ck(rc, "lda_get_counts(size)")
        thr = np.zeros(max(nnz, 1), np.uint32)
        al = np.zeros(max(nnz, 1), np.int32)
        mix = np.zeros(self.V, np.uint32)
        dthr = np.zeros(self.K, np.uint32)
        dal = np.zeros(self.K, np.int32)
        rc, B = lda_get_tables(self._h, thr, al, mix, dthr, dal)
        self._ck(rc, "lda_get_tables")
        return dict(sp_thr32=thr[:nnz], sp_alias=al[:nnz], mix32=mix, dn_thr32=dthr, dn_alias=dal,
                    dense_mass=B)

    def stats(self) -> dict:
        rc, s = lda_get_stats(self._h)
        self._ck(rc, "lda_get_stats")
        return s.as_dict()
