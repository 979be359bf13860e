"""Document-sharded data parallelism over several contexts (Section 6 of the paper, "Parameter
Server and Data Placement": documents are partitioned over the workers, the word-topic table is
shared and the workers' updates are aggregated after sampling).

One process (one GPU) holds one shard: a run of consecutive documents.  Its n_kd never leaves it.
n_kw travels as a dense V x K int32 matrix: every shard writes its own counts, ONE all-reduce (sum)
per sweep adds them up -- NCCL over NVLink when the ranks are GPUs -- and every shard rebuilds its
rows, its dense rows and n_k from the sum.  Because the counts are frozen during a sweep and the
Philox token key is the token's index in the WHOLE corpus, a sharded run produces exactly the
assignments of one context holding all the documents, whatever the number of shards.

This module is orchestration only (which call follows which, and the collective); every step of
the sweep runs in the library's kernels.  The `engine` is a context object with the library's
method names (``binding.LightLDA``); any object with the same methods can stand in for it.
"""

from __future__ import annotations

import numpy as np


def shard_documents(doc_offsets, world: int, rank: int):
    """Document range [d0, d1) of shard `rank` out of `world`: consecutive documents, cut where the
    running token count passes rank/world of the total (so shards hold about equally many tokens)."""
    off = np.asarray(doc_offsets, dtype=np.int64)
    n_docs, n_tokens = off.size - 1, int(off[-1])
    cuts = [int(np.searchsorted(off, n_tokens * r / world, side="left")) for r in range(world + 1)]
    cuts[0], cuts[-1] = 0, n_docs
    for r in range(1, world + 1):
        cuts[r] = max(cuts[r], cuts[r - 1])
    return cuts[rank], cuts[rank + 1]


def term_frequencies(word_ids, V: int) -> np.ndarray:
    """Tokens per word over the whole corpus: what ``lda_set_shard`` sizes the n_kw rows with."""
    return np.bincount(np.asarray(word_ids), minlength=V).astype(np.int32)


def torch_all_reduce(matrix):
    """Sum `matrix` (a torch tensor, or a numpy array whose memory a torch tensor can share) over
    the default process group, in place."""
    import torch
    import torch.distributed as dist
    t = matrix if isinstance(matrix, torch.Tensor) else torch.from_numpy(matrix)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)


class ShardedSweep:
    """One shard's side of a document-sharded run.

    engine      context with set_shard / load_corpus / init / sweep / word_counts_to_dense /
                word_counts_from_dense / loglik
    matrix      the exchange buffer: V*K int32 (a CUDA tensor for the library; whatever the engine's
                word_counts_to_dense / _from_dense take)
    all_reduce  callable(matrix): sums the buffer over all shards in place
    """

    def __init__(self, engine, matrix, all_reduce=torch_all_reduce):
        self.engine, self.matrix, self.all_reduce = engine, matrix, all_reduce

    def load(self, word_ids, doc_offsets, d0: int, d1: int, global_term_freq):
        """Loads documents [d0, d1) of the corpus given whole (word_ids, doc_offsets in host memory)."""
        off = np.asarray(doc_offsets, dtype=np.int64)
        first = int(off[d0])
        self.engine.set_shard(first, global_term_freq)
        self.engine.load_corpus(np.asarray(word_ids)[first:int(off[d1])], off[d0:d1 + 1] - first)
        self.first_token = first

    def exchange(self):
        """Own counts out, sum over the shards, summed counts in: the one collective of a sweep."""
        self.engine.word_counts_to_dense(self.matrix)
        self.all_reduce(self.matrix)
        self.engine.word_counts_from_dense(self.matrix)

    def init(self, seed: int):
        self.engine.init(seed)
        self.exchange()

    def sweep(self, iters: int, mh_steps: int):
        for _ in range(iters):
            self.engine.sweep(1, mh_steps)
            self.exchange()

    def loglik_parts(self):
        """(word part of the shared counts, document part of this shard's documents); the corpus'
        log-likelihood is the word part once plus the document parts of all shards."""
        _, word, doc = self.engine.loglik()
        return word, doc
