"""Seeded synthetic LDA corpora shaped like the paper's workloads (Table 1).

This module only produces INPUTS (word ids grouped by document).  It holds
none of the sampler's arithmetic and is the one module that both the CUDA path
and the CPU oracle's tests draw their inputs from.

Recipe (LDA generative process, Section 3, collapsed so that no K x V or
D x K matrix is ever materialised -- the big configurations have K*V = 1e11):

* document lengths: fixed / Poisson / log-normal as the configuration says;
* topics: with theta_d ~ Dirichlet(alpha) integrated out, the topics of a
  document follow a Polya urn -- token n (0-based) repeats the topic of a
  uniformly chosen earlier token of the document with probability
  n / (n + K*alpha), else draws a fresh topic uniformly from K;
* words: with phi_k ~ Dirichlet(V*beta * m) integrated out (m = base measure
  over the vocabulary), the words of a topic follow the same urn -- the n-th
  token of topic k repeats the word of an earlier token of topic k with
  probability n / (n + V*beta), else draws a fresh word from m;
* m is Zipf(s) over frequency ranks, and ranks are mapped to word ids through
  a random permutation, so word id carries no frequency information
  (the tiny configuration uses the uniform base measure).

Both urns are resolved in parallel by pointer doubling (every token points at
an earlier token of its group or at itself; follow pointers until all point at
roots), which runs on CPU or GPU with plain torch ops.  Output is
deterministic in (configuration, seed, device type).
"""

from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch

# The five workloads.  "mh_steps" is the number of individual MH proposals per
# token per sweep the workload is run with.
CONFIGS = {
    "tiny": dict(V=500, K=16, D=200, length=("fixed", 50), zipf_s=None,
                 alpha=0.1, beta=0.01, mh_steps=2),
    "small": dict(V=10_000, K=100, D=20_000, length=("poisson", 100.0), zipf_s=1.05,
                  alpha=0.5, beta=0.01, mh_steps=2),
    "mid": dict(V=100_000, K=1_000, D=300_000, length=("poisson", 330.0), zipf_s=1.05,
                alpha=0.1, beta=0.01, mh_steps=2),
    "large": dict(V=141_000, K=10_000, D=8_200_000, length=("poisson", 90.0), zipf_s=1.1,
                  alpha=0.01, beta=0.01, mh_steps=4),
    "big": dict(V=1_000_000, K=100_000, D=10_000_000, length=("lognormal", 100.0, 1.0),
                zipf_s=1.0, alpha=0.01, beta=0.01, mh_steps=2),
}


@dataclass
class Corpus:
    """A corpus in the caller's document order."""

    V: int
    K: int
    alpha: float
    beta: float
    word_ids: torch.Tensor      # int32 [N], tokens grouped by document
    doc_offsets: torch.Tensor   # int64 [D+1], doc d owns [doc_offsets[d], doc_offsets[d+1])
    stats: dict = field(default_factory=dict)

    @property
    def n_tokens(self) -> int:
        return int(self.word_ids.numel())

    @property
    def n_docs(self) -> int:
        return int(self.doc_offsets.numel()) - 1


def _resolve_urn(group_start: torch.Tensor, pos: torch.Tensor, conc: float,
                 gen: torch.Generator) -> torch.Tensor:
    """For every element return the index of the root it copies from.

    ``group_start[i]`` is the index of the first element of i's group and
    ``pos[i]`` its 0-based position inside the group.  Element i is a root
    with probability conc / (pos + conc), else it points at a uniformly chosen
    earlier element of its group; pointers are then followed to the roots.
    """
    n = pos.numel()
    dev = pos.device
    u = torch.rand(n, generator=gen, device=dev, dtype=torch.float64)
    posf = pos.to(torch.float64)
    is_root = u * (posf + conc) >= posf
    del u
    v = torch.rand(n, generator=gen, device=dev, dtype=torch.float64)
    local = torch.minimum((v * posf).to(torch.int64), torch.clamp(pos - 1, min=0))
    del v, posf
    parent = torch.where(is_root, group_start + pos, group_start + local)
    del local, is_root
    for _ in range(64):
        nxt = parent[parent]
        if torch.equal(nxt, parent):
            break
        parent = nxt
    return parent


def _lengths(kind, D: int, gen: torch.Generator, dev) -> torch.Tensor:
    if kind[0] == "fixed":
        return torch.full((D,), int(kind[1]), dtype=torch.int64, device=dev)
    if kind[0] == "poisson":
        rate = torch.full((D,), float(kind[1]), dtype=torch.float32, device=dev)
        return torch.poisson(rate, generator=gen).to(torch.int64)
    if kind[0] == "lognormal":
        mean, sigma = float(kind[1]), float(kind[2])
        mu = math.log(mean) - 0.5 * sigma * sigma
        g = torch.randn(D, generator=gen, device=dev, dtype=torch.float32)
        return torch.clamp(torch.round(torch.exp(mu + sigma * g)), min=1).to(torch.int64)
    raise ValueError(f"unknown length law {kind!r}")


def generate(V: int, K: int, D: int, length, zipf_s, alpha: float, beta: float,
             seed: int = 0, device: str = "cpu", **_unused) -> Corpus:
    """Draw a corpus from the collapsed LDA generative process described above."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(0x1DA0000 + int(seed))

    n_d = _lengths(length, D, gen, dev)
    doc_offsets = torch.zeros(D + 1, dtype=torch.int64, device=dev)
    torch.cumsum(n_d, 0, out=doc_offsets[1:])
    N = int(doc_offsets[-1].item())
    if N >= 2 ** 31:
        raise ValueError("corpus too large for 32-bit token ids")

    # --- topics: Polya urn inside each document -------------------------------
    idx = torch.arange(N, dtype=torch.int64, device=dev)
    doc_start = torch.repeat_interleave(doc_offsets[:-1], n_d)
    pos = idx - doc_start
    root = _resolve_urn(doc_start, pos, K * alpha, gen)
    del doc_start, pos
    fresh_topic = torch.randint(0, K, (N,), generator=gen, device=dev, dtype=torch.int64)
    z = fresh_topic[root]
    del fresh_topic, root

    # --- words: Polya urn inside each topic ------------------------------------
    z_sorted, order = torch.sort(z, stable=True)
    del z
    n_k = torch.bincount(z_sorted, minlength=K)
    k_start = torch.zeros(K + 1, dtype=torch.int64, device=dev)
    torch.cumsum(n_k, 0, out=k_start[1:])
    grp_start = k_start[:-1][z_sorted]
    pos = idx - grp_start
    del z_sorted, idx
    root = _resolve_urn(grp_start, pos, V * beta, gen)
    del grp_start, pos

    if zipf_s is None:
        fresh_rank = torch.randint(0, V, (N,), generator=gen, device=dev, dtype=torch.int64)
    else:
        ranks = torch.arange(1, V + 1, dtype=torch.float64, device=dev)
        cdf = torch.cumsum(ranks.pow(-float(zipf_s)), 0)
        cdf = cdf / cdf[-1]
        u = torch.rand(N, generator=gen, device=dev, dtype=torch.float64)
        fresh_rank = torch.clamp(torch.searchsorted(cdf, u), max=V - 1)
        del u, cdf, ranks
    perm = torch.randperm(V, generator=gen, device=dev)
    w_sorted = perm[fresh_rank[root]]
    del fresh_rank, root
    word_ids = torch.empty(N, dtype=torch.int32, device=dev)
    word_ids[order] = w_sorted.to(torch.int32)
    del order, w_sorted

    tf = torch.bincount(word_ids.to(torch.int64), minlength=V)
    tf_sorted, _ = torch.sort(tf, descending=True)
    top10 = int(tf_sorted[: max(1, V // 10)].sum().item())
    stats = dict(N=N, D=D, V=V, K=K, tokens_per_word=N / V, tokens_per_doc=N / max(D, 1),
                 top10pct_vocab_token_share=top10 / max(N, 1),
                 max_tf=int(tf_sorted[0].item()), words_present=int((tf > 0).sum().item()),
                 max_doc_len=int(n_d.max().item()) if D else 0)
    return Corpus(V=V, K=K, alpha=float(alpha), beta=float(beta),
                  word_ids=word_ids, doc_offsets=doc_offsets, stats=stats)


def make(name: str, seed: int = 0, device: str = "cpu", scale: float = 1.0) -> Corpus:
    """Generate one of the named workloads; ``scale`` < 1 shrinks D (same shape)."""
    cfg = dict(CONFIGS[name])
    if scale != 1.0:
        cfg["D"] = max(1, int(round(cfg["D"] * scale)))
    return generate(seed=seed, device=device, **cfg)
