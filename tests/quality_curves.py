"""Log-likelihood per sweep of the MH sweep against the exact-conditional yardsticks (Section 7.2,
Figures 11-14 in kind: "quality per iteration").  Not a test: run by hand on a GPU machine,

    python tests/quality_curves.py --workload small --sweeps 100
    python tests/quality_curves.py --workload mid --scale 0.05 --sweeps 100

It prints one markdown table: total log-likelihood at a few sweeps for
  - the frozen MH sweep of the library with 2, 4 and 8 steps (cycle), 2 word-only, 2 doc-only steps,
  - the library's frozen exact-conditional sweep (lda_gibbs_sweep),
  - the oracle's sequential collapsed Gibbs sampler (host, one core; skipped with --no-sequential).
All chains start from the same uniform random assignment.
"""
import argparse
import os
import sys
import time

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from oracle import ldaref  # noqa: E402
from paper_1412_1576_b200 import binding, synth  # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="small")
    ap.add_argument("--scale", type=float, default=1.0)
    ap.add_argument("--sweeps", type=int, default=100)
    ap.add_argument("--seed", type=int, default=7)
    ap.add_argument("--no-sequential", action="store_true")
    a = ap.parse_args()
    c = synth.make(a.workload, seed=0, scale=a.scale)
    marks = sorted({m for m in (1, 2, 5, 10, 20, 30, 50, 75, 100, 150, 200) if m <= a.sweeps} | {a.sweeps})
    w, off = c.word_ids.numpy(), c.doc_offsets.numpy()

    def gpu_chain(step):
        g = binding.LightLDA(c.V, c.K, c.alpha, c.beta)
        g.load_corpus(w, off)
        g.init(a.seed)
        out, done = [g.loglik()[0]], 0
        for m in marks:
            step(g, m - done)
            done = m
            out.append(g.loglik()[0])
        return out

    def mh(steps, mode=binding.PROPOSALS_CYCLE):
        def step(g, n):
            g.set_proposals(mode)
            g.sweep(n, steps)
        return step

    chains = {
        "MH cycle, 2 steps": mh(2), "MH cycle, 4 steps": mh(4), "MH cycle, 8 steps": mh(8),
        "MH word-proposal only, 2 steps": mh(2, binding.PROPOSALS_WORD),
        "MH doc-proposal only, 2 steps": mh(2, binding.PROPOSALS_DOC),
        "exact conditional, frozen (lda_gibbs_sweep)": lambda g, n: g.gibbs_sweep(n),
    }
    rows = {}
    for name, step in chains.items():
        t0 = time.time()
        rows[name] = gpu_chain(step)
        print(f"# {name}: {time.time() - t0:.1f} s", file=sys.stderr)
    if not a.no_sequential:
        o = ldaref.Oracle(c.V, c.K, c.alpha, c.beta)
        o.load_corpus(w, off)
        o.init(a.seed)
        out, done = [o.loglik()[0]], 0
        t0 = time.time()
        for m in marks:
            o.gibbs_sweep_sequential(m - done)
            done = m
            out.append(o.loglik()[0])
        rows["sequential collapsed Gibbs (oracle, host)"] = out
        print(f"# sequential Gibbs: {time.time() - t0:.1f} s", file=sys.stderr)
    print(f"workload {a.workload} x{a.scale}: V={c.V} K={c.K} D={c.n_docs} N={c.n_tokens}; total log-likelihood / 1e6")
    print("| sampler | start | " + " | ".join(f"sweep {m}" for m in marks) + " |")
    print("|---|" + "---|" * (len(marks) + 1))
    for name, vals in rows.items():
        print(f"| {name} | " + " | ".join(f"{v / 1e6:.3f}" for v in vals) + " |")


if __name__ == "__main__":
    main()
