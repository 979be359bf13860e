#!/usr/bin/env python
"""Benchmark of the frozen-counts LightLDA sweep on B200.

    python bench.py --gpus N --steps K --warmup W [--impl reference]

A "step" is one whole sweep (alias tables, token MH kernel, count rebuild) over
a synthetic corpus of the chosen workload.  Prints ONE JSON line on rank 0.
``--impl reference`` times the CPU oracle instead (rank 0 only).
"""

from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

PHASES = ("ms_alias_dense", "ms_alias_sparse", "ms_sample", "ms_count_wk", "ms_count_k", "ms_count_dk", "ms_total",
          "ms_propose", "ms_doc_side", "ms_accept")
METRIC = "sampled tokens/sec per sweep"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large", choices=["tiny", "small", "mid", "large", "big"])
    ap.add_argument("--scale", type=float, default=1.0, help="shrink the number of documents")
    ap.add_argument("--mh-steps", type=int, default=2)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--sharded", action="store_true",
                    help="document-sharded run of ONE corpus over the ranks (one all-reduce of n_kw per sweep) "
                         "instead of independent replicas; strong scaling, off by default")
    ap.add_argument("--alias-slices", type=int, default=1,
                    help="vocabulary slices whose word-proposal tables are in memory one at a time (default 1: all)")
    ap.add_argument("--no-windows", action="store_true", help="skip the late-sweep and own-step-count windows")
    ap.add_argument("--late-sweep", type=int, default=50, help="first sweep of the late window")
    return ap.parse_args()


def hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100", "-i", str(self.gpu)],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        try:
            self.proc.terminate()
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        try:
            for ln in open(self.path):
                f = [x.strip() for x in ln.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                      "sw_power_cap"), f[5:9]):
                    if val.lower() == "active":
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


def workload_config(args):
    from paper_1412_1576_b200 import synth
    cfg = dict(synth.CONFIGS[args.workload])
    cfg["D"] = max(1, int(round(cfg["D"] * args.scale)))
    return cfg


def algorithmic_bytes_per_token(mh_steps: int, topic_bytes: int, rho_wk: float) -> dict:
    """Traffic of THIS DESIGN per token and kernel: what each kernel reads and writes once (no
    sector or line overfetch), exchange buffers between the three passes of the MH step included.
    T = topic bytes, M = steps, W = word-proposal steps, rho = nnz(n_kw) / N.  The unit is one
    token; one launch processes all N tokens.  The method's own bytes: method_bytes_per_token()."""
    T, M = topic_bytes, mh_steps
    W = (M + 1) // 2
    return {
        # token id, block-major index, one alias bin per draw, proposed topics and acceptance uniforms out
        "propose": 4 + 4 + 8 * W + T * W + 4 * W,
        # block-major index, z in, proposed topics in, gathered words out (own record, one word per
        # step, one acceptance uniform per doc step, padded to 16 bytes)
        "doc_side": 4 + T + T * W + 4 * ((1 + M + M // 2 + 3) // 4 * 4),
        # block-major index, gathered words and the word steps' uniforms in, z out in both orders,
        # n_kw row once per nonzero
        "accept": 4 + 4 * ((1 + M + M // 2 + 3) // 4 * 4) + 4 * W + 2 * T + 8.0 * rho_wk,
        "count_wk": T + 8.0 * rho_wk,
        "count_k": 8.0 * rho_wk,   # the rebuilt rows read again
        # row in, table out (split point, alias, packed bin), construction scratch out and in
        "alias_sparse": (8 + 8 + 8 + 40) * rho_wk,
    }


def method_bytes_per_token(mh_steps: int, topic_bytes: int, rho_wk: float, rho_dk: float) -> float:
    """Bytes the METHOD has to move per token and sweep, whatever the kernel design: the token's
    ids and its topic streamed in and out in both orders (8 + 3T), the document-side gathers of the
    chain (T per doc-proposal, 4 per n_kd lookup at the start topic and at every proposed one), the
    rebuild re-reading z in both orders and writing n_kd (2T + 4 rho_d), and per nonzero of n_kw
    its row entry plus the alias bin written and read (T + 20).  M = 2, T = 2: 32 + 4 rho_d + 22 rho."""
    T, M = topic_bytes, mh_steps
    return (8 + 3 * T) + (M // 2) * T + 4 * (M + 1) + 2 * T + 4.0 * rho_dk + (T + 20.0) * rho_wk


def over_ranks(dist, device, ms: float, n_tokens: float):
    """Replicas only: the job's time is the slowest rank's, its work the sum over ranks.
    Returns (max over ranks of ms, sum over ranks of n_tokens); identity without a process group."""
    if dist is None:
        return float(ms), float(n_tokens)
    import torch
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    n = torch.tensor([float(n_tokens)], device=device, dtype=torch.float64)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), float(n.item())


def run_ours(args):
    import numpy as np
    import torch
    from paper_1412_1576_b200 import binding, synth

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    cfg = workload_config(args)
    M = args.mh_steps
    # independent replicas: every rank draws its own corpus of the same shape
    t0 = time.time()
    corpus = synth.generate(seed=args.seed + rank, device="cuda", **cfg)
    torch.cuda.synchronize()
    gen_s = time.time() - t0
    N, D = corpus.n_tokens, corpus.n_docs
    stream = torch.cuda.current_stream()
    lda = binding.LightLDA(cfg["V"], cfg["K"], cfg["alpha"], cfg["beta"], stream=stream.cuda_stream,
                           options={"alias_slices": args.alias_slices} if args.alias_slices != 1 else None)
    torch.cuda.empty_cache()
    t0 = time.time()
    lda.load_corpus(corpus.word_ids, corpus.doc_offsets)
    load_s = time.time() - t0
    gen_stats = corpus.stats
    del corpus
    torch.cuda.empty_cache()
    lda.init(1234 + rank)
    lda.sweep(1, M)            # first launches of every kernel (module load), on a state that is thrown away
    lda.init(1234 + rank)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed_sweeps(n, steps):
        """n sweeps in one call between two events on the launch stream; returns (ms, stats of the call)."""
        torch.cuda.synchronize()
        ev0.record(stream)
        lda.sweep(n, steps)
        ev1.record(stream)
        torch.cuda.synchronize()
        return ev0.elapsed_time(ev1), binding.lda_get_stats(lda._h)[1]

    def window(first, n, ms, st):
        return {"sweeps": [first, first + n], "ms_per_step": ms / n, "value": N / (ms / n * 1e-3),
                "nnz_wk": st.nnz_wk, "nnz_dk": st.nnz_dk,
                "phases_ms_per_step": {k: getattr(st, k) / n for k in PHASES}}

    # the first two sweeps from the uniform random start (dense model), reported beside the main window
    windows = {}
    ms_a, st_a = timed_sweeps(2, M)
    windows["first"] = window(0, 2, ms_a, st_a)
    for _ in range(max(0, args.warmup - 2)):
        lda.sweep(1, M)
    st0 = lda.stats()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    phases = {k: 0.0 for k in PHASES}
    launches = 0
    rho_sum = 0.0
    barrier()
    ev0.record(stream)
    lda.sweep(args.steps, M)          # K sweeps in one call: nothing but the sweeps is inside the timed region
    ev1.record(stream)
    barrier()
    ms = own_ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop() if rank == 0 else None
    s = binding.lda_get_stats(lda._h)[1]   # phase times and launches summed over the K sweeps
    for k in phases:
        phases[k] = getattr(s, k)
    launches = s.kernel_launches
    accept_stats = {k: getattr(s, k) for k in ("word_proposed", "word_accepted", "doc_proposed", "doc_accepted")
                    if hasattr(s, k)}
    rho_sum = args.steps * s.nnz_wk / max(N, 1)
    rho_dk = s.nnz_dk / max(N, 1)
    ms, total_tokens = over_ranks(dist, "cuda", ms, N)
    ms_per_step = ms / args.steps
    value = total_tokens / (ms_per_step * 1e-3)
    st1 = lda.stats()
    windows["main"] = window(st0["sweeps_done"], args.steps, own_ms, s)

    # later sweeps (sparser model) and the configuration's own step count, outside the main window
    if not args.no_windows:
        done = st1["sweeps_done"]
        if done < args.late_sweep:
            lda.sweep(args.late_sweep - done, M)
            done = args.late_sweep
        ms_c, st_c = timed_sweeps(10, M)
        windows["late"] = window(done, 10, ms_c, st_c)
        own_steps = cfg.get("mh_steps", M)
        if own_steps != M:
            lda.sweep(1, own_steps)      # lays the exchange buffers out for the other step count
            ms_d, st_d = timed_sweeps(5, own_steps)
            windows[f"mh{own_steps}"] = dict(window(done + 11, 5, ms_d, st_d), mh_steps=own_steps)
            lda.sweep(1, M)
        st1 = dict(st1, sweeps_done=lda.stats()["sweeps_done"])

    # --- end to end through the host-buffer entry points -----------------------------------
    e2e = None
    if not args.no_e2e and args.e2e_steps > 0:
        # topics cross the host link in 16 bits when the library stores them so (K <= 65536)
        narrow = cfg["K"] <= 65536
        zb = 2 if narrow else 4
        z_host = torch.empty(N, dtype=torch.int16 if narrow else torch.int32).pin_memory()
        set_z = binding.lda_set_assignments_u16_ptr if narrow else binding.lda_set_assignments_ptr
        get_z = binding.lda_get_assignments_u16_ptr if narrow else binding.lda_get_assignments_ptr
        get_z_async = binding.lda_get_assignments_u16_async_ptr if narrow else binding.lda_get_assignments_async_ptr
        get_z(lda._h, z_host.data_ptr())
        # one untimed round trip first (first touch of the pinned buffer, lazy initialisations)
        rc = set_z(lda._h, z_host.data_ptr(), 1234 + rank, st1["sweeps_done"])
        assert rc == 0, binding.lda_last_error(lda._h)
        barrier()
        t0 = time.perf_counter()
        ev0.record(stream)
        ll = None
        for i in range(args.e2e_steps):
            rc = set_z(lda._h, z_host.data_ptr(), 1234 + rank, st1["sweeps_done"] + i)
            assert rc == 0, binding.lda_last_error(lda._h)
            lda.sweep(1, M)
            # the result leaves for the host while the log-likelihood of the same state is computed
            rc = get_z_async(lda._h, z_host.data_ptr())
            assert rc == 0
            ll = lda.loglik()
            lda.wait()              # z_host is complete from here on
        ev1.record(stream)
        barrier()
        e_ms = ev0.elapsed_time(ev1)
        wall_ms = (time.perf_counter() - t0) * 1e3
        e_ms = max(e_ms, wall_ms)   # host-side work between calls counts too
        e_ms, _ = over_ranks(dist, "cuda", e_ms, N)
        sfx = "_u16" if narrow else ""
        e2e = {"value": total_tokens / (e_ms / args.e2e_steps * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": zb * N, "d2h_bytes_per_step": zb * N + 24,
               "steps": args.e2e_steps, "loglik": ll[0] if ll else None,
               "what": f"lda_set_assignments{sfx}(host z) + lda_sweep(1) + lda_get_assignments{sfx}_async(host z) + lda_loglik + lda_wait"}
        del z_host

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = hbm_peak()
    topic_bytes = 4 if cfg["K"] > 65536 else 2
    rho = rho_sum / args.steps
    b_alg = algorithmic_bytes_per_token(M, topic_bytes, rho)
    per_ms = {k: phases["ms_" + k] / args.steps for k in b_alg}
    kernels = {"propose": "k_word_hot/k_word_cold (pass 1)", "doc_side": "k_doc_tile",
               "accept": "k_word_hot/k_word_cold (pass 3)", "count_wk": "n_kw rebuild kernels",
               "count_k": "k_nk_from_dense/k_nk_from_sparse", "alias_sparse": "k_alias_sparse_*"}
    top = max(per_ms, key=per_ms.get)          # the dominant kernel of the sweep, by measured time
    top_ms = per_ms[top]
    achieved = b_alg[top] * N / (top_ms * 1e-3) / 1e9 if top_ms > 0 else 0.0
    roofline = {"bound": "hbm", "kernel": kernels[top], "phase": top, "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak, "peak_kind": peak_kind, "traffic": None,
                "algorithmic_bytes_per_token": b_alg[top], "avg_launch_ms": top_ms,
                "share_of_step": top_ms / ms_per_step if ms_per_step else None}
    sweep_bytes = sum(b_alg.values())
    sweep_ms = phases["ms_total"] / args.steps
    # the method's own bytes (whatever the kernel design) and what they say about the whole sweep
    b_method = method_bytes_per_token(M, topic_bytes, rho, rho_dk)
    tokens_per_s_1gpu = N / (sweep_ms * 1e-3) if sweep_ms > 0 else 0.0
    roofline["survey_b_alg_bytes_per_token"] = b_method
    roofline["useful_frac"] = tokens_per_s_1gpu * b_method / 1e9 / peak
    roofline["useful_frac_what"] = ("tokens/s x the method's bytes per token (8 + 3T + floor(M/2) T + 4 (M+1) + 2T + "
                                    "4 rho_d + (T+20) rho, with this run's rho = nnz(n_kw)/N and rho_d = nnz(n_kd)/N) "
                                    "over the measured copy bandwidth")
    roofline["rho_wk"], roofline["rho_dk"] = rho, rho_dk
    roofline["whole_sweep"] = {
        "what": "traffic of this design (exchange buffers between the three passes included), not the method's bytes",
        "design_bytes_per_token": sweep_bytes,
        "achieved": sweep_bytes * N / (sweep_ms * 1e-3) / 1e9 if sweep_ms > 0 else 0.0,
        "frac": (sweep_bytes * N / (sweep_ms * 1e-3) / 1e9) / peak if sweep_ms > 0 else 0.0,
        "per_kernel": {k: {"ms": per_ms[k], "design_bytes_per_token": b_alg[k],
                           "frac": (b_alg[k] * N / (per_ms[k] * 1e-3) / 1e9 / peak) if per_ms[k] > 0 else None}
                       for k in b_alg}}
    prof = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(prof):
        try:
            table = json.load(open(prof))
            def per_token(entry):
                # a kernel's measured DRAM bytes per token: the part that follows the tokens plus the
                # part that follows the nonzeros of n_kw, at this run's rho
                return entry.get("dram_bytes_per_token", 0.0) + entry.get("dram_bytes_per_nnz", 0.0) * rho
            tr = table.get(top, {})
            if tr.get("workload") == args.workload and tr.get("mh_steps") == M:
                roofline["traffic"] = per_token(tr) * N
                roofline["traffic_source"] = tr.get("source")
                if "issue_active_pct" in tr:   # ncu smsp__issue_active of the same capture
                    roofline["issue_active_pct"] = tr["issue_active_pct"]
            # bytes moved by the whole sweep: measured DRAM bytes per token of every per-sweep kernel
            need = ("alias_dense", "alias_sparse", "propose", "doc_side", "accept", "count_wk", "count_k")
            have = {k: table[k] for k in need if k in table and table[k].get("workload") == args.workload
                    and table[k].get("mh_steps") == M}
            if len(have) == len(need) and sweep_ms > 0:
                moved = sum(per_token(v) for v in have.values())
                roofline["bytes_moved_per_token"] = moved
                roofline["bytes_moved_frac"] = moved * N / (sweep_ms * 1e-3) / 1e9 / peak
                roofline["bytes_moved_what"] = ("ncu dram__bytes_read.sum + dram__bytes_write.sum of every per-sweep "
                                                "kernel (profiles/traffic.json, per token) x N over the sweep time, "
                                                "over the measured copy bandwidth")
        except Exception:
            pass

    cpu = None
    if not args.no_cpu:
        cpu = cpu_baseline(args, args.cpu_seconds)

    line = {
        "metric": f"{METRIC} (mh_steps={M})", "value": value, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": f"{args.workload} LDA" + (f" x{args.scale}" if args.scale != 1.0 else ""),
                   "V": cfg["V"], "K": cfg["K"], "D": D, "n_tokens": N, "mh_steps": M,
                   "alpha": cfg["alpha"], "beta": cfg["beta"], "topic_bytes": topic_bytes,
                   "alias_slices": args.alias_slices,
                   "parallelism": "replicas only" if world > 1 else "1 GPU",
                   "l2": "inputs larger than L2" if N * 14 > 126e6 else "inputs fit in L2",
                   "sweeps_timed": [st0["sweeps_done"], st0["sweeps_done"] + args.steps],
                   "top10pct_vocab_token_share": gen_stats["top10pct_vocab_token_share"]},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline,
        "cpu_baseline": cpu, "windows": windows, "accept_counts": accept_stats,
        "phases_ms_per_step": {k: v / args.steps for k, v in phases.items()},
        "state": {"nnz_wk": st1["nnz_wk"], "nnz_dk": st1["nnz_dk"], "dense_words": st1["n_dense_words"],
                  "device_bytes": st1["device_bytes"], "generate_s": gen_s, "load_s": load_s},
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_sharded(args):
    """One corpus, its documents sharded over the ranks (paper_1412_1576_b200/sharded.py): per sweep
    every rank sweeps its documents against the shared counts, then ONE all-reduce (NCCL) sums the
    ranks' n_kw matrices.  Total work is fixed as the ranks grow: strong scaling."""
    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_1412_1576_b200 import binding, sharded, synth

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1 or "MASTER_ADDR" in os.environ:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        reduce = sharded.torch_all_reduce
    else:
        reduce = lambda m: None        # one shard: the sum over the shards is the matrix itself
    cfg = workload_config(args)
    M = args.mh_steps
    corpus = synth.generate(seed=args.seed, device="cuda", **cfg)      # the same corpus on every rank
    w = corpus.word_ids.cpu().numpy()
    off = corpus.doc_offsets.cpu().numpy()
    N = corpus.n_tokens
    del corpus
    torch.cuda.empty_cache()
    stream = torch.cuda.current_stream()
    matrix = torch.zeros(cfg["V"] * cfg["K"], dtype=torch.int32, device="cuda")
    run = sharded.ShardedSweep(binding.LightLDA(cfg["V"], cfg["K"], cfg["alpha"], cfg["beta"], stream=stream.cuda_stream),
                               matrix, all_reduce=reduce)
    d0, d1 = sharded.shard_documents(off, world, rank)
    run.load(w, off, d0, d1, sharded.term_frequencies(w, cfg["V"]))
    n_local = int(off[d1] - off[d0])
    del w
    run.init(1234)
    run.sweep(max(1, args.warmup), M)

    def barrier():
        torch.cuda.synchronize()
        if dist.is_initialized():
            dist.barrier()
        torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    barrier()
    ev0.record(stream)
    run.sweep(args.steps, M)
    ev1.record(stream)
    barrier()
    ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop() if rank == 0 else None
    if dist.is_initialized():
        t = torch.tensor([ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    word, doc = run.loglik_parts()
    if dist.is_initialized():
        t = torch.tensor([doc], device="cuda", dtype=torch.float64)
        dist.all_reduce(t)
        doc = float(t.item())
        dist.destroy_process_group()
    if rank != 0:
        return
    ms_per_step = ms / args.steps
    print(json.dumps({
        "metric": f"{METRIC} (mh_steps={M})", "value": N / (ms_per_step * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "strong", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{args.workload} LDA" + (f" x{args.scale}" if args.scale != 1.0 else ""),
                   "V": cfg["V"], "K": cfg["K"], "n_tokens": N, "tokens_on_rank_0": n_local, "mh_steps": M,
                   "parallelism": f"documents sharded over {world} rank(s), one all-reduce of n_kw "
                                  f"({cfg['V'] * cfg['K'] * 4} bytes) per sweep"},
        "clocks": clocks, "loglik": word + doc,
        "what": "lda_sweep + lda_word_counts_to_dense + all-reduce + lda_word_counts_from_dense per step"}))


def host_cores() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except Exception:
        return max(1, os.cpu_count() or 1)


def _oracle_setup(args, tokens_cap):
    """The oracle on a bounded sample of the workload: the same generator with
    fewer documents (same V, K, length law, priors)."""
    from oracle import ldaref
    from paper_1412_1576_b200 import synth
    cfg = workload_config(args)
    avg_len = cfg["length"][1]
    cfg["D"] = max(1, min(cfg["D"], int(tokens_cap / max(avg_len, 1))))
    c = synth.generate(seed=args.seed, device="cpu", **cfg)
    o = ldaref.Oracle(c.V, c.K, c.alpha, c.beta)
    o.load_corpus(c.word_ids.numpy(), c.doc_offsets.numpy())
    o.init(1234)
    return o, c


def cpu_baseline(args, seconds):
    """The oracle as it stands on the host cores: one WHOLE sweep (table build, token loop, count
    rebuild) over a bounded corpus of the workload's generator with the token loop on all cores,
    and the token loop alone on one core beside it."""
    cores = host_cores()
    M = args.mh_steps
    o, c = _oracle_setup(args, 2e6)                       # probe: how fast is this host?
    sec = o.sweep_threads(1, M, cores)
    rate = c.n_tokens / max(float(sec.sum()), 1e-6)
    o.close()
    o, c = _oracle_setup(args, min(40e6, max(2e6, rate * seconds * 0.5)))
    sec = o.sweep_threads(1, M, cores)                    # the timed sample
    whole = float(sec.sum())
    n1 = int(min(c.n_tokens, max(100_000, 1.0e6 * seconds * 0.4)))
    t0 = time.perf_counter(); o.sweep_prefix(n1, M); dt1 = time.perf_counter() - t0
    return {"value": c.n_tokens / whole, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"one whole oracle sweep (alias tables + token loop on {cores} threads + count rebuild) over "
                      f"{c.n_docs} documents ({c.n_tokens} tokens) of the same generator, mh_steps={M}",
            "phases_s": {"tables": float(sec[0]), "token_loop": float(sec[1]), "count_rebuild": float(sec[2])},
            "token_loop_only": {"value": c.n_tokens / max(float(sec[1]), 1e-9), "cores": cores},
            "one_core": {"value": n1 / dt1, "cores": 1,
                         "sample": f"token loop over the first {n1} tokens of the next sweep, tables prebuilt"}}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = host_cores()
    M = args.mh_steps
    o, c = _oracle_setup(args, 2e6)                       # probe
    sec = o.sweep_threads(1, M, cores)
    rate = c.n_tokens / max(float(sec.sum()), 1e-6)
    o.close()
    budget = 90.0 / max(1, args.steps + args.warmup)      # seconds per step
    o, c = _oracle_setup(args, min(40e6, max(2e5, rate * budget)))
    for _ in range(args.warmup):
        o.sweep_threads(1, M, cores)
    t0 = time.perf_counter()
    o.sweep_threads(args.steps, M, cores)
    dt = time.perf_counter() - t0
    value = c.n_tokens * args.steps / dt
    sample = (f"each step = one whole oracle sweep (alias tables + token loop on {cores} threads + count rebuild) over "
              f"{c.n_docs} documents ({c.n_tokens} tokens) of the same generator, mh_steps={M}")
    cfg = workload_config(args)
    line = {
        "impl": "reference", "metric": f"{METRIC} (mh_steps={M})", "value": value, "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{args.workload} LDA" + (f" x{args.scale}" if args.scale != 1.0 else ""),
                   "V": cfg["V"], "K": cfg["K"], "mh_steps": M, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    elif a.sharded:
        run_sharded(a)
    else:
        run_ours(a)
