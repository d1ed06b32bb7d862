#!/usr/bin/env python
"""Benchmark of the GPU-resident retrieval path (stages 1-5 behind chimera_search).

A step is one chimera_search call over one batch of synthetic queries.  The headline workload is the Large corpus
(8.8M documents, ~600M tokens, 262,144 centroids, 2-bit residual codes; nprobe 4, n_prune 4096, k 100), the largest
configuration that fits one GPU: `value` is queries per second at batch 256 with the queries already on the device;
`e2e` is the same through chimera_search_host with pinned host buffers (host->device and device->host copies inside
the timed region); `qps_batch1` follows the paper's protocol of one synchronised query at a time.  Unless --config
names a single workload, the same line carries, under `configs`, a shorter measurement of every other workload (Tiny,
Mid, the four long-document variants) and of the two paper pipelines (partial-score refinement, RaBitQ 1-bit codes).

The path does not shard: with --gpus N every rank runs an independent replica (one process per GPU; the ranks are
started here when the script is not already running under torchrun).  --sharded times the document-sharded search.

`--impl reference` times the CPU oracle (as it stands, one thread) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from synth import CONFIGS, make_corpus, make_queries  # noqa: E402

UNIT = "queries/s"
HEADLINE = "large"
DTYPE = "int32 fixed point (stages 1-3) + f32 (stage 4)"
TARGET = 0.60          # the task's target for the code-scan stages: 60 % of HBM peak


def metric_name(cfg, batch):
    return "QPS at batch %d (%s corpus, nprobe %d, n_prune %d, k %d)" % (batch, cfg.name.capitalize(), cfg.nprobe,
                                                                         cfg.n_prune, cfg.k)


def candidate_capacity(index, q, nq, P, n_prune, k):
    """max_candidates for a workload: all documents for small corpora, else 1.25x the largest candidate count seen on
    a few probe queries (bounds the workspace on corpora with millions of documents)."""
    if index.N <= 1_000_000:
        return 0
    nb = min(8, q.shape[0])
    taps = index.alloc_taps(nb, nq, P, n_prune, table=False, ci=False)
    index.search(q[:nb].contiguous(), P, n_prune, k, taps=taps)
    assert index.status() == 0
    worst = int(taps.n_cand.max())
    del taps
    index._ws = None
    torch.cuda.empty_cache()
    return min(index.N, (int(worst * 1.25) + 1023) // 1024 * 1024)


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def measured_int8_tops():
    """Dense int8 tensor peak: the measured bf16 burst figure x the nominal 2:1 int8:bf16 ratio (TOP/s)."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return 2.0 * float(json.load(f)["bf16_tflops"]), "measured bf16 x 2"
    except Exception:
        return 2.0 * 1590.0, "fallback bf16 x 2"


def isolated_int8_mma_tops():
    """TOP/s of a back-to-back loop of tcgen05.mma kind::i8 instructions (M 128, N 256, K 32) on all SMs, from the
    library's own microbenchmark when its binary has been built (build.build_microbench); None otherwise.  Reported
    beside the stage-1 roofline entry as context: the entry's peak stays the measured bf16 rate x 2."""
    exe = os.path.join(ROOT, "paper_2608_23553_b200", "build", "mma_rate")
    if not os.path.exists(exe):
        return None
    try:
        out = subprocess.run([exe], capture_output=True, text=True, timeout=60).stdout
        for line in out.splitlines():
            if line.startswith("N=256 A in TMEM") and "TOP/s" in line:
                return float(line.split("ms,")[1].split("TOP/s")[0])
    except Exception:
        pass
    return None


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the dominant kernel, from stored ncu
# captures on small cases (a full-size launch is too large to capture; the profile named beside each figure gives the
# command).  The stage-3 bound scan reads each query's 8-bit table once (batch x K x q_len bytes) and otherwise moves
# a fixed number of bytes per algorithmic byte (centroid ids, ranges, ids, bounds), so a full-size launch is
# ratio x algorithmic bytes + batch x K x q_len.
NCU_CI_DRAM_PER_ALGORITHMIC_BYTE = {
    "large": (1.243, "profiles/ncu_ci_coarse_large_slice.md (Large recipe, 1M documents, batch 16)"),
    None: (0.939, "profiles/ncu_ci_coarse_mid.md (Mid corpus, batch 8)"),
}
NCU_PARTIAL_DRAM_PER_QUERY = (1527e6 / 64.0, "profiles/ncu_partial_score_mid.md (Mid corpus, batch 64; bytes per query)")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows = []
        self.proc = None
        self.gpu = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
            time.sleep(0.15)                      # let the first sample arrive before the timed region starts
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            parts = [p.strip() for p in r.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def whole_job_qps(local_ms: float, queries_per_rank: int, dist=None, device="cpu"):
    """(QPS over all ranks, slowest rank's milliseconds): every rank ran `queries_per_rank` queries on its own replica;
    the job takes as long as its slowest rank."""
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    world = 1
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        world = dist.get_world_size()
    ms = float(t.item())
    return world * queries_per_rank / (ms / 1e3), ms


def build_workload(cfg, device, rabitq=False):
    t0 = time.time()
    corp = make_corpus(cfg, device=device, rabitq=rabitq)
    q = make_queries(cfg, device=device)
    torch.cuda.synchronize() if device.type == "cuda" else None
    return corp, q, time.time() - t0


def oracle_index(corp, cfg):
    import oracle
    return oracle.make_index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)


def time_oracle(oix, q_np, cfg, budget_s, min_q, max_q):
    """Runs the oracle pipeline on queries 0.. until the time budget is used; returns (queries, seconds)."""
    import oracle
    n, t0 = 0, time.perf_counter()
    while n < max_q and (n < min_q or time.perf_counter() - t0 < budget_s):
        oracle.pipeline(q_np[n % q_np.shape[0]], oix, cfg.nprobe, cfg.n_prune, cfg.k)
        n += 1
    return n, time.perf_counter() - t0


def host_cpu():
    """(logical cores of the host, CPU model name)."""
    model = "unknown"
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    return os.cpu_count() or 1, model


def run_reference(args, cfg, rank, world):
    """The CPU oracle as the reference arm: rank 0 only; a step is one query (a bounded sample of a batch)."""
    if rank != 0:
        return
    device = torch.device("cuda:0") if torch.cuda.is_available() else torch.device("cpu")
    corp, q, _ = build_workload(cfg, device)
    oix = oracle_index(corp, cfg)
    q_np = q.cpu().numpy()
    del corp
    import oracle
    for s in range(args.warmup):
        oracle.pipeline(q_np[s % len(q_np)], oix, cfg.nprobe, cfg.n_prune, cfg.k)
    t0 = time.perf_counter()
    for s in range(args.steps):
        oracle.pipeline(q_np[(args.warmup + s) % len(q_np)], oix, cfg.nprobe, cfg.n_prune, cfg.k)
    dt = time.perf_counter() - t0
    qps = args.steps / dt
    cores, model = host_cpu()
    sample = "1 query per step (of the %d-query batch), %d steps, single thread" % (args.batch, args.steps)
    print(json.dumps({
        "impl": "reference", "metric": metric_name(cfg, args.batch), "value": qps, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int64+f64", "data": "synthetic",
        "config": {"workload": cfg.name, "batch": 1, "sample": sample},
        "cpu_baseline": {"value": qps, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
                         "host_cores": cores, "host_cpu": model},
        "e2e": {"value": qps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def brute_force_maxsim(centroids, cids, codes, doclens, nbits, res_lo, res_hi, q, q_group=64, chunk_tokens=1 << 18):
    """Exhaustive MaxSim (Definition 1) of EVERY document for every query, written out from the definition with
    plain torch operations: the ground truth of the recall sweeps.  It shares nothing with the library (no call into
    it, none of its kernels or layouts) and is itself compared with the CPU oracle's exhaustive scores in the GPU tests.

    score(q, d) = sum_i max_{t in d} <q_i, c_cid(t) + r(code_t)>, computed per token as <q_i, c> + <q_i, r>:
      * <q_i, c> for all centroids: one fp32 matmul (TF32 off);
      * <q_i, r>: the decoded residual levels are exact in bfloat16 and q_i is split exactly into three bfloat16
        terms (8 + 8 + 8 significant bits), so a bf16 matmul with fp32 accumulation over the three terms loses
        nothing but fp32 summation rounding (~1e-7 relative);
      * max over a document's tokens (segment maximum), then the sum over query tokens in fp32.
    Returns scores [n_queries, n_docs] float32 on q's device."""
    dev = q.device
    Bq, nq, D = q.shape
    N = doclens.numel()
    per, mask = 8 // nbits, (1 << nbits) - 1
    delta = (res_hi - res_lo) / (1 << nbits)
    levels = torch.tensor([res_lo + (u + 0.5) * delta for u in range(1 << nbits)], dtype=torch.float32, device=dev)
    assert torch.equal(levels.bfloat16().float(), levels), "residual levels must be exact in bfloat16"
    shifts = torch.arange(per, device=dev, dtype=torch.int32) * nbits
    lens = doclens.to(torch.int64)
    off = torch.cat([torch.zeros(1, dtype=torch.int64, device=dev), torch.cumsum(lens, 0)]).cpu().numpy()
    # document chunks of at most chunk_tokens tokens (at least one document each)
    bounds, d0 = [], 0
    while d0 < N:
        d1 = int(np.searchsorted(off, off[d0] + chunk_tokens, side="right")) - 1
        d1 = min(max(d1, d0 + 1), N)
        bounds.append((d0, d1))
        d0 = d1
    scores = torch.empty(Bq, N, dtype=torch.float32, device=dev)
    tf32 = torch.backends.cuda.matmul.allow_tf32
    red = torch.backends.cuda.matmul.allow_bf16_reduced_precision_reduction
    torch.backends.cuda.matmul.allow_tf32 = False
    torch.backends.cuda.matmul.allow_bf16_reduced_precision_reduction = False
    try:
        cent = centroids.to(torch.float32)
        for g0 in range(0, Bq, q_group):
            qg = q[g0:g0 + q_group].reshape(-1, D).to(torch.float32)            # [cols, D]
            G = qg.shape[0] // nq
            s_cent = cent @ qg.t()                                               # [K, cols]  <q_i, c>
            hi = qg.bfloat16()
            rem = qg - hi.float()
            mid = rem.bfloat16()
            low = (rem - mid.float()).bfloat16()
            assert torch.equal(hi.float() + mid.float() + low.float(), qg)
            qcat = torch.cat([hi, mid, low], dim=1).t().contiguous()              # [3 D, cols]
            for a, b in bounds:
                t0, t1 = int(off[a]), int(off[b])
                u = ((codes[t0:t1].to(torch.int32)[:, :, None] >> shifts) & mask).reshape(t1 - t0, D)
                r = levels[u.long()].bfloat16()
                if dev.type == "cuda":
                    val = torch.mm(r.repeat(1, 3), qcat, out_dtype=torch.float32)    # [tokens, cols]  <q_i, r>
                else:                                  # CPU (tests of this function's logic): the same sum in fp32
                    val = r.float().repeat(1, 3) @ qcat.float()
                val += s_cent[cids[t0:t1].long()]
                best = torch.segment_reduce(val, "max", lengths=lens[a:b], axis=0, unsafe=True)   # [docs, cols]
                scores[g0:g0 + G, a:b] = best.view(b - a, G, nq).sum(dim=2).t()
            del s_cent
    finally:
        torch.backends.cuda.matmul.allow_tf32 = tf32
        torch.backends.cuda.matmul.allow_bf16_reduced_precision_reduction = red
    return scores


def exhaustive_truth(corp, cfg, q, k_max):
    """Ground truth for Recall@k (Definition 3): the k_max best documents per query by exhaustive MaxSim over the
    decoded corpus, from brute_force_maxsim (ties: smaller id)."""
    scores = brute_force_maxsim(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi, q)
    top = torch.topk(scores, k_max, dim=1)
    return top.indices.to(torch.int32), top.values


def run_sweep(args, cfg, pkg, index, corp, q):
    """QPS (batch `--batch`) and Recall@k (Def. 3, against exhaustive MaxSim over the decoded corpus, on the first
    `--sweep-queries` queries) for nprobe x n_prune x k.  Prints one JSON line per point."""
    dev = q.device
    B, nq = args.batch, cfg.q_len
    nrec = min(args.sweep_queries, q.shape[0])
    qrec = q[:nrec].contiguous()
    t0 = time.time()
    truth_ids, _ = exhaustive_truth(corp, cfg, qrec, 1000)
    torch.cuda.synchronize()
    truth_s = time.time() - t0
    n_batches = max(1, min(3, q.shape[0] // B))
    batches = q[:n_batches * B].view(n_batches, B, nq, cfg.dim).contiguous()
    print(json.dumps({"sweep": cfg.name, "batch": B, "recall_queries": nrec, "ground_truth": "brute_force_maxsim "
                      "(plain torch, independent of the library; checked against the CPU oracle in the GPU tests), "
                      "top-1000 per query", "ground_truth_s": round(truth_s, 1)}))
    for P in (1, 2, 4, 8, 16, 32):
        if P > index.K:
            continue
        maxc = candidate_capacity(index, q, nq, P, 256, 10)
        for n_prune in (256, 1024, 4096, 16384):
            for k in (10, 100, 1000):
                out = (torch.empty(B, k, dtype=torch.int32, device=dev), torch.empty(B, k, dtype=torch.float32, device=dev))
                point = {"nprobe": P, "n_prune": n_prune, "k": k, "max_candidates": maxc}
                for mode, kw in (("", {}), ("partial_", {"partial": True}), ("rabitq_", {"rabitq": True})):
                    index.search(batches[0], P, n_prune, k, max_candidates=maxc, out=out, **kw)
                    torch.cuda.synchronize()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    for s in range(args.steps):
                        index.search(batches[s % n_batches], P, n_prune, k, max_candidates=maxc, out=out, **kw)
                    e1.record()
                    torch.cuda.synchronize()
                    ms = e0.elapsed_time(e1) / args.steps
                    assert index.status() == 0
                    ids, _ = index.search(qrec, P, n_prune, k, max_candidates=maxc, **kw)
                    hits = (ids[:, :, None] == truth_ids[:, None, :k]).any(dim=2).sum(dim=1).float()
                    # how many of the ground-truth top-10 are among the k returned (the use of a GPU filter stage)
                    top10 = (truth_ids[:, :10, None] == ids[:, None, :]).any(dim=2).sum(dim=1).float()
                    point.update({mode + "qps": B / (ms * 1e-3), mode + "ms_per_step": ms,
                                  mode + "recall": float((hits / k).mean()),
                                  mode + "top10_in_k": float((top10 / 10).mean())})
                print(json.dumps(point))


def run_sharded(args, cfg, pkg, rank, world, local_rank, device):
    """Document-sharded search (the scaling sketch of Sec. 3.3): every rank indexes its contiguous range of the
    documents, the queries are the same everywhere, and one step is ShardedSearcher.search -- local stages 1-3,
    all-gather of ids and integer scores, global selection, stages 4-5 on the rank's own survivors, all-gather, merge.
    The corpus is fixed while ranks are added, so scaling is strong.  With one rank the result is also compared with
    the plain search.  Prints one JSON line on rank 0."""
    import torch.distributed as dist
    from paper_2608_23553_b200.sharded import ShardEngine, ShardedSearcher, shard_ranges
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29533")
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=device)
    corp, q, gen_s = build_workload(cfg, device, rabitq=args.rabitq)
    lo, hi = shard_ranges(cfg.n_docs, world)[rank]
    off = torch.cat([torch.zeros(1, dtype=torch.int64, device=device), torch.cumsum(corp.doclens.to(torch.int64), 0)])
    t0, t1 = int(off[lo]), int(off[hi])
    index = pkg.Index(corp.centroids, corp.cids[t0:t1].contiguous(), corp.codes[t0:t1].contiguous(),
                      corp.doclens[lo:hi].contiguous(), cfg.nbits, cfg.res_lo, cfg.res_hi)
    mode = "rabitq" if args.rabitq else ("partial" if args.partial else "ci")
    if args.partial or args.rabitq:
        index.enable_partial()
    if args.rabitq:
        index.attach_rabitq(corp.rotation, corp.rq_bits[t0:t1].contiguous(), corp.rq_inv_dot[t0:t1].contiguous())
    # check=False: no host synchronisation inside the timed steps; the exchanged status words are read once at the end
    searcher = ShardedSearcher(ShardEngine(index, lo, mode), check=False)
    B, nq, P, n_prune, k = args.batch, cfg.q_len, cfg.nprobe, cfg.n_prune, cfg.k
    n_batches = max(1, min(args.steps + args.warmup, (q.shape[0] + B - 1) // B + 1))
    idx = (torch.arange(n_batches * B, device=device) % q.shape[0]).view(n_batches, B)
    batches = q[idx].contiguous()
    equal = None
    if world == 1:                       # one shard holding everything: must equal the plain search bit for bit
        ids_s, sc_s = searcher.search(batches[0], P, n_prune, k)
        ids_p, sc_p = index.search(batches[0], P, n_prune, k, partial=args.partial, rabitq=args.rabitq)
        equal = bool(torch.equal(ids_s, ids_p) and torch.equal(sc_s, sc_p))
    for s in range(args.warmup):
        searcher.search(batches[s % n_batches], P, n_prune, k)
    dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for s in range(args.steps):
        searcher.search(batches[(args.warmup + s) % n_batches], P, n_prune, k)
    e1.record()
    dist.barrier()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    t = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_total = float(t.item())
    status_words = [int(w) for w in searcher.last_status.cpu().tolist()]
    assert not any(status_words), "a rank reported a device-side failure: %s" % status_words
    if rank == 0:
        qps = B * args.steps / (ms_total / 1e3)        # every rank works on the same queries: the job's rate
        print(json.dumps({
            "metric": metric_name(cfg, B) + ", document-sharded", "value": qps, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": DTYPE, "data": "synthetic",
            "config": {"workload": cfg.name, "batch": B, "pruning": mode,
                       "parallelism": "documents sharded over %d ranks, two all-gathers of ids and scores per step" % world,
                       "docs_per_rank": hi - lo, "equals_plain_search": equal},
            "clocks": clocks}))
    dist.destroy_process_group()


def run_graph_eval(args, cfg, pkg, index, corp, q):
    """The centroid-graph search against the exhaustive scan it replaces (stage 1 + stage 2a), probe stage alone:
    time per batch and recall of the exhaustive top-nprobe / of the best centroid, for several (entry points, list
    size), on the workload's own centroids and on a structured centroid set of the same size (unit vectors of an
    8-dimensional subspace, where a nearest-neighbour graph has local structure to navigate by; the workloads'
    centroids are near-orthogonal random directions).  One JSON line per point."""
    dev = q.device
    B, nq, P, R = args.batch, cfg.q_len, cfg.nprobe, args.graph_degree
    qb = q[:B].contiguous()

    def timed(fn, reps=5):
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    def evaluate(name, ix, queries):
        taps = ix.alloc_taps(B, nq, P, 16, max_candidates=1024, table=False, ci=False)
        ix.run_stages(1, 2, queries, B, nq, P, 16, 1, taps, max_candidates=1024)
        exact = taps.probes.clone()
        pkg.profile_enable(True)
        pkg.profile_read()
        for _ in range(3):
            ix.run_stages(1, 2, queries, B, nq, P, 16, 1, taps, max_candidates=1024)
        ms, _ = pkg.profile_read()
        pkg.profile_enable(False)
        exact_ms = (ms["score_table"] + ms["probes"]) / 3
        t0 = time.time()
        ix.build_graph(R)
        build_s = time.time() - t0
        for E, beam in ((64, 32), (256, 32), (1024, 32), (4096, 32), (4096, 64), (16384, 64)):
            if E > ix.K:
                continue
            pr, sc, nvis, _ = ix.graph_probes(queries, P, beam, E)
            ms_g = timed(lambda: ix.graph_probes(queries, P, beam, E))
            hit = (pr[:, :, :, None] == exact[:, :, None, :]).any(dim=3).float().mean().item()
            first = (pr[:, :, 0] == exact[:, :, 0]).float().mean().item()
            print(json.dumps({"graph_eval": name, "n_centroids": ix.K, "degree": R, "n_entries": E, "beam": beam,
                              "batch": B, "graph_probe_ms": ms_g, "exhaustive_ms": exact_ms,
                              "probe_recall": hit, "best_centroid_recall": first,
                              "visited_per_token": float(nvis.float().mean()), "graph_build_s": round(build_s, 2)}))

    evaluate(cfg.name + " centroids (random directions)", index, qb)
    # structured centroids: unit vectors of a random 8-dimensional subspace; query tokens = a centroid plus noise
    g = torch.Generator(device=dev)
    g.manual_seed(1234)
    basis = torch.linalg.qr(torch.randn(cfg.dim, 8, generator=g, device=dev)).Q            # [D, 8] orthonormal
    z = torch.randn(cfg.n_centroids, 8, generator=g, device=dev)
    cent = (z / z.norm(dim=1, keepdim=True)) @ basis.t()
    qi = torch.randint(0, cfg.n_centroids, (B * nq,), generator=g, device=dev)
    qs = cent[qi] + 0.02 * torch.randn(B * nq, cfg.dim, generator=g, device=dev)
    qs = (qs / qs.norm(dim=1, keepdim=True)).view(B, nq, cfg.dim).contiguous()
    ix2 = pkg.Index(cent.contiguous(), corp.cids[:1024].contiguous(), corp.codes[:1024].contiguous(),
                    torch.full((16,), 64, dtype=torch.int32, device=dev), cfg.nbits, cfg.res_lo, cfg.res_hi)
    evaluate("structured centroids (8-dimensional subspace)", ix2, qs)


PRUNING_TEXT = {"rabitq_graph": "probes from the centroid graph, then the RaBitQ pipeline",
                "ci": "centroid interaction over every candidate token",
                "partial": "partial scores of retrieved tokens (Algorithm 2)",
                "rabitq": "partial 1-bit RaBitQ scores of retrieved tokens, then complete 1-bit scores"}


def measure(pkg, cfg, corp, q, index, args, device, mode="ci", dist=None, local_rank=0, steps=None, batch1_n=None,
            full=True):
    """Times one workload in one pruning mode on this rank and returns the result fields (QPS at the batch size and at
    batch 1, per-stage CUDA-event times, the roofline of the dominant kernel and of each stage).  full=False leaves
    out the end-to-end run through the host entry point and the CUDA-graph variant of batch 1."""
    kw = {"partial": mode == "partial", "rabitq": mode in ("rabitq", "rabitq_graph")}
    if mode == "rabitq_graph":
        kw["graph"] = (args.graph_beam, args.graph_entries, 1 << 30)
    B = args.batch if args.batch > 0 else (64 if cfg.name.startswith("long") else 16 if cfg.name == "tiny" else 256)
    nq, P, n_prune, k = cfg.q_len, cfg.nprobe, cfg.n_prune, cfg.k
    steps = args.steps if steps is None else steps
    warmup = args.warmup
    batch1_n = args.batch1_queries if batch1_n is None else batch1_n
    maxc = candidate_capacity(index, q, nq, P, n_prune, k)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # batches cycle through the config's query set
    n_batches = max(1, min(steps + warmup, (q.shape[0] + B - 1) // B + 1))
    idx = (torch.arange(n_batches * B, device=device) % q.shape[0]).view(n_batches, B)
    batches = q[idx].contiguous()                                   # [n_batches, B, nq, D] on the device
    out = (torch.empty(B, k, dtype=torch.int32, device=device), torch.empty(B, k, dtype=torch.float32, device=device))

    # algorithmic work per batch (outside the timed region): candidate documents and their tokens, from the taps
    doclens64 = corp.doclens.to(torch.int64)
    list_len = torch.bincount(corp.cids.to(torch.int64).view(-1), minlength=cfg.n_centroids)   # posting-list sizes
    work = []
    for bi in range(n_batches):
        taps = index.alloc_taps(B, nq, P, n_prune, max_candidates=maxc, table=False, ci=False)
        index.search(batches[bi], P, n_prune, k, max_candidates=maxc, taps=taps, **kw)
        assert index.status() == 0
        mask = torch.arange(taps.cand.shape[1], device=device)[None, :] < taps.n_cand[:, None].to(torch.int64)
        toks = (doclens64[taps.cand.to(torch.int64).clamp_(0, index.N - 1)] * mask).sum()
        pr = taps.pruned.to(torch.int64)
        toks4 = (doclens64[pr.clamp(min=0)] * (pr >= 0)).sum()
        work.append({"cand": int(taps.n_cand.sum()), "cand_tokens": int(toks), "pruned_tokens": int(toks4),
                     "contenders": int(taps.n_contenders.sum()),
                     "retrieved": int(list_len[taps.probes.to(torch.int64)].sum())})
        del taps, mask
    del list_len
    torch.cuda.empty_cache()

    # ---- device-resident timing: W warm-up steps, then exactly K timed steps ------------------------------------
    for s in range(warmup):
        index.search(batches[s % n_batches], P, n_prune, k, max_candidates=maxc, out=out, **kw)
    barrier()
    pkg.profile_enable(True)
    pkg.profile_read()
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for s in range(steps):
        index.search(batches[(warmup + s) % n_batches], P, n_prune, k, max_candidates=maxc, out=out, **kw)
    e1.record()
    barrier()
    clocks = sampler.stop()
    ms_total = e0.elapsed_time(e1)
    stage_ms, launches = pkg.profile_read()
    pkg.profile_enable(False)
    qps, ms_total = whole_job_qps(ms_total, B * steps, dist, device)
    ms_per_step = ms_total / steps

    dq = torch.empty_like(batches[0])

    def host_search(hq, hout, dbuf, dout):
        if mode == "ci":
            index.search_host(hq, P, n_prune, k, max_candidates=maxc, out=hout)
        else:       # the host entry point has no such variant: pinned copies around the device entry point
            dbuf.copy_(hq, non_blocking=True)
            index.search(dbuf, P, n_prune, k, max_candidates=maxc, out=dout, **kw)
            hout[0].copy_(dout[0], non_blocking=True)
            hout[1].copy_(dout[1], non_blocking=True)
            torch.cuda.synchronize()

    e2e = None
    if full:
        # ---- end to end through the host entry point: pinned host queries in, host ids/scores out ----------------
        host_batches = batches.cpu().pin_memory()
        host_out = (torch.empty(B, k, dtype=torch.int32).pin_memory(), torch.empty(B, k, dtype=torch.float32).pin_memory())
        for s in range(2):
            host_search(host_batches[s % n_batches], host_out, dq, out)
        barrier()
        w0 = time.perf_counter()
        for s in range(steps):
            host_search(host_batches[(warmup + s) % n_batches], host_out, dq, out)
        torch.cuda.synchronize()
        e2e_s = time.perf_counter() - w0
        e2e_qps, _ = whole_job_qps(e2e_s * 1e3, B * steps, dist, device)
        e2e = {"value": e2e_qps, "unit": UNIT, "h2d_bytes_per_step": B * nq * cfg.dim * 4, "d2h_bytes_per_step": B * k * 8}

    # ---- batch 1: one synchronised query at a time (the paper's protocol: latency = 1 / QPS) --------------------
    n1 = min(batch1_n, q.shape[0])
    out1 = (torch.empty(1, k, dtype=torch.int32, device=device), torch.empty(1, k, dtype=torch.float32, device=device))
    for i in range(5):
        index.search(q[i % q.shape[0]:i % q.shape[0] + 1], P, n_prune, k, max_candidates=maxc, out=out1, **kw)
    torch.cuda.synchronize()
    lat = []
    pkg.profile_enable(True)
    pkg.profile_read()
    for i in range(n1):
        a = time.perf_counter()
        index.search(q[i:i + 1], P, n_prune, k, max_candidates=maxc, out=out1, **kw)
        torch.cuda.synchronize()
        lat.append(time.perf_counter() - a)
    stage_ms1, _ = pkg.profile_read()
    pkg.profile_enable(False)
    lat = np.array(lat)
    res = {
        "metric": metric_name(cfg, B) + (" with partial-score refinement" if mode == "partial" else "")
        + (" on RaBitQ 1-bit codes (paper pipeline)" if mode == "rabitq" else "")
        + (" on RaBitQ 1-bit codes with probes from the centroid graph (degree %d, %d entry points, list of %d)"
           % (args.graph_degree, args.graph_entries, args.graph_beam) if mode == "rabitq_graph" else ""),
        "value": qps, "unit": UNIT, "ms_per_step": ms_per_step, "steps": steps, "batch": B,
        "qps_batch1": float(1.0 / lat.mean()),
        "stage_ms_batch1": {name: round(v / min(n1, 256), 4) for name, v in stage_ms1.items()},
        "latency_ms_batch1": {"mean": float(lat.mean() * 1e3), "p50": float(np.percentile(lat, 50) * 1e3),
                              "p95": float(np.percentile(lat, 95) * 1e3), "p99": float(np.percentile(lat, 99) * 1e3)},
        "gpu_launches": int(sum(launches.values())), "clocks": clocks, "max_candidates": maxc if maxc else cfg.n_docs,
    }
    if full:
        # the same protocol with the search captured once in a CUDA graph (same kernels; no per-kernel launch gaps)
        graphed = pkg.GraphedSearch(index, 1, nq, P, n_prune, k, max_candidates=maxc, **kw)
        for i in range(5):
            graphed(q[i:i + 1])
        torch.cuda.synchronize()
        lat_g = []
        for i in range(n1):
            a = time.perf_counter()
            graphed(q[i:i + 1])
            torch.cuda.synchronize()
            lat_g.append(time.perf_counter() - a)
        res["qps_batch1_cuda_graph"] = float(1.0 / np.mean(lat_g))
        del graphed
        host_q1 = q[:n1].cpu().pin_memory()
        hout1 = (torch.empty(1, k, dtype=torch.int32).pin_memory(), torch.empty(1, k, dtype=torch.float32).pin_memory())
        w0 = time.perf_counter()
        dq1 = torch.empty_like(q[:1])
        for i in range(n1):
            host_search(host_q1[i:i + 1], hout1, dq1, out1)
        e2e["batch1_value"] = n1 / (time.perf_counter() - w0)
        res["e2e"] = e2e

    # ---- roofline of the dominant kernel -------------------------------------------------------------------------
    peak, peak_kind = measured_peaks()
    used = [work[(warmup + s) % n_batches] for s in range(steps)]
    mean = lambda key: float(np.mean([u[key] for u in used]))       # noqa: E731
    n_prof = min(steps, 256)                                         # the library times at most 256 calls per read
    ci_ms = stage_ms["centroid_interaction"] / n_prof
    gbs = lambda nbytes, ms: nbytes / (ms * 1e-3) / 1e9 if ms > 0 else 0.0   # noqa: E731
    # algorithmic HBM bytes of one launch of the stage-3 bound scan: the centroid id of every candidate token (4 B) +
    # 8 B per candidate document (its token offsets); the kernel's own id / range / bound traffic is not the method's
    ci_bytes = 4.0 * mean("cand_tokens") + 8.0 * mean("cand")
    # what binds it: one table-row lookup per candidate token; a lookup is one distinct 128-byte line for the SM's
    # load pipe, which retires one line per cycle, so the roof is SMs x SM clock row lookups per second (derived from
    # the device's SM count and the clock sampled during the timed region; not a measured peak)
    rows = mean("cand_tokens")
    sm_count = torch.cuda.get_device_properties(device).multi_processor_count
    sm_hz = 1e6 * (clocks["sm_mhz"] or clocks["sm_max_mhz"] or 1965.0)
    lookup_roof = sm_count * sm_hz
    g4_ms = stage_ms["residual_scores"] / n_prof
    # stage 4 reads per survivor token its centroid id + residual code (or its 1-bit code + scale on the RaBitQ path);
    # the centroid term additionally gathers one int32 table row (q_len x 4 B) per token, which is the implementation's
    # traffic, reported beside the method's
    rq_mode = mode in ("rabitq", "rabitq_graph")
    g4_bytes = mean("pruned_tokens") * ((cfg.dim // 8 + 4.0) if rq_mode else (4.0 + cfg.code_bytes))
    g4_row_bytes = 0.0 if rq_mode else mean("pruned_tokens") * nq * 4.0
    stages = {name: round(v / n_prof, 4) for name, v in stage_ms.items()}
    if mode == "ci":
        ratio, src = NCU_CI_DRAM_PER_ALGORITHMIC_BYTE.get(cfg.name, NCU_CI_DRAM_PER_ALGORITHMIC_BYTE[None])
        frac = gbs(ci_bytes, ci_ms) / peak
        roofline = {
            "kernel": "ci_coarse_rng_kernel (stage 3 bound scan over every candidate token)", "bound": "hbm",
            "achieved": gbs(ci_bytes, ci_ms), "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": frac,
            "frac_of_nominal_8_tb_s": gbs(ci_bytes, ci_ms) / 8000.0,       # the task quotes ~8 TB/s; context only
            "traffic": ratio * ci_bytes + float(B) * cfg.n_centroids * nq,
            "traffic_kind": "stored ncu figure, not measured in this run: %.3f DRAM bytes per algorithmic byte from %s, "
                            "x this launch's algorithmic bytes, + each query's 8-bit table once" % (ratio, src),
            "ms_per_launch": ci_ms, "algorithmic_bytes_per_launch": ci_bytes,
            "target": {"frac": TARGET, "met": bool(frac >= TARGET),
                       "note": "the task's 60 % of HBM peak for the code-scan stages is NOT met: every 4-byte centroid "
                               "id costs one 32-byte table-row lookup through L1/L2, which binds the kernel"},
            "contender_fraction": mean("contenders") / max(mean("cand"), 1.0),
            "binding_roof": {"bound": "table-row lookups (one 128-byte line per SM cycle); derived from SM count x "
                                      "sampled SM clock, not a driver-measured peak",
                             "lookups_per_launch": rows, "achieved_glookups_s": rows / (ci_ms * 1e-3) / 1e9 if ci_ms > 0 else 0.0,
                             "peak_glookups_s": lookup_roof / 1e9, "sm_count": sm_count, "sm_mhz": sm_hz / 1e6,
                             "frac": rows / (ci_ms * 1e-3) / lookup_roof if ci_ms > 0 else 0.0,
                             "l2_bytes_per_launch": rows * nq},
        }
    else:
        # candidate refinement by partial scores replaces the scan: the dominant stage-3 kernel visits every token of
        # the nq * nprobe probed posting lists.  Algorithmic bytes per visit: the list entry (token id + document id,
        # 8 B) and the token's code (residual code, or 1-bit code + its 4-byte scale); per candidate document its
        # partial score (4 B).  The table of running maxima is the implementation's, not the method's, and is not
        # counted.  The slot times the clear, the scoring kernel and (RaBitQ) the summation together.
        code_b = (cfg.dim // 8 + 4.0) if rq_mode else float(cfg.code_bytes)
        ps_bytes = mean("retrieved") * (8.0 + code_b) + mean("cand") * 4.0
        frac = gbs(ps_bytes, ci_ms) / peak
        traffic, tk = None, None
        if cfg.name == "mid" and mode == "partial":
            per_query, src = NCU_PARTIAL_DRAM_PER_QUERY
            traffic, tk = per_query * B, "stored ncu figure, not measured in this run: " + src + " x batch"
        roofline = {
            "kernel": ("rabitq_partial_kernel" if rq_mode else "partial_score_kernel")
            + " (+ its clear kernel): partial scores of the retrieved tokens, Algorithm 2", "bound": "hbm",
            "achieved": gbs(ps_bytes, ci_ms), "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": frac,
            "traffic": traffic, "traffic_kind": tk, "ms_per_launch": ci_ms, "algorithmic_bytes_per_launch": ps_bytes,
            "target": {"frac": TARGET, "met": bool(frac >= TARGET)},
            "visits_per_launch": mean("retrieved"),
            "note": "scattered 32-byte sectors (codes of random tokens, read-modify-write of 4-byte cells): the roof "
                    "of such accesses is below the streaming-copy peak this fraction is taken against"}
        ci_bytes = ps_bytes
    roofline["stage_ms_per_step"] = stages
    # per-stage achieved fraction of the roof that the stage's algorithmic work is measured against
    i8_peak, i8_kind = measured_int8_tops()

    def frac_entry(bound, amount, ms, pk, unit, **more):
        ach = amount / (ms * 1e-3) if ms > 0 else 0.0
        e = {"bound": bound, "achieved": ach, "peak": pk, "unit": unit, "frac": ach / pk if pk else 0.0}
        e.update(more)
        return e

    g1_ms = stage_ms["score_table"] / n_prof
    pr_ms = stage_ms["probes"] / n_prof
    g4_frac = gbs(g4_bytes, g4_ms) / peak
    roofline["per_stage"] = {
        "score_table": frac_entry("tensor (int8, %s)" % i8_kind, 2.0 * 9.0 * B * nq * cfg.n_centroids * cfg.dim / 1e12,
                                  g1_ms, i8_peak, "TOP/s",
                                  table_write_gbs=gbs(B * nq * cfg.n_centroids * 5.0, g1_ms)),
        "probes": frac_entry("hbm", B * nq * cfg.n_centroids * 4.0 / 1e9, pr_ms, peak, "GB/s"),
        ("partial_scores" if mode != "ci" else "centroid_interaction_bounds"):
            frac_entry("hbm", ci_bytes / 1e9, ci_ms, peak, "GB/s", target_frac=TARGET, target_met=bool(frac >= TARGET)),
        "residual_scores": frac_entry("hbm (code + centroid-id bytes)", g4_bytes / 1e9, g4_ms, peak, "GB/s",
                                      target_frac=TARGET, target_met=bool(g4_frac >= TARGET),
                                      with_table_row_gathers_gbs=gbs(g4_bytes + g4_row_bytes, g4_ms),
                                      surviving_tokens_per_launch=mean("pruned_tokens")),
        "residual_scores_tensor": frac_entry("tensor (int8, %s)" % i8_kind,
                                             2.0 * 3.0 * mean("pruned_tokens") * nq * cfg.dim / 1e12, g4_ms, i8_peak,
                                             "TOP/s"),
    }
    res["roofline"] = roofline
    res["pruning"] = PRUNING_TEXT[mode]
    if full and dist is None:                  # (one process: the microbenchmark runs on device 0)
        iso = isolated_int8_mma_tops()
        if iso:
            roofline["per_stage"]["score_table"]["isolated_mma_loop_tops"] = iso
    joint = index.probe_plan(B, nq, P) if mode != "rabitq_graph" else 0
    if joint:
        # stages 1 and 2a run together: the stage-1 slot also times the scans of the sampled rows, and the probes
        # slot only the selection from the queues; the finished table is not read again
        roofline["per_stage"]["score_table"]["includes"] = "bounds and queues of the probe stage (sample stride %d)" % joint
        roofline["per_stage"]["probes"] = {"bound": "selection from the queues filled by the score table's epilogue "
                                                    "(the table is not read again)", "frac": None,
                                           "ms_per_launch": pr_ms}
    if mode == "rabitq_graph":
        # stage 1 does not run and the probes slot times the graph search, which streams no table
        roofline["per_stage"]["score_table"] = {"bound": "not run (probes come from the centroid graph)", "frac": None}
        roofline["per_stage"]["probes"] = {"bound": "latency of dependent expansions (graph search)", "frac": None,
                                           "ms_per_launch": pr_ms}
        # how many of the exhaustive top-nprobe centroids (and of the best ones) the graph search found, first batch
        t = index.alloc_taps(B, nq, P, 16, max_candidates=1024, table=False, ci=False)
        index.run_stages(1, 2, batches[0], B, nq, P, 16, 1, t, max_candidates=1024)
        pr, _, nvis, _ = index.graph_probes(batches[0], P, args.graph_beam, args.graph_entries)
        res["graph"] = {"degree": args.graph_degree, "n_entries": args.graph_entries, "beam": args.graph_beam,
                        "probe_recall": (pr[:, :, :, None] == t.probes[:, :, None, :]).any(dim=3).float().mean().item(),
                        "best_centroid_recall": (pr[:, :, 0] == t.probes[:, :, 0]).float().mean().item(),
                        "visited_per_query_token": float(nvis.float().mean()), "n_centroids": cfg.n_centroids}
        del t
    return res


def summary(r):
    """The short form of a measurement kept under `configs` in the headline line."""
    per = r["roofline"]["per_stage"]
    return {"metric": r["metric"], "value": r["value"], "unit": UNIT, "batch": r["batch"], "steps": r["steps"],
            "ms_per_step": r["ms_per_step"], "qps_batch1": r["qps_batch1"],
            "latency_ms_batch1": r["latency_ms_batch1"], "stage_ms_per_step": r["roofline"]["stage_ms_per_step"],
            "roofline_frac": r["roofline"]["frac"], "roofline_kernel": r["roofline"]["kernel"].split(" ")[0],
            "target_met": r["roofline"]["target"]["met"],
            "stage4_code_frac_of_hbm": per["residual_scores"]["frac"],
            "score_table_frac_of_int8_peak": per["score_table"]["frac"], "probes_frac_of_hbm": per["probes"]["frac"],
            "clocks": r["clocks"], "gpu_launches": r["gpu_launches"], **({"graph": r["graph"]} if "graph" in r else {})}


def run_other_configs(pkg, args, device, headline_done):
    """A shorter measurement (fewer steps, no end-to-end leg) of every workload and pipeline other than the headline's
    centroid-interaction line.  Errors are recorded, not raised: the headline line must still be printed."""
    out = {}
    steps = max(3, min(args.steps, 10))
    plan = [("mid", ("ci", "partial", "rabitq")), ("tiny", ("ci",)), ("long_d128_b2", ("ci", "partial")),
            ("long_d128_b1", ("ci",)), ("long_d96_b2", ("ci",)), ("long_d96_b1", ("ci",))]
    for name, modes in plan:
        if name in headline_done:
            continue
        try:
            cfg = CONFIGS[name]
            corp, q, _ = build_workload(cfg, device, rabitq="rabitq" in modes)
            index = pkg.Index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
            for mode in modes:
                if mode == "partial":
                    index.enable_partial()
                if mode == "rabitq":
                    index.attach_rabitq(corp.rotation, corp.rq_bits, corp.rq_inv_dot)
                key = name if mode == "ci" else name + "_" + mode
                out[key] = summary(measure(pkg, cfg, corp, q, index, args, device, mode, steps=steps, batch1_n=50,
                                           full=False))
            index.close()
            if name in ("tiny", "mid") and not args.no_cpu_baseline:
                # the oracle on one host core: Tiny all 16 queries, Mid ten queries
                n_o = 16 if name == "tiny" else 10
                oix = oracle_index(corp, cfg)
                n, secs = time_oracle(oix, q.cpu().numpy(), cfg, budget_s=0.0, min_q=n_o, max_q=n_o)
                out[name]["cpu_baseline"] = {"value": n / secs, "unit": UNIT, "cores": 1, "kind": "oracle",
                                             "sample": "first %d queries, all stages, %.1f s" % (n, secs)}
                del oix
            del index, corp, q
        except Exception as e:          # noqa: BLE001
            out[name + "_error"] = "%s: %s" % (type(e).__name__, e)
        torch.cuda.empty_cache()
    return out


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch_ranks(n):
    """Start n ranks of this script (one process per GPU) under torch.distributed.run on this node and return their
    exit code.  Used when `--gpus n` is given and the script is not already running under a launcher."""
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")             # keep the communicator's init lines (ranks, transport) in the log
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n), "--master-addr",
           "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd, env=env)


def dry_launch(args, rank, world):
    """The multi-rank plumbing of the replica benchmark without a GPU: `world` gloo ranks on the CPU, each with a made-up
    step time, reduced as in the real run (rank r reports 100 + 50 r ms for 512 queries)."""
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("gloo")
    qps, ms = whole_job_qps(100.0 + 50.0 * rank, 512, dist)
    if rank == 0:
        print(json.dumps({"dry_launch": True, "n_gpus": world, "value": qps, "unit": UNIT, "ms": ms, "scaling": "weak"}))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="", help="one workload only (tiny, mid, large, long_d128_b2, ...); default: the "
                    "Large headline plus a short measurement of every other workload")
    ap.add_argument("--docs", type=int, default=0, help="keep only this many documents of the workload (same recipe; "
                    "for profiler captures, which need a small case)")
    ap.add_argument("--batch", type=int, default=0, help="queries per call (default 256; 64 for the long-document configs, 16 for Tiny)")
    ap.add_argument("--partial", action="store_true",
                    help="prune with the paper's partial scores (chimera_search_partial) instead of stage 3")
    ap.add_argument("--rabitq", action="store_true",
                    help="the paper's pipeline on RaBitQ 1-bit codes (chimera_search_rabitq)")
    ap.add_argument("--graph", action="store_true",
                    help="with --rabitq: probes from the proximity graph over the centroids (chimera_search_rabitq_graph)")
    ap.add_argument("--graph-eval", action="store_true",
                    help="graph search vs exhaustive centroid scan: time and probe recall (see run_graph_eval)")
    ap.add_argument("--graph-degree", type=int, default=32)
    ap.add_argument("--graph-beam", type=int, default=32)
    ap.add_argument("--graph-entries", type=int, default=256)
    ap.add_argument("--sweep", action="store_true", help="QPS vs recall over nprobe x n_prune x k (see run_sweep)")
    ap.add_argument("--sweep-queries", type=int, default=200)
    ap.add_argument("--batch1-queries", type=int, default=200)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true", help="headline workload only")
    ap.add_argument("--sharded", action="store_true",
                    help="document-sharded search over the ranks (one JSON line; see run_sharded) instead of replicas")
    ap.add_argument("--dry-launch", action="store_true",
                    help="exercise the rank launch and the timing reduction with gloo ranks on the CPU (no GPU work)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    # one process per GPU: when not already under a launcher, start the ranks here
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        sys.exit(launch_ranks(args.gpus))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.dry_launch:
        dry_launch(args, rank, world)
        return

    single = bool(args.config) or args.partial or args.rabitq or args.sweep or args.sharded or args.graph_eval
    cfg = CONFIGS[args.config or HEADLINE]
    if args.docs > 0:
        cfg = cfg.replace(n_docs=args.docs)
    if args.impl == "reference":
        if args.batch <= 0:
            args.batch = 64 if cfg.name.startswith("long") else 256
        run_reference(args, cfg, rank, world)
        return

    import paper_2608_23553_b200 as pkg
    pkg.lib()                                    # fails loudly if the CUDA library is missing
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if args.sharded:
        if args.batch <= 0:
            args.batch = 64 if cfg.name.startswith("long") else 256
        run_sharded(args, cfg, pkg, rank, world, local_rank, device)
        return
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    mode = ("rabitq_graph" if args.graph else "rabitq") if args.rabitq else ("partial" if args.partial else "ci")
    corp, q, gen_s = build_workload(cfg, device, rabitq=args.rabitq or args.sweep or (not single and world == 1))
    t0 = time.time()
    index = pkg.Index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    build_s = time.time() - t0
    if args.partial or args.sweep:
        index.enable_partial()
    if args.rabitq or args.sweep:
        index.attach_rabitq(corp.rotation, corp.rq_bits, corp.rq_inv_dot)
    if args.sweep:
        if args.batch <= 0:
            args.batch = 256
        if rank == 0:
            run_sweep(args, cfg, pkg, index, corp, q)
        return
    if args.graph_eval:
        if args.batch <= 0:
            args.batch = 256
        if rank == 0:
            run_graph_eval(args, cfg, pkg, index, corp, q)
        return
    if args.graph:
        index.build_graph(args.graph_degree)

    r = measure(pkg, cfg, corp, q, index, args, device, mode, dist, local_rank)
    nq = cfg.q_len
    result = {
        "metric": r["metric"], "value": r["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": r["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": DTYPE, "data": "synthetic",
        "config": {"workload": cfg.name, "batch": r["batch"], "n_docs": cfg.n_docs, "n_tokens": corp.n_tokens,
                   "n_centroids": cfg.n_centroids, "dim": cfg.dim, "nbits": cfg.nbits, "q_len": nq,
                   "nprobe": cfg.nprobe, "n_prune": cfg.n_prune, "k": cfg.k,
                   "parallelism": "replicas only" if world > 1 else "single GPU",
                   "max_candidates": r["max_candidates"], "pruning": r["pruning"],
                   "l2": "inputs larger than L2 (index %.1f GB, score table %.1f GB per batch); no flush"
                         % ((corp.cids.numel() * 4 + corp.codes.numel()) / 1e9,
                            r["batch"] * cfg.n_centroids * nq * 4 / 1e9),
                   "gen_s": round(gen_s, 1), "index_build_s": round(build_s, 2)},
        "qps_batch1": r["qps_batch1"], "qps_batch1_cuda_graph": r.get("qps_batch1_cuda_graph"),
        "stage_ms_batch1": r["stage_ms_batch1"], "latency_ms_batch1": r["latency_ms_batch1"],
        "e2e": r["e2e"], "gpu_launches": r["gpu_launches"], "clocks": r["clocks"], "roofline": r["roofline"],
    }
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    if world == 1 and not args.no_cpu_baseline:
        oix = oracle_index(corp, cfg)
        n, secs = time_oracle(oix, q.cpu().numpy(), cfg, budget_s=12.0, min_q=3, max_q=16)
        cores, model = host_cpu()
        result["cpu_baseline"] = {"value": n / secs, "unit": UNIT, "cores": 1, "kind": "oracle",
                                  "sample": "first %d queries of the workload, all stages, %.1f s" % (n, secs),
                                  "host_cores": cores, "host_cpu": model}
        del oix
    if world == 1 and not single and not args.no_other_configs:
        others = {}
        try:                            # the two paper pipelines on the headline corpus, then every other workload
            index.enable_partial()
            others[cfg.name + "_partial"] = summary(measure(pkg, cfg, corp, q, index, args, device, "partial",
                                                            steps=max(3, min(args.steps, 10)), batch1_n=50, full=False))
            index.attach_rabitq(corp.rotation, corp.rq_bits, corp.rq_inv_dot)
            others[cfg.name + "_rabitq"] = summary(measure(pkg, cfg, corp, q, index, args, device, "rabitq",
                                                           steps=max(3, min(args.steps, 10)), batch1_n=50, full=False))
            index.build_graph(args.graph_degree)
            others[cfg.name + "_rabitq_graph"] = summary(measure(pkg, cfg, corp, q, index, args, device, "rabitq_graph",
                                                                 steps=max(3, min(args.steps, 10)), batch1_n=20,
                                                                 full=False))
        except Exception as e:          # noqa: BLE001
            others[cfg.name + "_paper_pipelines_error"] = "%s: %s" % (type(e).__name__, e)
        index.close()
        del index, corp, q
        torch.cuda.empty_cache()
        others.update(run_other_configs(pkg, args, device, {cfg.name}))
        result["configs"] = others
    print(json.dumps(result))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
