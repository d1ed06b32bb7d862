#!/usr/bin/env python
"""Benchmark of the GPU-resident retrieval path (stages 1-5 behind chimera_search).

A step is one chimera_search call over one batch of synthetic queries on the Mid corpus (500k documents, ~60M
tokens, 65,536 centroids, 2-bit residual codes; nprobe 4, n_prune 1024, k 10).  `value` is queries per second at
batch 256 with the queries already on the device; `e2e` is the same through chimera_search_host with pinned host
buffers (host->device and device->host copies inside the timed region); `qps_batch1` follows the paper's protocol of
one synchronised query at a time.  The path does not shard: with --gpus N every rank runs an independent replica.

`--impl reference` times the CPU oracle (as it stands, one thread) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
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


def ncu_traffic(cfg, batch):
    """DRAM bytes (read + write) of one launch of the dominant kernel from an ncu capture, or None.  The capture
    (profiles/ncu_ci_coarse_mid.md) was taken on the Mid corpus at batch 8; traffic is proportional to the number of
    queries (every query has its own table and candidate list), so it is scaled by batch / 8."""
    if cfg.name == "mid" and NCU_CI_COARSE_MID_B8_BYTES:
        return NCU_CI_COARSE_MID_B8_BYTES * batch / 8.0
    return None


NCU_CI_COARSE_MID_B8_BYTES = 443.5e6    # dram__bytes_read.sum + dram__bytes_write.sum of one launch at batch 8
NCU_PARTIAL_MID_B64_BYTES = 1527e6      # the same for partial_score_kernel<2> at batch 64 (profiles/ncu_partial_score_mid.md)


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
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
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
    sample = "1 query per step (of the %d-query batch), %d steps, single thread" % (args.batch, args.steps)
    print(json.dumps({
        "impl": "reference", "metric": metric_name(cfg, args.batch), "value": qps, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int64+f64", "data": "synthetic",
        "config": {"workload": cfg.name, "batch": 1, "sample": sample},
        "cpu_baseline": {"value": qps, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": qps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def exhaustive_truth(index, q, cfg, k_max, chunk=16384):
    """Ground truth for Recall@k: the stage-4 score (residual-decode MaxSim) of EVERY document for each query, through
    the library's stage-isolated entry point in chunks of `chunk` documents, then the k_max best per query.  The
    stage-4 kernel is itself parity-tested against the CPU oracle; here it only replaces candidate generation and
    pruning by "all documents"."""
    dev = q.device
    B, nq = q.shape[0], cfg.q_len
    taps = index.alloc_taps(B, nq, cfg.nprobe, chunk, max_candidates=1024, table=True, ci=False)
    index.run_stages(1, 1, q, B, nq, cfg.nprobe, chunk, 1, taps, max_candidates=1024)
    scores = torch.empty(B, index.N, dtype=torch.float32, device=dev)
    taps.n_pruned = torch.full((B,), chunk, dtype=torch.int32, device=dev)
    for d0 in range(0, index.N, chunk):
        ids = torch.arange(d0, d0 + chunk, device=dev, dtype=torch.int32)
        ids[ids >= index.N] = -1
        taps.pruned = ids[None, :].expand(B, chunk).contiguous()
        index.run_stages(4, 4, q, B, nq, cfg.nprobe, chunk, 1, taps, max_candidates=1024)
        n = min(chunk, index.N - d0)
        scores[:, d0:d0 + n] = taps.score4[:, :n]
    top = torch.topk(scores, k_max, dim=1)
    del scores, taps
    index._ws = None
    torch.cuda.empty_cache()
    return top.indices.to(torch.int32), top.values


def run_sweep(args, cfg, pkg, index, corp, q):
    """QPS (batch `--batch`) and Recall@k (Def. 3, against exhaustive MaxSim over the decoded corpus, on the first
    `--sweep-queries` queries) for nprobe x n_prune x k.  Prints one JSON line per point."""
    dev = q.device
    B, nq = args.batch, cfg.q_len
    nrec = min(args.sweep_queries, q.shape[0])
    qrec = q[:nrec].contiguous()
    t0 = time.time()
    truth_ids, _ = exhaustive_truth(index, qrec, cfg, 1000)
    truth_s = time.time() - t0
    n_batches = max(1, min(3, q.shape[0] // B))
    batches = q[:n_batches * B].view(n_batches, B, nq, cfg.dim).contiguous()
    print(json.dumps({"sweep": cfg.name, "batch": B, "recall_queries": nrec, "ground_truth": "library stage 4 over "
                      "every document (chunks of 16384), top-1000 per query", "ground_truth_s": round(truth_s, 1)}))
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
    searcher = ShardedSearcher(ShardEngine(index, lo, mode))
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
    if rank == 0:
        qps = B * args.steps / (ms_total / 1e3)        # every rank works on the same queries: the job's rate
        print(json.dumps({
            "metric": metric_name(cfg, B) + ", document-sharded", "value": qps, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "int32 fixed point (stages 1-3) + f32 (stage 4)",
            "data": "synthetic",
            "config": {"workload": cfg.name, "batch": B, "pruning": mode,
                       "parallelism": "documents sharded over %d ranks, two all-gathers of ids and scores per step" % world,
                       "docs_per_rank": hi - lo, "equals_plain_search": equal},
            "clocks": clocks}))
    dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="mid")
    ap.add_argument("--batch", type=int, default=0, help="queries per call (default 256; 64 for the long-document configs)")
    ap.add_argument("--partial", action="store_true",
                    help="prune with the paper's partial scores (chimera_search_partial) instead of stage 3")
    ap.add_argument("--rabitq", action="store_true",
                    help="the paper's pipeline on RaBitQ 1-bit codes (chimera_search_rabitq)")
    ap.add_argument("--sweep", action="store_true", help="QPS vs recall over nprobe x n_prune x k (see run_sweep)")
    ap.add_argument("--sweep-queries", type=int, default=200)
    ap.add_argument("--batch1-queries", type=int, default=200)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sharded", action="store_true",
                    help="document-sharded search over the ranks (one JSON line; see run_sharded) instead of replicas")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    cfg = CONFIGS[args.config]
    if args.batch <= 0:
        args.batch = 64 if cfg.name.startswith("long") else 256
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, cfg, rank, world)
        return

    import paper_2608_23553_b200 as pkg
    pkg.lib()                                    # fails loudly if the CUDA library is missing
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if args.sharded:
        run_sharded(args, cfg, pkg, rank, world, local_rank, device)
        return
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    corp, q, gen_s = build_workload(cfg, device, rabitq=args.rabitq or args.sweep)
    t0 = time.time()
    index = pkg.Index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    build_s = time.time() - t0
    B, nq, P, n_prune, k = args.batch, cfg.q_len, cfg.nprobe, cfg.n_prune, cfg.k
    if args.partial or args.sweep:
        index.enable_partial()
    if args.rabitq or args.sweep:
        index.attach_rabitq(corp.rotation, corp.rq_bits, corp.rq_inv_dot)
    mode = {"partial": args.partial, "rabitq": args.rabitq}
    if args.sweep:
        if rank == 0:
            run_sweep(args, cfg, pkg, index, corp, q)
        return
    maxc = candidate_capacity(index, q, nq, P, n_prune, k)

    # batches cycle through the config's query set
    n_batches = max(1, min(args.steps + args.warmup, (q.shape[0] + B - 1) // B + 1))
    idx = (torch.arange(n_batches * B, device=device) % q.shape[0]).view(n_batches, B)
    batches = q[idx].contiguous()                                   # [n_batches, B, nq, D] on the device
    host_batches = batches.cpu().pin_memory()
    out = (torch.empty(B, k, dtype=torch.int32, device=device), torch.empty(B, k, dtype=torch.float32, device=device))
    host_out = (torch.empty(B, k, dtype=torch.int32).pin_memory(), torch.empty(B, k, dtype=torch.float32).pin_memory())

    # algorithmic work per batch (outside the timed region): candidate documents and their tokens, from the taps
    doclens64 = corp.doclens.to(torch.int64)
    list_len = torch.bincount(corp.cids.to(torch.int64).view(-1), minlength=cfg.n_centroids)   # posting-list sizes
    work = []
    for bi in range(n_batches):
        taps = index.alloc_taps(B, nq, P, n_prune, max_candidates=maxc, table=False, ci=False)
        index.search(batches[bi], P, n_prune, k, max_candidates=maxc, taps=taps, **mode)
        assert index.status() == 0
        mask = torch.arange(taps.cand.shape[1], device=device)[None, :] < taps.n_cand[:, None].to(torch.int64)
        toks = (doclens64[taps.cand.to(torch.int64).clamp_(0, index.N - 1)] * mask).sum()
        pr = taps.pruned.to(torch.int64)
        toks4 = (doclens64[pr.clamp(min=0)] * (pr >= 0)).sum()
        work.append({"cand": int(taps.n_cand.sum()), "cand_tokens": int(toks), "pruned_tokens": int(toks4),
                     "contenders": int(taps.n_contenders.sum()),
                     "retrieved": int(list_len[taps.probes.to(torch.int64)].sum())})
        del taps, mask
    torch.cuda.empty_cache()

    # ---- device-resident timing: W warm-up steps, then exactly K timed steps ------------------------------------
    for s in range(args.warmup):
        index.search(batches[s % n_batches], P, n_prune, k, max_candidates=maxc, out=out, **mode)
    barrier()
    pkg.profile_enable(True)
    pkg.profile_read()
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for s in range(args.steps):
        index.search(batches[(args.warmup + s) % n_batches], P, n_prune, k, max_candidates=maxc, out=out,
                     **mode)
    e1.record()
    barrier()
    clocks = sampler.stop()
    ms_total = e0.elapsed_time(e1)
    stage_ms, launches = pkg.profile_read()
    pkg.profile_enable(False)
    qps, ms_total = whole_job_qps(ms_total, B * args.steps, dist, device)
    ms_per_step = ms_total / args.steps

    # ---- end to end through the host entry point: pinned host queries in, host ids/scores out -------------------
    dq = torch.empty_like(batches[0])

    def host_search(hq, hout, dbuf, dout):
        if not (args.partial or args.rabitq):
            index.search_host(hq, P, n_prune, k, max_candidates=maxc, out=hout)
        else:       # the host entry point has no such variant: pinned copies around the device entry point
            dbuf.copy_(hq, non_blocking=True)
            index.search(dbuf, P, n_prune, k, max_candidates=maxc, out=dout, **mode)
            hout[0].copy_(dout[0], non_blocking=True)
            hout[1].copy_(dout[1], non_blocking=True)
            torch.cuda.synchronize()

    for s in range(2):
        host_search(host_batches[s % n_batches], host_out, dq, out)
    barrier()
    w0 = time.perf_counter()
    for s in range(args.steps):
        host_search(host_batches[(args.warmup + s) % n_batches], host_out, dq, out)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - w0
    e2e_qps, _ = whole_job_qps(e2e_s * 1e3, B * args.steps, dist, device)
    h2d = B * nq * cfg.dim * 4
    d2h = B * k * 8

    # ---- batch 1: one synchronised query at a time (the paper's protocol: latency = 1 / QPS) --------------------
    n1 = min(args.batch1_queries, q.shape[0])
    out1 = (torch.empty(1, k, dtype=torch.int32, device=device), torch.empty(1, k, dtype=torch.float32, device=device))
    for i in range(5):
        index.search(q[i:i + 1], P, n_prune, k, max_candidates=maxc, out=out1, **mode)
    torch.cuda.synchronize()
    lat = []
    pkg.profile_enable(True)
    pkg.profile_read()
    for i in range(n1):
        a = time.perf_counter()
        index.search(q[i:i + 1], P, n_prune, k, max_candidates=maxc, out=out1, **mode)
        torch.cuda.synchronize()
        lat.append(time.perf_counter() - a)
    stage_ms1, _ = pkg.profile_read()
    pkg.profile_enable(False)
    lat = np.array(lat)
    # the same protocol with the search captured once in a CUDA graph (same kernels; no per-kernel launch gaps)
    graphed = pkg.GraphedSearch(index, 1, nq, P, n_prune, k, max_candidates=maxc, **mode)
    for i in range(5):
        graphed(q[i:i + 1])
    torch.cuda.synchronize()
    lat_g = []
    for i in range(n1):
        a = time.perf_counter()
        graphed(q[i:i + 1])
        torch.cuda.synchronize()
        lat_g.append(time.perf_counter() - a)
    lat_g = np.array(lat_g)
    host_q1 = q[:n1].cpu().pin_memory()
    hout1 = (torch.empty(1, k, dtype=torch.int32).pin_memory(), torch.empty(1, k, dtype=torch.float32).pin_memory())
    w0 = time.perf_counter()
    dq1 = torch.empty_like(q[:1])
    for i in range(n1):
        host_search(host_q1[i:i + 1], hout1, dq1, out1)
    e2e1_qps = n1 / (time.perf_counter() - w0)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel: the stage-3 bound scan over every candidate token (ci_coarse_rng_kernel) ---
    peak, peak_kind = measured_peaks()
    used = [work[(args.warmup + s) % n_batches] for s in range(args.steps)]
    mean = lambda key: float(np.mean([u[key] for u in used]))       # noqa: E731
    n_prof = min(args.steps, 256)                                    # the library times at most 256 calls per read
    ci_ms = stage_ms["centroid_interaction"] / n_prof
    # algorithmic HBM bytes of one launch: the centroid id of every candidate token (4 B) + per candidate document
    # its id (4 B), two token offsets (16 B) and the two bounds written (8 B)
    ci_bytes = 4.0 * mean("cand_tokens") + 28.0 * mean("cand")
    ci_gbs = ci_bytes / (ci_ms * 1e-3) / 1e9 if ci_ms > 0 else 0.0
    # what binds it: one table-row lookup per candidate token; a lookup is one distinct 128-byte line for the SM's
    # load pipe, which retires one line per cycle, so the roof is SMs x SM clock row lookups per second
    rows = mean("cand_tokens")
    lookup_roof = 148 * 1.965e9
    cont_frac = mean("contenders") / max(mean("cand"), 1.0)
    g4_ms = stage_ms["residual_scores"] / n_prof
    # stage 4 reads per survivor token its centroid id + residual code (or its 1-bit code + scale on the RaBitQ path)
    g4_bytes = mean("pruned_tokens") * ((cfg.dim // 8 + 4.0) if args.rabitq else (4.0 + cfg.code_bytes))
    stages = {name: round(v / n_prof, 4) for name, v in stage_ms.items()}
    roofline = {
        "kernel": "ci_coarse_rng_kernel (stage 3 bound scan over every candidate token)", "bound": "hbm",
        "achieved": ci_gbs, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
        "frac": ci_gbs / peak, "traffic": ncu_traffic(cfg, B), "ms_per_launch": ci_ms,
        "algorithmic_bytes_per_launch": ci_bytes, "contender_fraction": cont_frac,
        "binding_roof": {"bound": "table-row lookups (one 128-byte line per SM cycle)", "lookups_per_launch": rows,
                         "achieved_glookups_s": rows / (ci_ms * 1e-3) / 1e9 if ci_ms > 0 else 0.0,
                         "peak_glookups_s": lookup_roof / 1e9,
                         "frac": rows / (ci_ms * 1e-3) / lookup_roof if ci_ms > 0 else 0.0,
                         "l2_bytes_per_launch": rows * nq},
        "stage_ms_per_step": stages,
        "stage4": {"kernel": "residual_maxsim_umma (tcgen05 kind::i8)", "ms_per_launch": g4_ms,
                   "code_gbs": g4_bytes / (g4_ms * 1e-3) / 1e9 if g4_ms > 0 else 0.0,
                   "int8_tops": 2.0 * 3.0 * mean("pruned_tokens") * nq * cfg.dim / (g4_ms * 1e-3) / 1e12 if g4_ms > 0 else 0.0},
    }
    if args.partial or args.rabitq:
        # candidate refinement by partial scores replaces the scan: the dominant stage-3 kernel visits every token of
        # the nq * nprobe probed posting lists.  Algorithmic bytes per visit: the list entry (token id + document id,
        # 8 B) and the token's code (residual code, or 1-bit code + its 4-byte scale); per candidate document its
        # partial score (4 B).  The table of running maxima is the implementation's, not the method's, and is not
        # counted.  The slot times the clear, the scoring kernel and (RaBitQ) the summation together.
        code_b = (cfg.dim // 8 + 4.0) if args.rabitq else float(cfg.code_bytes)
        ps_bytes = mean("retrieved") * (8.0 + code_b) + mean("cand") * 4.0
        ps_gbs = ps_bytes / (ci_ms * 1e-3) / 1e9 if ci_ms > 0 else 0.0
        traffic = None
        if cfg.name == "mid" and args.partial and not args.rabitq:
            traffic = NCU_PARTIAL_MID_B64_BYTES * B / 64.0
        for key in ("binding_roof", "contender_fraction"):
            roofline.pop(key)
        roofline.update({
            "kernel": ("rabitq_partial_kernel" if args.rabitq else "partial_score_kernel")
            + " (+ its clear kernel): partial scores of the retrieved tokens, Algorithm 2",
            "achieved": ps_gbs, "frac": ps_gbs / peak, "traffic": traffic, "algorithmic_bytes_per_launch": ps_bytes,
            "visits_per_launch": mean("retrieved"),
            "note": "scattered 32-byte sectors (codes of random tokens, read-modify-write of 4-byte cells): the roof "
                    "of such accesses is below the streaming-copy peak this fraction is taken against"})
    # per-stage achieved fraction of the roof that the stage's algorithmic work is measured against
    i8_peak, i8_kind = measured_int8_tops()

    def frac_entry(bound, work, ms, peak, unit):
        ach = work / (ms * 1e-3) if ms > 0 else 0.0
        return {"bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak if peak else 0.0}

    g1_ms = stage_ms["score_table"] / n_prof
    pr_ms = stage_ms["probes"] / n_prof
    roofline["per_stage"] = {
        "score_table": frac_entry("tensor (int8, %s)" % i8_kind, 2.0 * 9.0 * B * nq * cfg.n_centroids * cfg.dim / 1e12,
                                  g1_ms, i8_peak, "TOP/s"),
        "probes": frac_entry("hbm", B * nq * cfg.n_centroids * 4.0 / 1e9, pr_ms, peak, "GB/s"),
        ("partial_scores" if args.partial or args.rabitq else "centroid_interaction_bounds"):
            frac_entry("hbm", (ps_bytes if args.partial or args.rabitq else ci_bytes) / 1e9, ci_ms, peak, "GB/s"),
        "residual_scores": frac_entry("hbm (code + centroid-id bytes)", g4_bytes / 1e9, g4_ms, peak, "GB/s"),
        "residual_scores_tensor": frac_entry("tensor (int8, %s)" % i8_kind,
                                             2.0 * 3.0 * mean("pruned_tokens") * nq * cfg.dim / 1e12, g4_ms, i8_peak,
                                             "TOP/s"),
    }

    result = {
        "metric": metric_name(cfg, B) + (" with partial-score refinement" if args.partial else "")
        + (" on RaBitQ 1-bit codes (paper pipeline)" if args.rabitq else ""), "value": qps,
        "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int32 fixed point (stages 1-3) + f32 (stage 4)", "data": "synthetic",
        "config": {"workload": cfg.name, "batch": B, "n_docs": cfg.n_docs, "n_tokens": corp.n_tokens,
                   "n_centroids": cfg.n_centroids, "dim": cfg.dim, "nbits": cfg.nbits, "q_len": nq, "nprobe": P,
                   "n_prune": n_prune, "k": k, "parallelism": "replicas only" if world > 1 else "single GPU",
                   "max_candidates": maxc if maxc else cfg.n_docs,
                   "pruning": "partial 1-bit RaBitQ scores of retrieved tokens, then complete 1-bit scores" if args.rabitq
                   else "partial scores of retrieved tokens (Algorithm 2)" if args.partial
                   else "centroid interaction over every candidate token",
                   "l2": "inputs larger than L2 (index %.1f GB, score table %.1f GB per batch); no flush"
                         % ((corp.cids.numel() * 4 + corp.codes.numel()) / 1e9, B * cfg.n_centroids * nq * 4 / 1e9),
                   "gen_s": round(gen_s, 1), "index_build_s": round(build_s, 2)},
        "qps_batch1": float(1.0 / lat.mean()),
        "qps_batch1_cuda_graph": float(1.0 / lat_g.mean()),
        "stage_ms_batch1": {name: round(v / min(n1, 256), 4) for name, v in stage_ms1.items()},
        "latency_ms_batch1": {"mean": float(lat.mean() * 1e3), "p50": float(np.percentile(lat, 50) * 1e3),
                              "p95": float(np.percentile(lat, 95) * 1e3), "p99": float(np.percentile(lat, 99) * 1e3)},
        "e2e": {"value": e2e_qps, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "batch1_value": e2e1_qps},
        "gpu_launches": int(sum(launches.values())),
        "clocks": clocks,
        "roofline": roofline,
    }

    if world == 1 and not args.no_cpu_baseline:
        oix = oracle_index(corp, cfg)
        n, secs = time_oracle(oix, q.cpu().numpy(), cfg, budget_s=12.0, min_q=3, max_q=16)
        result["cpu_baseline"] = {"value": n / secs, "unit": UNIT, "cores": 1, "kind": "oracle",
                                  "sample": "first %d queries of the workload, all stages, %.1f s" % (n, secs)}
    print(json.dumps(result))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
