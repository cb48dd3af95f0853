#!/usr/bin/env python
"""Benchmark of the speculative-decoding hot path: one step = draft k tokens per sequence (n-gram
drafter) + verify the k+1 rows in one forward + greedy accept/commit, for one batch.

    python bench.py --gpus 1 --steps 64 --warmup 8
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference          (the CPU oracle on a bounded sample of the same workload)

Prints ONE JSON line.  Workload: configuration 1 (SLM-135M shape, bf16) at batch 16, k = 5, prompts of
256 tokens, synthetic corpus / prompts / random-init weights.  `value` = tokens committed by all
sequences on all ranks per second of device time over the K timed steps (prefill excluded, inputs
resident in HBM); `e2e` = the same with the step's token buffers copied from pinned host memory and
the results read back inside the timed region.
"""
from __future__ import annotations

import argparse
import datetime
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workload import configs, corpus, weights as W  # noqa: E402

METRIC = "generated tokens/s with n-gram spec decode @1 B200; verify-step HBM GB/s vs peak"
UNIT = "tokens/s"


# DRAM bytes per fused-GEMM launch from the ncu capture of the default workload (config 1, B=16, k=5), summarised in
# profiles/gemm_fused_kernel_config1_b16_ncu.md: per layer 1.40 + 1.15 + 3.81 + 2.62 MB (QKV, O, gate/up, down) and
# 28.4 MB for the LM head, over the step's 121 launches.  Valid for the kernel source whose digest is given;
# any change of gemm_fused.cu makes the figure stale and `traffic` null.
NCU_TRAFFIC = {"workload": (1, 16, 5), "bytes_per_launch": (30 * (1.418 + 1.151 + 3.807 + 2.625) * 1e6 + 56.88e6) / 121,
               "kernel_sha256_16": "49f85da8cd34d69a"}


def kernel_digest():
    import hashlib
    path = os.path.join(ROOT, "paper_2602_24174_b200", "csrc", "gemm_fused.cu")
    return hashlib.sha256(open(path, "rb").read()).hexdigest()[:16]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"], "source": "measured (MEASURED_PEAKS.json)"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback (earlier measurement on this pool)"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi (every 20 ms) from before the timed region on; the
    samples whose time stamps fall inside the region [mark_begin, mark_end] are the ones reported."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.samples, self.proc = index, [], None
        self.t0 = self.t1 = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
            t_wait = time.time()
            while not self.samples and time.time() - t_wait < 3.0:      # running before the region starts
                time.sleep(0.01)
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append(line.strip())

    def mark_begin(self):
        self.t0 = datetime.datetime.now()

    def mark_end(self):
        self.t1 = datetime.datetime.now()

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.05)
        self.proc.terminate()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        rows = []
        for s in self.samples:
            f = [x.strip() for x in s.split(",")]
            if len(f) < 7:
                continue
            try:
                when = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f")
            except ValueError:
                when = None
            try:
                rows.append((when, float(f[1]), float(f[2]), f[3:7]))
            except ValueError:
                continue
        stamped = all(r[0] is not None for r in rows) and self.t0 is not None and self.t1 is not None
        if not stamped:                                       # time stamps in a form not understood: every sample counts
            rows = [(self.t0, r[1], r[2], r[3]) for r in rows]
        inside = [r for r in rows if stamped and self.t0 <= r[0] <= self.t1] if stamped else list(rows)
        where = "inside the timed region" if stamped else "whole sampling window"
        if not inside and rows and stamped:                   # a region shorter than the sampling period: the nearest samples
            mid = self.t0 + (self.t1 - self.t0) / 2
            inside = sorted(rows, key=lambda r: abs((r[0] - mid).total_seconds()))[:2]
            where = "nearest to the timed region"
        reasons = set()
        for r in inside:
            for name, val in zip(names, r[3]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm = [r[1] for r in inside]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": inside[0][2] if inside else None,
                "reasons": sorted(reasons), "samples": len(sm), "sampled": where if sm else "no samples"}


# ----------------------------------------------------------------------------------------------- replicas
# The path does not shard: sequences are independent, so N GPUs run N independent replicas (own prompts,
# replicated weights and tables) with no data-path collective.  Only the timing is reduced over ranks.
def shard_prompts(prompts_all, rank: int, per_rank: int):
    """Rows of the global prompt array that belong to `rank` (per_rank sequences each)."""
    return prompts_all[rank * per_rank:(rank + 1) * per_rank]


def reduce_over_ranks(x: float, op: str, world: int, device) -> float:
    """max or sum of a scalar over all ranks (identity for one rank)."""
    if world == 1:
        return x
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX if op == "max" else dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_throughput(units_local: float, ms_local: float, world: int, device) -> tuple:
    """(units all ranks processed / slowest rank's time, that time in ms)."""
    ms = reduce_over_ranks(ms_local, "max", world, device)
    return reduce_over_ranks(units_local, "sum", world, device) / (ms * 1e-3), ms


def step_bytes(shape, B, k, ctx_lens):
    """Algorithmic HBM bytes of one verify step: every weight once, every live KV byte once, the new KV rows."""
    wbytes = shape.matmul_params() * 2
    kv = sum(ctx_lens) * shape.kv_bytes_per_token() + B * (k + 1) * shape.kv_bytes_per_token()
    return wbytes, kv


def gemm_bytes_per_step(shape, M):
    """Algorithmic bytes of all fused-GEMM launches of one step: every weight matrix once, the (hi, lo) bf16
    activation rows each launch reads, and what its epilogue writes (q float32 + K/V bf16; residual rows
    read + written and the next (hi, lo) rows; SiLU*up (hi, lo) rows; nothing for the LM-head argmax)."""
    s = shape
    hilo = lambda cols: 2 * M * cols * 2
    per_layer = (
        s.qkv_rows * s.d_model * 2 + hilo(s.d_model) + M * s.q_dim * 4 + M * 2 * s.kv_dim * 2        # QKV + RoPE + KV append
        + s.d_model * s.q_dim * 2 + hilo(s.q_dim) + 2 * M * s.d_model * 4 + hilo(s.d_model)         # O + residual
        + 2 * s.d_ff * s.d_model * 2 + hilo(s.d_model) + hilo(s.d_ff)                               # gate/up + SiLU*mul
        + s.d_model * s.d_ff * 2 + hilo(s.d_ff) + 2 * M * s.d_model * 4 + hilo(s.d_model))          # down + residual
    return s.n_layers * per_layer + s.vocab * s.d_model * 2 + hilo(s.d_model)


# ----------------------------------------------------------------------------------------------- oracle legs
def oracle_sample(cfg, B_sample, n_steps, k, prompts):
    """Times the CPU oracle (as it stands) on a bounded sample: B_sample sequences, prompt prefilled,
    n_steps speculative steps each.  Returns (tokens/s over the decode steps, threads used, description)."""
    from oracle import decode as G, drafter as D
    from oracle.model import OracleModel
    tokens, offsets = corpus.make_corpus(cfg, n_docs=min(cfg.corpus.n_docs, 20000))
    ng = D.build_corpus_ngrams_sorted(tokens, offsets, cfg.n_max, cfg.p_min, cfg.model.vocab)
    om = OracleModel(cfg.model, W.make_weights(cfg.model, cfg.seed_weights), np.float32)
    committed_total, t_total = 0, 0.0
    for i in range(B_sample):
        committed = list(map(int, prompts[i]))
        cache = om.new_cache(len(committed) + n_steps * (k + 1) + k + 2)
        om.prefill(committed[:-1], cache)
        t0 = time.perf_counter()
        for _ in range(n_steps):
            drafts = D.draft(ng, committed, k, cfg.lambda_num, cfg.lambda_den)
            st = G.verify_step(om, cache, committed[-1], drafts)
            committed += st.drafts[:st.n_accepted] + [st.next_token]
            committed_total += st.n_accepted + 1
        t_total += time.perf_counter() - t0
    cores = os.cpu_count() or 1
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        pass
    desc = (f"config {cfg.index} ({cfg.name}): {B_sample} of the batch's sequences, prompt {cfg.prompt_len} prefilled "
            f"(untimed), {n_steps} speculative steps each (k={k}), numpy float32, corpus tables from 20000 docs")
    return committed_total / t_total, cores, desc, t_total / (B_sample * n_steps)


def run_reference(args, cfg, B, k):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    prompts = corpus.make_prompts(cfg, 2)
    # warm-up and timed steps are both bounded samples: 1 sequence, a few steps per "step"
    n = max(1, min(args.steps, 16))
    val, cores, desc, s_per_step = oracle_sample(cfg, 1, max(1, min(args.warmup, 2)) + n, k, prompts)
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": s_per_step * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"config {cfg.index} ({cfg.name}) B={B} k={k} prompt {cfg.prompt_len}: bounded sample", "sample": desc},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------- device arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1)
    ap.add_argument("--batch", type=int, default=16)
    ap.add_argument("--k", type=int, default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--only-timed", action="store_true",
                    help="device-resident timed region only (no per-kernel pass, e2e, generate or CPU legs): the command ncu wraps")
    ap.add_argument("--sweep", action="store_true", help="also report the teacher-forced acceptance sweep (forced a = 0..k)")
    ap.add_argument("--no-graph", action="store_true", help="launch every step's kernels from the host instead of replaying a CUDA graph")
    ap.add_argument("--corpus-docs", type=int, default=None, help="build the drafter from the first N corpus documents only")
    args = ap.parse_args()
    cfg = configs.get(args.config)
    B = args.batch
    k = args.k or cfg.k
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args, cfg, B, k)
        return

    import torch
    import torch.distributed as dist
    from paper_2602_24174_b200 import binding as b      # raises if libtasc.so is missing: there is no fallback

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)
    shape = cfg.model

    # ---- inputs (seeded, synthetic); every rank is an independent replica with its own prompts
    host_w = W.make_weights(shape, cfg.seed_weights)
    ctoks, coffs = corpus.make_corpus(cfg, n_docs=args.corpus_docs)
    prompts_all = corpus.make_prompts(cfg, B * world)
    if cfg.n_merged_tokens:
        # configuration 3: merged n-gram tokens on top of the vocabulary (rows = constituent means), corpus and
        # prompts re-tokenised by greedy longest match; selection from the first 20,000 documents
        from dataclasses import replace
        from workload import vocab_expand as VE
        base = shape.vocab
        sel = min(len(coffs) - 1, 20000)
        merges = VE.select_merges(ctoks[:coffs[sel]], coffs[:sel + 1], cfg.n_merged_tokens, n_max=4, vocab=base)
        host_w = VE.expand_weights(host_w, merges)
        ctoks, coffs = VE.retokenize(ctoks, coffs, merges, vocab=base)
        re = [VE.retokenize(pr, np.array([0, pr.size]), merges, vocab=base)[0] for pr in prompts_all]
        plen = min(len(r) for r in re)
        prompts_all = np.stack([r[:plen] for r in re]).astype(np.int32)
        shape = replace(shape, vocab=base + len(merges))
    model = b.Model(shape, b.weights_to_device(host_w, shape.dtype, dev), max_positions=cfg.prompt_len + cfg.max_new + 4096,
                    page_size=cfg.page_size)
    del host_w
    # the corpus tables (once per task): built once untimed (allocator, module load), then timed with the corpus resident
    d_ctoks, d_coffs = torch.from_numpy(ctoks).to(dev), torch.from_numpy(coffs).to(dev)
    drafter = b.tasc_drafter_build(d_ctoks, d_coffs, cfg.n_max, cfg.p_min, shape.vocab)
    del drafter
    torch.cuda.synchronize()
    t_build = time.perf_counter()
    drafter = b.tasc_drafter_build(d_ctoks, d_coffs, cfg.n_max, cfg.p_min, shape.vocab)
    torch.cuda.synchronize()
    t_build = time.perf_counter() - t_build
    n_updates = int(sum(np.maximum(np.diff(coffs) - n, 0).sum() for n in range(1, cfg.n_max + 1)))
    build_report = {"ms": t_build * 1e3, "corpus_tokens": int(ctoks.size), "documents": int(coffs.size - 1),
                    "count_updates": n_updates, "updates_per_s": n_updates / t_build, "timed": "host wall clock around tasc_drafter_build"}
    del d_ctoks, d_coffs
    prompts = shard_prompts(prompts_all, rank, B)
    P = prompts.shape[1]
    total_steps = args.warmup + args.steps
    stride = P + (total_steps + args.steps + 4) * (k + 1) + k + 2       # timed pass + instrumented pass share one state
    if stride > 12288:
        raise SystemExit("too many steps for one token buffer")
    ws = model.new_workspace(B, k, dev)

    def fresh_state():
        tokens = torch.zeros((B, stride), dtype=torch.int32, device=dev)
        tokens[:, :P] = torch.from_numpy(prompts).to(dev)
        length = torch.full((B,), P, dtype=torch.int32, device=dev)
        pool, bt, kv = model.new_kv(B, stride + b.MAX_ROWS, dev)
        seqs = b.make_seqs(tokens, length)
        b.tasc_prefill(model, kv, seqs, B, P, ws)
        return tokens, length, (pool, bt, kv), seqs

    drafts = torch.empty((B, k), dtype=torch.int32, device=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        return reduce_over_ranks(x, "max", world, dev)

    def sum_over_ranks(x: float) -> float:
        return reduce_over_ranks(x, "sum", world, dev)

    def one_step(kvs, seqs, tokens, length):
        b.tasc_draft(drafter, tokens, length, k, cfg.lambda_num, cfg.lambda_den, out=drafts)
        return b.tasc_verify_step(model, kvs[2], seqs, drafts, ws)

    # ---- device-resident timing: `value`.  One step (draft + verify, ~5 launches per layer) is captured into a
    # CUDA graph after the warm-up and replayed K times; the state (tokens, lengths, KV) lives on the device,
    # so the replays decode on exactly as separate launches would.
    tokens, length, kvs, seqs = fresh_state()
    for _ in range(args.warmup):
        one_step(kvs, seqs, tokens, length)
    b.tasc_poll_status(ws)
    graph, launches_per_step = None, None
    if not args.no_graph:
        cap_stream = torch.cuda.Stream(device=dev)
        cap_stream.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(cap_stream):
            c0 = sum(b.tasc_launch_counts().values())
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=cap_stream):
                one_step(kvs, seqs, tokens, length)
            launches_per_step = sum(b.tasc_launch_counts().values()) - c0      # kernels recorded in the graph
        torch.cuda.current_stream().wait_stream(cap_stream)
        torch.cuda.synchronize()
    run_step = (lambda: graph.replay()) if graph is not None else (lambda: one_step(kvs, seqs, tokens, length))
    len0 = length.clone()
    launches0 = sum(b.tasc_launch_counts().values())
    sampler = ClockSampler(local_rank)
    sampler.start()
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.mark_begin()
    ev0.record()
    for _ in range(args.steps):
        run_step()
    ev1.record()
    barrier()
    sampler.mark_end()
    clocks = sampler.stop()
    launches = (launches_per_step * args.steps) if graph is not None else sum(b.tasc_launch_counts().values()) - launches0
    b.tasc_poll_status(ws)
    ms = max_over_ranks(ev0.elapsed_time(ev1))
    committed = float((length - len0).sum().item())
    committed_all = sum_over_ranks(committed)
    value = committed_all / (ms * 1e-3)
    ctx_mid = (len0.float().mean().item() + length.float().mean().item()) / 2

    if args.only_timed:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "ms_per_step": ms / args.steps, "steps": args.steps,
                              "warmup": args.warmup, "gpu_launches": int(launches), "only_timed": True}), flush=True)
        return

    # ---- per-kernel timing of the same steps in a separate, instrumented pass (events around every launch)
    b.tasc_profile_enable(True)
    b.tasc_profile_read()
    for _ in range(args.steps):
        one_step(kvs, seqs, tokens, length)
    prof = b.tasc_profile_read()
    b.tasc_profile_enable(False)
    peaks = load_peaks()
    M = B * (k + 1)
    gemm_ms = prof["gemm"][0] + prof["gemm_lm_head_argmax"][0]
    gemm_launches = prof["gemm"][1] + prof["gemm_lm_head_argmax"][1]
    gemm_bytes = gemm_bytes_per_step(shape, M) * args.steps
    achieved = gemm_bytes / (gemm_ms * 1e-3) / 1e9 if gemm_ms > 0 else 0.0
    wbytes, kvbytes = step_bytes(shape, B, k, [ctx_mid] * B)
    step_gbs = (wbytes + kvbytes) / (ms / args.steps * 1e-3) / 1e9
    roofline = {
        "bound": "hbm", "kernel": "gemm_fused_kernel (tcgen05 + TMA, cluster split-K, fused epilogues; 4 launches per layer + LM head)",
        "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
        "traffic": (NCU_TRAFFIC["bytes_per_launch"] if (cfg.index, B, k) == NCU_TRAFFIC["workload"]
                    and kernel_digest() == NCU_TRAFFIC["kernel_sha256_16"] else None),
        "peak_source": peaks["source"],
        "bytes_per_launch_avg": gemm_bytes / max(gemm_launches, 1), "us_per_launch_avg": gemm_ms * 1e3 / max(gemm_launches, 1),
        "launches": gemm_launches,
        "verify_step": {"bytes_per_step": wbytes + kvbytes, "weight_bytes": wbytes, "kv_bytes": kvbytes,
                        "achieved_gbs": step_gbs, "frac_of_measured_peak": step_gbs / peaks["hbm_gbs"],
                        "frac_of_nominal_8000": step_gbs / 8000.0},
        "kernel_ms_share": {kname: round(v[0] / max(sum(x[0] for x in prof.values()), 1e-9), 4) for kname, v in prof.items() if v[1]},
    }

    # ---- end to end: host token buffers in pinned memory, copied in and results copied out every step
    tokens, length, kvs, seqs = fresh_state()
    h_tokens = torch.zeros((B, stride), dtype=torch.int32).pin_memory()
    h_tokens[:, :P] = torch.from_numpy(prompts)
    h_len = torch.full((B,), P, dtype=torch.int32).pin_memory()
    h_acc = torch.zeros(B, dtype=torch.int32).pin_memory()
    h_next = torch.zeros(B, dtype=torch.int32).pin_memory()
    h_drafts = torch.zeros((B, k), dtype=torch.int32).pin_memory()

    # the step itself is the same captured graph as in the device-resident timing (fresh buffers, so a fresh capture)
    e2e_graph = None
    if not args.no_graph:
        for _ in range(2):
            one_step(kvs, seqs, tokens, length)
        cap_stream = torch.cuda.Stream(device=dev)
        cap_stream.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(cap_stream):
            e2e_graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(e2e_graph, stream=cap_stream):
                e2e_out = one_step(kvs, seqs, tokens, length)
        torch.cuda.current_stream().wait_stream(cap_stream)
        torch.cuda.synchronize()
    np_tokens, np_len = h_tokens.numpy(), h_len.numpy()        # views of the pinned buffers
    np_acc, np_next, np_drafts = h_acc.numpy(), h_next.numpy(), h_drafts.numpy()
    rows_idx = np.arange(B)

    def e2e_step():
        tokens.copy_(h_tokens, non_blocking=True)
        length.copy_(h_len, non_blocking=True)
        if e2e_graph is not None:
            e2e_graph.replay()
            n_acc, nxt = e2e_out[0], e2e_out[1]
        else:
            n_acc, nxt, _, _ = one_step(kvs, seqs, tokens, length)
        h_acc.copy_(n_acc, non_blocking=True)
        h_next.copy_(nxt, non_blocking=True)
        h_drafts.copy_(drafts, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        for j in range(k):                       # host-side commit of the step's result: accepted drafts, then the next token
            sel = np_acc > j
            np_tokens[rows_idx[sel], np_len[sel] + j] = np_drafts[sel, j]
        np_tokens[rows_idx, np_len + np_acc] = np_next
        np.add(np_len, np_acc + 1, out=np_len)

    for _ in range(args.warmup):
        e2e_step()
    len0_h = h_len.clone()
    barrier()
    ev0.record()
    for _ in range(args.steps):
        e2e_step()
    ev1.record()
    barrier()
    ms_e2e = max_over_ranks(ev0.elapsed_time(ev1))
    e2e_val = sum_over_ranks(float((h_len - len0_h).sum().item())) / (ms_e2e * 1e-3)
    e2e = {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": int(h_tokens.numel() * 4 + h_len.numel() * 4),
           "d2h_bytes_per_step": int((h_acc.numel() + h_next.numel() + h_drafts.numel()) * 4)}

    # ---- whole-loop generation through tasc_generate (prefill + decode, device-side loop control)
    gen = {}
    if rank == 0:
        def run_generate(mode, forced_accept=0, cont=None, max_new=cfg.max_new):
            gstride = P + max_new + k + 2
            gt = torch.zeros((B, gstride), dtype=torch.int32, device=dev)
            gt[:, :P] = torch.from_numpy(prompts).to(dev)
            gl = torch.full((B,), P, dtype=torch.int32, device=dev)
            gpool, gbt, gkv = model.new_kv(B, gstride + b.MAX_ROWS, dev)
            gen_stream = torch.cuda.Stream(device=dev)              # not the default stream: the loop replays a CUDA graph
            gen_stream.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(gen_stream):
                _, st = b.tasc_generate(model, drafter, gkv, b.make_seqs(gt, gl), B, max_new, k, ws, lambda_num=cfg.lambda_num,
                                        lambda_den=cfg.lambda_den, mode=mode, forced_accept=forced_accept, continuation=cont)
            torch.cuda.current_stream().wait_stream(gen_stream)
            hist = list(st.accepted_hist)[:k + 1]
            seq_steps = max(sum(hist), 1)
            return {"tokens_per_s": B * max_new / (st.decode_ms * 1e-3), "decode_ms": st.decode_ms, "prefill_ms": st.prefill_ms,
                    "steps": st.steps, "mean_committed_per_step": st.committed / seq_steps, "accepted_hist": hist}
        gen["greedy"] = run_generate(b.MODE_GREEDY)
        if not cfg.n_merged_tokens:          # held-out continuations are generated in the base vocabulary
            cont = torch.from_numpy(corpus.make_continuations(cfg, prompts, cfg.max_new + k + 1)).to(dev)
            gen["teacher_forced_continuation"] = run_generate(b.MODE_CONTINUATION, cont=cont)
        if args.sweep:
            gen["forced_accept_sweep"] = {str(a): run_generate(b.MODE_FORCED_ACCEPT, forced_accept=a) for a in range(k + 1)}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, cores, desc, _ = oracle_sample(cfg, 2, 12, k, prompts_all[:2])
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if shape.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": f"config {cfg.index} ({cfg.name}): B={B} per GPU, k={k}, n_max={cfg.n_max}, prompt {P}, "
                                   f"context {int(len0.float().mean().item())}->{int(length.float().mean().item())}, real greedy targets",
                       "launch": "one CUDA graph replay per step" if graph is not None else "host launches",
                       "l2": "inputs larger than L2: weights %.0f MB are streamed once per step" % (wbytes / 1e6),
                       "parallelism": "replicas only (independent batches per GPU, no collective)" if world > 1 else "single GPU"},
            "mean_committed_per_step": committed_all / (args.steps * B * world),
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
            "generate": gen, "drafter_build": build_report,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
