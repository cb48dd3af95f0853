#!/usr/bin/env python
"""Benchmark of the speculative-decoding hot path: one step = draft k tokens per sequence (n-gram
drafter) + verify the k+1 rows in one forward + greedy accept/commit, for one batch.

    python bench.py --gpus 1 --steps 64 --warmup 8
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference          (the CPU oracle on a bounded sample of the same workload)

Prints ONE JSON line.  Headline workload: configuration 4 (1.5B shape, bf16, the largest configuration) at
batch 1, k = 6, prompts of 1,024 tokens, synthetic corpus / prompts / random-init weights.  The K timed
steps are the first K steps of the generation (they start at the end of the prefilled prompt), replayed
from one CUDA graph.  `value` = tokens committed by all sequences on all ranks per second of device time
over those steps (prefill excluded, inputs resident in HBM); `e2e` = the same steps with the token
buffers copied from pinned host memory and the results read back inside the timed region.
`roofline` is the whole verify step: its algorithmic bytes (every weight once, every live KV byte once,
the new KV rows) or its 2 P M flops, whichever bound is the slower, over the replayed step time.
`workloads` carries the same figures for the other batch sizes and configurations (device-resident
timing only), `generate` the whole workload through tasc_generate.
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


# DRAM traffic of the fused GEMM kernel from an ncu capture (dram__bytes_read.sum + dram__bytes_write.sum summed
# over the step's launches of that kernel, per launch), keyed by (configuration, batch, k).  A figure is valid for
# the kernel source whose digest is stored with it; after any change of gemm_fused.cu `traffic` reads null.
NCU_TRAFFIC = {
    # configuration 4, B = 1, k = 6: per layer 6.48 + 4.92 + 55.21 + 28.20 MB (QKV, O, gate/up, down) and 469.8 MB for the LM
    # head, captured on the same kernels with the model cut to 2 layers (--layers 2) and summed for 28 layers, over the
    # step's 113 launches (algorithmic: 27.55 MB per launch)
    (4, 1, 6): {"bytes_per_launch": (28 * 94798336 + 470330624) / 113, "kernel_sha256_16": "73c53c5da55f6b57"},
}


def kernel_digest():
    import hashlib
    path = os.path.join(ROOT, "paper_2602_24174_b200", "csrc", "gemm_fused.cu")
    return hashlib.sha256(open(path, "rb").read()).hexdigest()[:16]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured (MEASURED_PEAKS.json)"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback (an earlier measurement of the same GPU type)"}


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
def oracle_sample(cfg, B_sample, n_steps, k, prompts, host_w=None):
    """Times the CPU oracle (as it stands) on a bounded sample: B_sample sequences, prompt prefilled,
    n_steps speculative steps each.  Returns (tokens/s over the decode steps, threads used, description)."""
    from oracle import decode as G, drafter as D
    from oracle.model import OracleModel
    tokens, offsets = corpus.make_corpus(cfg, n_docs=min(cfg.corpus.n_docs, 20000))
    ng = D.build_corpus_ngrams_sorted(tokens, offsets, cfg.n_max, cfg.p_min, cfg.model.vocab)
    om = OracleModel(cfg.model, host_w if host_w is not None else W.make_weights(cfg.model, cfg.seed_weights), np.float32)
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
    n = max(1, min(args.steps, 8 if cfg.model.matmul_params() > 1e9 else 16))
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
def roofline_of_step(shape, B, k, ctx_mean, ms_step, peaks):
    """The verify step against its roofline: HBM (algorithmic bytes over the measured copy bandwidth) or tensor
    (2 P M flops over the sustained bf16 rate), whichever takes longer."""
    wbytes, kvbytes = step_bytes(shape, B, k, [ctx_mean] * B)
    M = B * (k + 1)
    flops = 2.0 * shape.matmul_params() * M
    t_mem = (wbytes + kvbytes) / (peaks["hbm_gbs"] * 1e9)
    t_tc = flops / (peaks["bf16_tflops_sustained"] * 1e12)
    t = ms_step * 1e-3
    if t_tc > t_mem:
        bound, achieved, peak, unit = "tensor", flops / t / 1e12, peaks["bf16_tflops_sustained"], "TFLOP/s"
    else:
        bound, achieved, peak, unit = "hbm", (wbytes + kvbytes) / t / 1e9, peaks["hbm_gbs"], "GB/s"
    return {"bound": bound, "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak,
            "bytes_per_step": wbytes + kvbytes, "weight_bytes": wbytes, "kv_bytes": kvbytes, "flops_per_step": flops,
            "rows": M, "roofline_us": max(t_mem, t_tc) * 1e6, "hbm_us": t_mem * 1e6, "tensor_us": t_tc * 1e6,
            "achieved_hbm_gbs": (wbytes + kvbytes) / t / 1e9, "frac_of_nominal_8000_gbs": (wbytes + kvbytes) / t / 8e12}


class Task:
    """One configuration on one device: weights, model handle, corpus tables, prompts."""

    def __init__(self, b, cfg, dev, n_prompts, corpus_docs=None, keep_host_weights=False):
        import torch
        self.b, self.cfg, self.dev = b, cfg, dev
        shape = cfg.model
        host_w = W.make_weights(shape, cfg.seed_weights)
        ctoks, coffs = corpus.make_corpus(cfg, n_docs=corpus_docs)
        prompts_all = corpus.make_prompts(cfg, n_prompts)
        dev_w = b.weights_to_device(host_w, shape.dtype, dev)
        self.tokenizer = None
        if cfg.n_merged_tokens:
            # configuration 3: the vocabulary is enriched on the device (Algorithm 1 of the paper on the first 20,000
            # documents, n-grams of up to 4 tokens), the new embedding / LM-head rows are the means of their constituents,
            # and corpus and prompts are re-encoded by longest match with the added tokens first
            from dataclasses import replace
            base = shape.vocab
            sel = min(len(coffs) - 1, 20000)
            t0 = time.perf_counter()
            merges, _, _ = b.tasc_tok_enrich(torch.from_numpy(ctoks[:coffs[sel]]).to(dev), torch.from_numpy(coffs[:sel + 1]).to(dev),
                                             base, cfg.n_merged_tokens, 4)
            torch.cuda.synchronize()
            t_enrich = time.perf_counter() - t0
            rows = b.tasc_tok_init_rows(dev_w["embed"], merges)
            tied = dev_w["lm_head"] is dev_w["embed"]
            lm_rows = rows if tied else b.tasc_tok_init_rows(dev_w["lm_head"], merges)
            dev_w["embed"] = torch.cat([dev_w["embed"], rows]).contiguous()
            dev_w["lm_head"] = dev_w["embed"] if tied else torch.cat([dev_w["lm_head"], lm_rows]).contiguous()
            n_before = int(ctoks.size)
            enc_t, enc_o = b.tasc_tok_encode(torch.from_numpy(ctoks).to(dev), torch.from_numpy(coffs).to(dev), base, merges)
            ctoks, coffs = enc_t.cpu().numpy(), enc_o.cpu().numpy()
            P0 = prompts_all.shape[1]
            p_t, p_o = b.tasc_tok_encode(torch.from_numpy(prompts_all.reshape(-1).astype(np.int32)).to(dev),
                                         torch.arange(0, prompts_all.size + 1, P0, dtype=torch.int64, device=dev), base, merges)
            p_t, p_o = p_t.cpu().numpy(), p_o.cpu().numpy()
            plen = int(np.diff(p_o).min())
            prompts_all = np.stack([p_t[p_o[i]:p_o[i] + plen] for i in range(prompts_all.shape[0])]).astype(np.int32)
            shape = replace(shape, vocab=base + int(merges.shape[0]))
            self.tokenizer = {"added_tokens": int(merges.shape[0]), "enrich_s": t_enrich, "selection_documents": sel,
                              "corpus_tokens_before": n_before, "corpus_tokens_after": int(ctoks.size),
                              "compression": n_before / max(int(ctoks.size), 1)}
            host_w = None
        self.shape, self.prompts_all = shape, prompts_all
        self.model = b.Model(shape, dev_w, max_positions=cfg.prompt_len + cfg.max_new + 4096, page_size=cfg.page_size)
        self.host_w = host_w if keep_host_weights else None
        del host_w
        # the corpus tables (once per task): built once untimed (allocator, module load), then timed with the corpus resident
        d_ctoks, d_coffs = torch.from_numpy(ctoks).to(dev), torch.from_numpy(coffs).to(dev)
        # the output variability of the task corpus (Section 3 of the paper), reported next to the speed figures
        self.corpus_stats = b.tasc_corpus_stats(d_ctoks, d_coffs, shape.vocab)
        drafter = b.tasc_drafter_build(d_ctoks, d_coffs, cfg.n_max, cfg.p_min, shape.vocab)
        del drafter
        torch.cuda.synchronize()
        t_build = time.perf_counter()
        self.drafter = b.tasc_drafter_build(d_ctoks, d_coffs, cfg.n_max, cfg.p_min, shape.vocab)
        torch.cuda.synchronize()
        t_build = time.perf_counter() - t_build
        n_updates = int(sum(np.maximum(np.diff(coffs) - n, 0).sum() for n in range(1, cfg.n_max + 1)))
        self.build_report = {"ms": t_build * 1e3, "corpus_tokens": int(ctoks.size), "documents": int(coffs.size - 1),
                             "count_updates": n_updates, "updates_per_s": n_updates / t_build,
                             "timed": "host wall clock around tasc_drafter_build"}


class Window:
    """K speculative steps of one batch, starting at the end of the prefilled prompts, one CUDA graph replay per step."""

    def __init__(self, task, prompts, k, warmup, steps, use_graph=True):
        import torch
        b, cfg, dev = task.b, task.cfg, task.dev
        self.task, self.k, self.steps = task, k, steps
        self.B, self.P = prompts.shape
        B, P = self.B, self.P
        self.stride = P + (max(warmup, steps) + 4) * (k + 1) + k + 2
        if self.stride > 12288:
            raise SystemExit("too many steps for one token buffer")
        self.ws = task.model.new_workspace(B, k, dev)
        self.tokens = torch.zeros((B, self.stride), dtype=torch.int32, device=dev)
        self.tokens[:, :P] = torch.from_numpy(prompts).to(dev)
        self.length = torch.full((B,), P, dtype=torch.int32, device=dev)
        self.kvs = task.model.new_kv(B, self.stride + b.MAX_ROWS, dev)
        self.seqs = b.make_seqs(self.tokens, self.length)
        self.drafts = torch.empty((B, k), dtype=torch.int32, device=dev)
        b.tasc_prefill(task.model, self.kvs[2], self.seqs, B, P, self.ws)       # first call: plans, attributes
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        b.tasc_prefill(task.model, self.kvs[2], self.seqs, B, P, self.ws)       # the same prompts again, timed
        e1.record()
        torch.cuda.synchronize()
        self.prefill_ms = e0.elapsed_time(e1)
        for _ in range(warmup):
            self.one_step()
        b.tasc_poll_status(self.ws)
        self.graph, self.launches_per_step, self.out = None, None, None
        if use_graph:
            cap_stream = torch.cuda.Stream(device=dev)
            cap_stream.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(cap_stream):
                c0 = sum(b.tasc_launch_counts().values())
                self.graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(self.graph, stream=cap_stream):
                    self.out = self.one_step()
                self.launches_per_step = sum(b.tasc_launch_counts().values()) - c0      # kernels recorded in the graph
            torch.cuda.current_stream().wait_stream(cap_stream)
            torch.cuda.synchronize()
        self.rewind()

    def one_step(self):
        b, t = self.task.b, self.task
        b.tasc_draft(t.drafter, self.tokens, self.length, self.k, t.cfg.lambda_num, t.cfg.lambda_den, out=self.drafts)
        return b.tasc_verify_step(t.model, self.kvs[2], self.seqs, self.drafts, self.ws)

    def rewind(self):
        """Back to the end of the prompt: the cache keeps the prompt's K/V (steps only write positions from P-1 on)."""
        self.length.fill_(self.P)

    def run_step(self):
        if self.graph is not None:
            self.graph.replay()
            return self.out
        return self.one_step()


def time_window(win, steps, barrier, reduce_max, sampler=None):
    import torch
    b = win.task.b
    win.rewind()
    launches0 = sum(b.tasc_launch_counts().values())
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if sampler:
        sampler.mark_begin()
    ev0.record()
    for _ in range(steps):
        win.run_step()
    ev1.record()
    barrier()
    if sampler:
        sampler.mark_end()
    b.tasc_poll_status(win.ws)
    ms = reduce_max(ev0.elapsed_time(ev1))
    launches = win.launches_per_step * steps if win.graph is not None else sum(b.tasc_launch_counts().values()) - launches0
    committed = float((win.length - win.P).sum().item())
    ctx_mid = win.P + committed / win.B / 2
    return ms, committed, ctx_mid, int(launches)


def kernel_shares(win, steps=6):
    """Share of each kind of kernel in the step, from a separate pass with an event pair around every launch (the
    pairs serialise the launches, so only the shares are used, never the absolute times)."""
    b = win.task.b
    win.rewind()
    b.tasc_profile_enable(True)
    b.tasc_profile_read()
    for _ in range(steps):
        win.one_step()
    prof = b.tasc_profile_read()
    b.tasc_profile_enable(False)
    total = max(sum(v[0] for v in prof.values()), 1e-9)
    return {name: {"share": round(v[0] / total, 4), "launches_per_step": v[1] / steps} for name, v in prof.items() if v[1]}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=4)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--k", type=int, default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--only-timed", action="store_true",
                    help="device-resident timed region only (no per-kernel pass, e2e, generate, other workloads or CPU legs): the command ncu wraps")
    ap.add_argument("--sweep", action="store_true", help="also report the teacher-forced acceptance sweep (forced a = 0..k)")
    ap.add_argument("--lambda-sweep", action="store_true",
                    help="also report the mixing-weight sweep (teacher-forced continuation mode) and the model-derived bigram drafter")
    ap.add_argument("--no-graph", action="store_true", help="launch every step's kernels from the host instead of replaying a CUDA graph")
    ap.add_argument("--corpus-docs", type=int, default=None, help="build the drafter from the first N corpus documents only")
    ap.add_argument("--layers", type=int, default=None,
                    help="run the configuration with this many layers only (a small case of the same kernels for profiler captures)")
    ap.add_argument("--no-workloads", action="store_true", help="skip the sub-records for the other batch sizes and configurations")
    args = ap.parse_args()
    cfg = configs.get(args.config)
    if args.layers:
        cfg = configs.shrunk(cfg, n_layers=args.layers)
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
    peaks = load_peaks()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    reduce_max = lambda x: reduce_over_ranks(x, "max", world, dev)
    reduce_sum = lambda x: reduce_over_ranks(x, "sum", world, dev)

    # ---- inputs (seeded, synthetic); every rank is an independent replica with its own prompts
    want_cpu = rank == 0 and world == 1 and not args.no_cpu_baseline and not args.only_timed
    task = Task(b, cfg, dev, B * world, args.corpus_docs, keep_host_weights=want_cpu)
    shape = task.shape
    prompts = shard_prompts(task.prompts_all, rank, B)
    P = prompts.shape[1]

    # ---- device-resident timing: `value`.  One step (draft + verify, ~5 launches per layer) is captured into a CUDA
    # graph after the warm-up and replayed K times from the end of the prompt; tokens, lengths and KV live on the device.
    win = Window(task, prompts, k, args.warmup, args.steps, use_graph=not args.no_graph)
    sampler = ClockSampler(local_rank)
    sampler.start()
    ms, committed, ctx_mid, launches = time_window(win, args.steps, barrier, reduce_max, sampler)
    clocks = sampler.stop()
    committed_all = reduce_sum(committed)
    value = committed_all / (ms * 1e-3)
    ms_step = ms / args.steps

    if args.only_timed:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "ms_per_step": ms_step, "steps": args.steps,
                              "warmup": args.warmup, "gpu_launches": launches, "only_timed": True}), flush=True)
        return

    roofline = roofline_of_step(shape, B, k, ctx_mid, ms_step, peaks)
    roofline["peak_source"] = peaks["source"]
    roofline["what"] = "whole verify step (draft, embedding, %d layers x 5 kernels, LM head + argmax, accept), graph-replayed" % shape.n_layers
    shares = kernel_shares(win)
    M = B * (k + 1)
    gemm_share = sum(shares[n]["share"] for n in ("gemm", "gemm_lm_head_argmax") if n in shares)
    gemm_launches = sum(shares[n]["launches_per_step"] for n in ("gemm", "gemm_lm_head_argmax") if n in shares)
    gemm_bytes = gemm_bytes_per_step(shape, M)
    gemm_us = gemm_share * ms_step * 1e3
    traffic = NCU_TRAFFIC.get((cfg.index, B, k))
    roofline["traffic"] = traffic["bytes_per_launch"] if traffic and traffic["kernel_sha256_16"] == kernel_digest() else None
    roofline["kernel_shares"] = shares
    roofline["dominant_kernel"] = {
        "name": "gemm_fused_kernel (tcgen05 + TMA, cluster split-K, fused epilogues; 4 launches per layer + LM head)",
        "share_of_step": gemm_share, "launches_per_step": gemm_launches,
        "bytes_per_launch": gemm_bytes / max(gemm_launches, 1), "us_per_launch": gemm_us / max(gemm_launches, 1),
        "achieved_gbs": gemm_bytes / max(gemm_us, 1e-9) / 1e3, "frac": gemm_bytes / max(gemm_us, 1e-9) / 1e3 / peaks["hbm_gbs"],
        "how": "algorithmic bytes of the step's launches / (share of the step x graph-replayed step time)"}

    # ---- end to end: host token buffers in pinned memory, copied in and results copied out every step
    h_tokens = torch.zeros((B, win.stride), dtype=torch.int32).pin_memory()
    h_tokens[:, :P] = torch.from_numpy(prompts)
    h_len = torch.full((B,), P, dtype=torch.int32).pin_memory()
    h_acc = torch.zeros(B, dtype=torch.int32).pin_memory()
    h_next = torch.zeros(B, dtype=torch.int32).pin_memory()
    h_drafts = torch.zeros((B, k), dtype=torch.int32).pin_memory()
    np_tokens, np_len = h_tokens.numpy(), h_len.numpy()        # views of the pinned buffers
    np_acc, np_next, np_drafts = h_acc.numpy(), h_next.numpy(), h_drafts.numpy()
    rows_idx = np.arange(B)

    def e2e_step():
        win.tokens.copy_(h_tokens, non_blocking=True)
        win.length.copy_(h_len, non_blocking=True)
        n_acc, nxt = win.run_step()[:2]
        h_acc.copy_(n_acc, non_blocking=True)
        h_next.copy_(nxt, non_blocking=True)
        h_drafts.copy_(win.drafts, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        for j in range(k):                       # host-side commit of the step's result: accepted drafts, then the next token
            sel = np_acc > j
            np_tokens[rows_idx[sel], np_len[sel] + j] = np_drafts[sel, j]
        np_tokens[rows_idx, np_len + np_acc] = np_next
        np.add(np_len, np_acc + 1, out=np_len)

    for _ in range(args.warmup):
        e2e_step()
    h_tokens[:, P:] = 0
    h_len.fill_(P)
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        e2e_step()
    ev1.record()
    barrier()
    ms_e2e = reduce_max(ev0.elapsed_time(ev1))
    e2e_val = reduce_sum(float((h_len - P).sum().item())) / (ms_e2e * 1e-3)
    e2e = {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": int(h_tokens.numel() * 4 + h_len.numel() * 4),
           "d2h_bytes_per_step": int((h_acc.numel() + h_next.numel() + h_drafts.numel()) * 4), "ms_per_step": ms_e2e / args.steps}

    # ---- whole-loop generation through tasc_generate (prefill + decode, device-side loop control)
    gen = {}
    if rank == 0:
        def run_generate(mode, forced_accept=0, cont=None, max_new=cfg.max_new, lam=(cfg.lambda_num, cfg.lambda_den), drafter=None):
            gstride = P + max_new + k + 2
            gt = torch.zeros((B, gstride), dtype=torch.int32, device=dev)
            gt[:, :P] = torch.from_numpy(prompts).to(dev)
            gl = torch.full((B,), P, dtype=torch.int32, device=dev)
            gpool, gbt, gkv = task.model.new_kv(B, gstride + b.MAX_ROWS, dev)
            gen_stream = torch.cuda.Stream(device=dev)              # not the default stream: the loop replays a CUDA graph
            gen_stream.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(gen_stream):
                _, st = b.tasc_generate(task.model, drafter or task.drafter, gkv, b.make_seqs(gt, gl), B, max_new, k, win.ws,
                                        lambda_num=lam[0], lambda_den=lam[1], mode=mode,
                                        forced_accept=forced_accept, continuation=cont)
            torch.cuda.current_stream().wait_stream(gen_stream)
            hist = list(st.accepted_hist)[:k + 1]
            seq_steps = max(sum(hist), 1)
            # acceptance by draft position (the statistic of the paper's position-wise acceptance figure): the share of
            # sequence-steps whose accepted prefix reaches position j
            by_pos = [sum(hist[j:]) / seq_steps for j in range(1, k + 1)]
            return {"tokens_per_s": B * max_new / (st.decode_ms * 1e-3), "decode_ms": st.decode_ms, "prefill_ms": st.prefill_ms,
                    "steps": st.steps, "ms_per_step": st.decode_ms / max(st.steps, 1),
                    "mean_committed_per_step": st.committed / seq_steps, "accepted_hist": hist,
                    "acceptance_by_position": [round(x, 4) for x in by_pos]}
        gen["greedy"] = run_generate(b.MODE_GREEDY)
        if not cfg.n_merged_tokens:          # held-out continuations are generated in the base vocabulary
            cont = torch.from_numpy(corpus.make_continuations(cfg, prompts, cfg.max_new + k + 1)).to(dev)
            gen["teacher_forced_continuation"] = run_generate(b.MODE_CONTINUATION, cont=cont)
        if args.sweep:
            gen["forced_accept_sweep"] = {str(a): run_generate(b.MODE_FORCED_ACCEPT, forced_accept=a) for a in range(k + 1)}
        if args.lambda_sweep and not cfg.n_merged_tokens:
            # the mixing-weight ablation of the paper's appendix in teacher-forced continuation mode (targets = held-out
            # continuations of the corpus generator): lambda = 1 is the corpus drafter alone, lambda = 0 the context
            # drafter alone; and the model-derived bigram (the comparison drafter of Section 6.2) alone and mixed
            sweep = {}
            for num, den in ((0, 1), (1, 4), (1, 2), (3, 4), (9, 10), (1, 1)):
                sweep[f"{num}/{den}"] = run_generate(b.MODE_CONTINUATION, cont=cont, lam=(num, den))
            gen["lambda_sweep_corpus_drafter"] = sweep
            Bt = 256
            t_bigram = time.perf_counter()
            bpool, bbt, bkv = task.model.new_kv(Bt, 16, dev)
            bws = task.model.new_workspace(Bt, 1, dev)
            table = b.tasc_bigram_table(task.model, bkv, Bt, bws)
            b.tasc_poll_status(bws)
            t_bigram = time.perf_counter() - t_bigram
            bigram = b.tasc_drafter_from_bigram(table, shape.vocab)
            del bpool, bbt, bws
            gen["model_bigram_drafter"] = {
                "table_build_s": t_bigram,
                "bigram_alone": run_generate(b.MODE_CONTINUATION, cont=cont, lam=(1, 1), drafter=bigram),
                "mixed_with_context_1/256": run_generate(b.MODE_CONTINUATION, cont=cont, lam=(1, 256), drafter=bigram),
                "mixed_with_context_1/4": run_generate(b.MODE_CONTINUATION, cont=cont, lam=(1, 4), drafter=bigram)}

    cpu = None
    if want_cpu:
        n_seq, n_st = (1, 6) if shape.matmul_params() > 1e9 else (2, 12)
        # (the enriched-vocabulary configuration is timed on the base vocabulary: the oracle's step cost is the same)
        cpu_prompts = corpus.make_prompts(cfg, n_seq) if cfg.n_merged_tokens else task.prompts_all[:n_seq]
        v, cores, desc, _ = oracle_sample(cfg, n_seq, n_st, k, cpu_prompts, host_w=task.host_w)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}
    task.host_w = None

    # ---- the other workloads: same model at the configuration's other batch sizes, then the smaller configurations
    workloads = []
    if rank == 0 and world == 1 and not args.no_workloads:
        def sub_record(t, Bw, kw, steps):
            pw = corpus_prompts(t, Bw)
            w = Window(t, pw, kw, 3, steps)
            ms_w, com_w, ctx_w, _ = time_window(w, steps, barrier, lambda x: x)
            r = roofline_of_step(t.shape, Bw, kw, ctx_w, ms_w / steps, peaks)
            return {"workload": f"config {t.cfg.index} ({t.cfg.name}) B={Bw} k={kw} prompt {pw.shape[1]}", "steps": steps,
                    "ms_per_step": ms_w / steps, "tokens_per_s_window": com_w / (ms_w * 1e-3),
                    "mean_committed_per_step": com_w / (steps * Bw), "bound": r["bound"], "frac": r["frac"],
                    "achieved": r["achieved"], "unit": r["unit"], "bytes_per_step": r["bytes_per_step"], "roofline_us": r["roofline_us"],
                    "gemm_rows_per_step": Bw * (kw + 1), "prefill_ms": w.prefill_ms,
                    # the prefill runs the layers, not the LM head, over all but the last prompt token
                    "prefill_tflops": 2.0 * (t.shape.matmul_params() - t.shape.vocab * t.shape.d_model) * Bw * (pw.shape[1] - 1)
                                      / (w.prefill_ms * 1e-3) / 1e12}

        def corpus_prompts(t, Bw):
            if t.prompts_all.shape[0] >= Bw:
                return t.prompts_all[:Bw]
            return corpus.make_prompts(t.cfg, Bw)
        for Bw in (16, 64):
            if cfg.index == 4 and Bw != B:
                workloads.append(sub_record(task, Bw, k, 48))
        del win
        for ci, runs in ((2, ((1, 5), (8, 5), (32, 5), (32, 8))), (1, ((1, 5), (16, 5)))):
            if ci == cfg.index:
                continue
            c = configs.get(ci)
            t = Task(b, c, dev, max(Bw for Bw, _ in runs), corpus_docs=min(c.corpus.n_docs, 50000))
            for Bw, kw in runs:
                workloads.append(sub_record(t, Bw, kw, 64))
            del t
            torch.cuda.empty_cache()

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if shape.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": f"config {cfg.index} ({cfg.name}{', cut to %d layers' % args.layers if args.layers else ''}): B={B} per GPU, k={k}, n_max={cfg.n_max}, prompt {P}, "
                                   f"the first {args.steps} steps after the prompt (context {P}->{int(2 * ctx_mid - P)}), real greedy targets, "
                                   f"corpus tables from {task.build_report['documents']} documents",
                       "launch": "one CUDA graph replay per step" if win_graph(args) else "host launches",
                       "l2": "inputs larger than L2: weights %.0f MB are streamed once per step" % (roofline["weight_bytes"] / 1e6),
                       "parallelism": "replicas only (independent batches per GPU, no collective)" if world > 1 else "single GPU"},
            "mean_committed_per_step": committed_all / (args.steps * B * world),
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches, "clocks": clocks,
            "generate": gen, "drafter_build": task.build_report, "corpus_statistics": task.corpus_stats,
            "tokenizer_enrichment": task.tokenizer, "workloads": workloads,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def win_graph(args):
    return not args.no_graph


if __name__ == "__main__":
    main()
