"""Critical path of one speculative step from per-CTA time stamps.

    python -m paper_2602_24174_b200.build --timeline
    python -m paper_2602_24174_b200.timeline --config 1 --batch 16

The instrumented library (same sources, -DTASC_TIMELINE) appends one record per CTA of the fused GEMM and the
attention kernels: start, end and up to six intermediate stamps on the GPU's global nanosecond timer.  One step
(draft + verify) is captured in a CUDA graph, replayed, and the records are grouped into kernels; for every kind
of kernel the table gives the time from the end of its predecessor to its own end ("period", the kernel's share
of the step's critical path) and where it goes.  Synthetic seeded inputs; a development aid, not a benchmark.
"""
from __future__ import annotations

import argparse
import collections
import ctypes as C
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

NAMES = {0: "plain", 1: "qkv", 2: "resid", 3: "swiglu", 4: "lm", 10: "attn"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=1)
    ap.add_argument("--batch", type=int, default=16)
    ap.add_argument("--prompt-len", type=int, default=None)
    ap.add_argument("--corpus-docs", type=int, default=5000)
    args = ap.parse_args()
    import paper_2602_24174_b200 as pkg
    pkg.LIBRARY_FILE = "libtasc_timeline.so"                   # before the binding is imported
    from paper_2602_24174_b200 import binding as b
    if not hasattr(b.lib, "tasc_debug_ctalog"):
        raise SystemExit("libtasc_timeline.so has no time stamps: rebuild it with `python -m paper_2602_24174_b200.build --timeline`")
    from workload import configs, corpus, weights as W
    cfg = configs.get(args.config)
    shape, k, B = cfg.model, cfg.k, args.batch
    dev = torch.device("cuda")
    model = b.Model(shape, b.weights_to_device(W.make_weights(shape, cfg.seed_weights), shape.dtype, dev),
                    max_positions=cfg.prompt_len + 4096, page_size=cfg.page_size)
    ct, co = corpus.make_corpus(cfg, n_docs=args.corpus_docs)
    drafter = b.tasc_drafter_build(torch.from_numpy(ct).to(dev), torch.from_numpy(co).to(dev), cfg.n_max, cfg.p_min, shape.vocab)
    prompts = corpus.make_prompts(cfg, B, prompt_len=args.prompt_len or cfg.prompt_len)
    P = prompts.shape[1]
    stride = P + 40 * (k + 1)
    tokens = torch.zeros((B, stride), dtype=torch.int32, device=dev)
    tokens[:, :P] = torch.from_numpy(prompts).to(dev)
    length = torch.full((B,), P, dtype=torch.int32, device=dev)
    pool, bt, kv = model.new_kv(B, stride + b.MAX_ROWS, dev)
    ws = model.new_workspace(B, k, dev)
    seqs = b.make_seqs(tokens, length)
    b.tasc_prefill(model, kv, seqs, B, P, ws)
    b.tasc_poll_status(ws)
    drafts = torch.empty((B, k), dtype=torch.int32, device=dev)

    def step():
        b.tasc_draft(drafter, tokens, length, k, cfg.lambda_num, cfg.lambda_den, out=drafts)
        b.tasc_verify_step(model, kv, seqs, drafts, ws)

    graph, stream = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    with torch.cuda.stream(stream):
        step(); step()
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=stream):
            step()
    torch.cuda.synchronize()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    b.lib.tasc_debug_ctalog.argtypes = [C.c_void_p, C.c_int, C.c_int]
    cap = 1 << 18
    buf = np.zeros((cap, 10), dtype=np.uint64)       # t0, t1, ta..tf, (tag, x), (y, z)
    b.lib.tasc_debug_ctalog(buf.ctypes.data, cap, 1)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(); graph.replay(); e1.record()
    torch.cuda.synchronize()
    n = b.lib.tasc_debug_ctalog(buf.ctypes.data, cap, 1)
    b.tasc_poll_status(ws)
    rec = buf[:n]
    t0, t1, ta, tb = (rec[:, i].astype(np.int64) for i in range(4))
    tx = [rec[:, 4 + i].astype(np.int64) for i in range(4)]
    tag = rec[:, 8:].copy().view(np.int32).reshape(n, 4)[:, 0]
    base = t0.min()
    us = lambda a: (a - base) / 1e3
    kernels, cur = [], None
    # a CTA leaves only after its grid's predecessor has finished, so end times (not start times: grids start ahead of
    # one another) separate the kernels of the chain; consecutive kernels have different tags
    for i in np.argsort(t1):
        if cur is None or tag[i] != cur[0]:
            cur = (int(tag[i]), [])
            kernels.append(cur)
        cur[1].append(i)
    print(f"config {cfg.index} ({cfg.name}), B={B}, k={k}, context {int(length.float().mean())}: step {e0.elapsed_time(e1) * 1e3:.1f} us, "
          f"{len(kernels)} stamped kernels, {n} CTAs")
    agg = collections.defaultdict(lambda: collections.defaultdict(float))
    prev_end = base
    for tg, idx in kernels:
        ix = np.array(idx)
        wait, acc, end = us(ta[ix].max()), us(tb[ix].max()), us(t1[ix].max())
        a = agg[NAMES.get(tg, str(tg))]
        a["n"] += 1; a["ctas"] += len(ix)
        a["period"] += end - us(prev_end); a["lag"] += wait - us(prev_end); a["main"] += acc - wait; a["tail"] += end - acc
        a["lead_first"] += us(prev_end) - us(t0[ix].min()); a["lead_last"] += us(prev_end) - us(t0[ix].max())
        st = [us(x[ix].max()) for x in tx]
        if tg == 10:
            a["p0"] += st[0] - wait; a["p1"] += st[1] - st[0]; a["p2"] += acc - st[1]
        else:
            a["p0"] += st[0] - acc; a["p1"] += st[1] - st[0]; a["p2"] += st[2] - st[1]; a["p3"] += st[3] - st[2]; a["p4"] += end - st[3]
        prev_end = t1[ix].max()
    print("kind     n   CTAs | period = wait lag + main + tail   (us, means)   | detail")
    for name, a in agg.items():
        c = a["n"]
        if name == "attn":
            det = f"Q staged {a['p0']/c:.2f}, first tiles landed {a['p1']/c:.2f}, tile loop {a['p2']/c:.2f}; tail = merge/write + exit"
        else:
            det = (f"tail: TMEM->smem {a['p0']/c:.2f}, cluster barrier {a['p1']/c:.2f}, split-K pull {a['p2']/c:.2f}, "
                   f"epilogue {a['p3']/c:.2f}, leave {a['p4']/c:.2f}")
        print(f"{name:7s} {int(c):3d} {int(a['ctas']/c):5d} | {a['period']/c:6.2f} = {a['lag']/c:5.2f} + {a['main']/c:5.2f} + {a['tail']/c:5.2f} | "
              f"started {a['lead_first']/c:.1f} .. {a['lead_last']/c:.1f} before | {det}")
    print("wait lag: predecessor's end -> last CTA past griddepcontrol.wait; main: -> accumulator complete (GEMM) / key tiles done "
          "(attention); tail: -> last CTA gone; started: first .. last CTA start, microseconds before the predecessor's end")


if __name__ == "__main__":
    main()
