#!/usr/bin/env python
"""Step time of san_decode_step on one workload, per kernel and per part of the step.

    python paper_1906_11024_b200/microbench/step_kernels.py --workload base \
        --select 1 --select 2 --select 2,0,2,64,0,1 [--parts both,self,enc] [--n-seqs 1,32,128,256]

Each --select is the argument list of san_step_kernel_select (kernel, spans_log2, heads per unit,
tile positions, layers per unit, grab multiplier; omitted values are the defaults).  "self" times
the step with no sentence in it, "enc" with no sequence; --n-seqs times the self-attention part
alone on the first n sequences (what a launch costs when almost nothing is in it).  Steps are
captured into a CUDA graph rotating over independent replicas of the device state, as in bench.py.
"""
from __future__ import annotations

import argparse
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="base")
    ap.add_argument("--select", action="append", default=[])
    ap.add_argument("--parts", default="both,self,enc")
    ap.add_argument("--n-seqs", default="")
    ap.add_argument("--replicas", type=int, default=6)
    ap.add_argument("--reps", type=int, default=300)
    ap.add_argument("--unshared", action="store_true", help="every block one layer (sharing off)")
    args = ap.parse_args()

    import torch
    import bench
    from paper_1906_11024_b200 import binding as B
    from paper_1906_11024_b200 import build as san_build
    from paper_1906_11024_b200 import synth
    san_build.build()
    B.lib()
    dev = torch.device("cuda:0")
    w = synth.WORKLOADS[args.workload]
    if args.unshared:
        w = synth.unshared(w)
    decs, sbs, _ = bench.build_replicas(w, args.replicas, dev)
    R = len(decs)

    def timed(n_seqs, n_sent):
        def one(r):
            d, sb = decs[r], sbs[r]
            kw = dict(d_seq_ids=sb.ids, n_seqs=n_seqs, max_len=sb.max_len, d_O_self=sb.O_self, d_q_enc=sb.q_enc,
                      d_sent_ids=sb.sent_ids, d_src_lens=sb.src_lens, n_sent=n_sent, max_src=sb.max_src, d_S_enc=sb.S_enc,
                      ld_s=d.ld_s, d_O_enc=sb.O_enc)
            if w.self_is_aan:
                kw.update(d_x_aan=sb.x_aan, d_t=sb.t_aan)
            else:
                kw.update(d_q_self=sb.q_self, d_k_new=sb.k_new, d_v_new=sb.v_new, d_pos=sb.pos, d_S_self=sb.S_self, ld_t=d.ld_t)
            B.check(B.san_decode_step(d.ctx, **kw), "san_decode_step")
        g = bench.capture(lambda: [one(r) for r in range(R)], dev)
        for _ in range(5):
            g.replay()
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.reps):
            g.replay()
        e1.record()
        torch.cuda.synchronize(dev)
        used = B.san_step_kernel_used(decs[0].ctx)
        return e0.elapsed_time(e1) * 1e3 / (args.reps * R), used[1], used[2]

    n, n_sent = w.n_seqs, w.n_sent
    for sel in args.select or ["0"]:
        vals = [int(x) for x in sel.split(",")]
        for d in decs:
            B.check(B.san_step_kernel_select(d.ctx, *vals), "san_step_kernel_select")
        for part in [p for p in args.parts.split(",") if p]:
            us, which, rpu = timed(n if part != "enc" else 0, n_sent if part != "self" else 0)
            print(f"{w.name} select {sel:>16s} {part:>4s}: {us:7.2f} us  (kernel {which}, heads per unit {rpu})", flush=True)
        for k in [int(x) for x in args.n_seqs.split(",") if x]:
            us, which, rpu = timed(min(k, n), 0)
            print(f"{w.name} select {sel:>16s} self-attention of {min(k, n):4d} sequences alone: {us:7.2f} us  (kernel {which})", flush=True)
        err = [d.device_status()[0] for d in decs]
        assert not any(err), err


if __name__ == "__main__":
    main()
