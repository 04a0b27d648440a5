#!/usr/bin/env python
"""Benchmark of the shared-attention decode step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload long|base|big|aan|tiny]
    python bench.py --impl reference ...          # the CPU oracle as the reference arm

The line's headline is the workload named by --workload (default: long, the single-GPU
configuration that moves most bytes per step); the other configurations are measured in
the same run with fewer steps and reported under "workloads".

A step is one decode step of the whole attention path (cache append, weights, apply for
self and encoder-decoder attention of every layer, or AAN + enc-dec) for every sequence of
the workload, at the decode run's average state (each sequence at the middle of its own
target length; the ragged configuration at its seeded prefix lengths).  Steps rotate over
several independent replicas of the device state so that consecutive steps touch disjoint
memory far larger than L2.  Prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode-step attention tokens/sec"
UNIT = "tokens/s"
L2_BYTES = 126e6
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# DRAM bytes read + written per launch of the step kernel, from ncu captures of this file's own
# command line (one workload, a dozen steps), and the digest of the sources they were taken with
# (the kernels and the host code that chooses kernel and cuts): once any of them changes the
# counters no longer describe the kernel, and the line reports null until a new capture is
# recorded here.
E2E_BATCHES = 4           # request batches in flight in the end-to-end leg
KERNEL_SOURCES = ("san_fused.cuh", "san_step.cuh", "san_rows.cuh", "san_kernels.cuh", "san_api.cu")
NCU_TRAFFIC = {"digest": "41b8c06f8c015c80",
               "fused": {"long": 734.8e6, "base": 70.2e6, "big": 426.9e6, "aan": 25.4e6,
                         "long-unshared": 1257.3e6, "base-unshared": 105.1e6}}


def kernel_digest():
    import hashlib
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_1906_11024_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def ncu_traffic(path, workload):
    if kernel_digest() != NCU_TRAFFIC["digest"]:
        return None
    return NCU_TRAFFIC.get(path, {}).get(workload)


# ------------------------------------------------------------------------------- workload state
def state_positions(w):
    """Row each sequence writes in the benchmarked step (its cache length is this + 1)."""
    T = np.repeat(w.tgt_lens(), w.beam).astype(np.int32)
    if w.ragged_prefix:
        return w.prefix_lens().astype(np.int32)
    return ((T + 1) // 2 - 1).astype(np.int32)               # middle of the run: length ceil(T/2)


def algorithmic_bytes(w, pos, fused=False):
    """Bytes the method itself must move per step (K/V reads are the roofline count).
    In the one-launch step S is written for the caller but never read back."""
    M, H, d, e = w.n_layers, w.n_heads, w.d_model, w.elem_bytes
    n = w.n_seqs
    src = w.src_lens().astype(np.int64)
    Ns, Ne = len(w.self_blocks), len(w.encdec_blocks)
    L = pos.astype(np.int64) + 1
    out = {}
    if w.self_is_aan:
        out["self_kv"] = 0
        out["aan"] = M * n * d * (2 * e + 8)
        s_self = 0
        small_self = 0
    else:
        out["self_kv"] = int((Ns + M) * L.sum() * d * e)
        out["aan"] = 0
        s_self = 8 * H * Ns * int(L.sum())
        small_self = Ns * n * d * e + M * n * d * e + (Ns + M) * n * d * e       # q, O, appended rows
    out["encdec_kv"] = int((Ne + M) * src.sum() * d * e)                          # once per sentence
    s_enc = 8 * H * Ne * int(np.repeat(src, w.beam).sum())
    small_enc = Ne * n * d * e + M * n * d * e
    out["S"] = (s_self + s_enc) // (2 if fused else 1)
    out["small"] = small_self + small_enc
    out["kv"] = out["self_kv"] + out["encdec_kv"] + out["aan"]
    out["total"] = out["kv"] + out["S"] + out["small"]
    return out


def measured_peak_gbs():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------------------------ clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        rows = [r for (t, r) in self.rows if t0 - 0.05 <= t <= t1 + 0.15] or [r for _, r in self.rows]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for nm, val in zip(names, r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------- the GPU arm
def build_replicas(w, n_rep, device, shared_context=False):
    import torch
    from paper_1906_11024_b200.driver import Decoder
    pos = state_positions(w)
    ids = np.arange(w.n_seqs, dtype=np.int32)
    decs, sbs = [], []
    for r in range(n_rep):
        dec = Decoder(w, device, encdec_shared_context=shared_context)
        gen = torch.Generator(device=device)
        gen.manual_seed(1000 + r)
        # cache contents: seeded N(0,1) in the storage dtype (the AAN running sums are float32)
        if w.self_is_aan:
            dec.cache.view(torch.float32).normal_(generator=gen)
            dec.load_encoder_memory()
        else:
            dec.cache.view(dec.tdtype).normal_(generator=gen)
        sb = dec.new_step_buffers()
        dec.fill_step_inputs(sb, r, ids, pos)
        sb.max_len = int(pos.max()) + 1
        sb.max_src = int(w.src_lens().max())
        decs.append(dec)
        sbs.append(sb)
    torch.cuda.synchronize(device)
    return decs, sbs, pos


def capture(fn, device):
    """Capture the launches fn() issues on torch's current stream into a CUDA graph."""
    import torch
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream(device)
    s.wait_stream(torch.cuda.current_stream(device))
    with torch.cuda.stream(s):
        fn()                                   # warm-up outside capture (module load, first launch)
    torch.cuda.current_stream(device).wait_stream(s)
    torch.cuda.synchronize(device)
    with torch.cuda.graph(g):
        fn()
    return g


def time_steps(decs, sbs, steps, warmup, device, barrier, fused=True):
    """W untimed + exactly K timed steps; steps rotate over the replicas.  Returns seconds."""
    import torch
    R = len(decs)
    launches = [0]

    def one(r):
        launches[0] = decs[r].step_fused(sbs[r]) if fused else decs[r].step(sbs[r])

    cycle = capture(lambda: [one(r) for r in range(R)], device)
    singles = [capture(lambda r=r: one(r), device) for r in range(max(steps % R, max(warmup, 3) % R))]

    def run(k):
        for _ in range(k // R):
            cycle.replay()
        for r in range(k % R):
            singles[r].replay()

    run(max(warmup, 3))
    barrier()
    torch.cuda.synchronize(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    e0.record()
    run(steps)
    e1.record()
    torch.cuda.synchronize(device)
    t1 = time.time()
    barrier()
    return e0.elapsed_time(e1) * 1e-3, launches[0], (t0, t1)


def time_dominant_kernel(w, decs, sbs, device, reps=20):
    """Average duration of one san_attn_apply launch over the self-attention caches (the
    kernel that moves most bytes), launches rotating over replicas and blocks."""
    import torch
    from paper_1906_11024_b200 import binding as B
    R = len(decs)
    if w.self_is_aan:
        kind, firsts, sizes = B.SAN_ENCDEC, decs[0].enc_first, decs[0].enc_sizes
    else:
        kind, firsts, sizes = B.SAN_SELF, decs[0].self_first, decs[0].self_sizes

    def launch_all():
        n = 0
        for r in range(R):
            d, sb = decs[r], sbs[r]
            for b, (first, size) in enumerate(zip(firsts, sizes)):
                if kind == B.SAN_SELF:
                    B.check(B.san_attn_apply(d.ctx, kind, b, first, first + size, sb.S_self[b], d.ld_t, sb.ids, None,
                                             sb.lens, sb.ids.shape[0], sb.max_len, sb.O_self[first], 0))
                else:
                    B.check(B.san_attn_apply(d.ctx, kind, b, first, first + size, sb.S_enc[b], d.ld_s, sb.sent_ids, None,
                                             sb.src_lens, sb.sent_ids.shape[0], sb.max_src, sb.O_enc[first], 0))
                n += 1
        return n

    count = [0]
    g = capture(lambda: count.__setitem__(0, launch_all()), device)
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize(device)
    return e0.elapsed_time(e1) * 1e-3 / (reps * count[0]), count[0] // R


def dominant_kernel_bytes(w, pos):
    """Algorithmic bytes of one san_attn_apply launch (mean over the blocks of the kind)."""
    H, d, e = w.n_heads, w.d_model, w.elem_bytes
    if w.self_is_aan:
        sizes = w.encdec_blocks
        rows = int(w.src_lens().astype(np.int64).sum())
        s_rows = int(np.repeat(w.src_lens(), w.beam).astype(np.int64).sum())
    else:
        sizes = w.self_blocks
        rows = int((pos.astype(np.int64) + 1).sum())
        s_rows = rows
    per = [pi * rows * d * e + 4 * H * s_rows + pi * w.n_seqs * d * e for pi in sizes]
    return float(np.mean(per))


def time_e2e(w, decs, sbs, steps, device, fused=True):
    """The same step with HOST buffers: every step copies its inputs from pinned host memory
    to the device, runs the library, and reads the outputs back.  On the one-launch path this
    is a single C-ABI call, san_decode_step_host, which issues the copies itself on the
    caller's stream.  A step of one request batch is a chain (copy in, kernel, copy out) that the
    next step of that batch has to wait for, so several batches (E2E_BATCHES contexts, each with its
    own stream and pinned buffers) take turns, the way a server keeps the GPU and PCIe busy in both
    directions: the copies of one batch overlap the kernels of the others.  Returns (seconds for
    `steps` steps with all batches in flight, seconds for `steps` steps of one batch alone, h2d bytes
    per step, d2h bytes per step, batches)."""
    import torch
    n_ctx = min(len(decs), E2E_BATCHES)
    hbs = [decs[i].host_buffers(sbs[i]) for i in range(n_ctx)]
    streams = [torch.cuda.Stream(device) for _ in range(n_ctx)]
    hb = hbs[0]
    lens_host = [sbs[i].lens.cpu().pin_memory() for i in range(n_ctx)]   # the separate calls take lengths, the one-launch step positions
    h2d = sum(hb[k].numel() * hb[k].element_size() for k in hb["_in"]) + (0 if fused else lens_host[0].numel() * 4)
    d2h = sum(hb[k].numel() * hb[k].element_size() for k in hb["_out"])
    dev_of = {"d_seq_ids": "ids", "d_pos": "pos", "d_sent_ids": "sent_ids", "d_src_lens": "src_lens",
              "d_q_enc": "q_enc", "d_q_self": "q_self", "d_k_new": "k_new", "d_v_new": "v_new",
              "d_x_aan": "x_aan", "d_t": "t_aan", "d_O_self": "O_self", "d_O_enc": "O_enc"}

    def one(i):
        dec, sb, hb = decs[i], sbs[i], hbs[i]
        with torch.cuda.stream(streams[i]):
            if fused:
                dec.step_fused_host(sb, hb, stream=streams[i])
                return
            for k in hb["_in"]:
                getattr(sb, dev_of[k]).copy_(hb[k], non_blocking=True)
            sb.lens.copy_(lens_host[i], non_blocking=True)
            dec.step(sb, stream=streams[i])
            for k in hb["_out"]:
                hb[k].copy_(getattr(sb, dev_of[k]), non_blocking=True)

    def timed(n_active):
        for i in range(3 * n_active):
            one(i % n_active)
        torch.cuda.synchronize(device)
        cur = torch.cuda.current_stream(device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(cur)
        for st in streams[:n_active]:
            st.wait_event(e0)
        for i in range(steps):
            one(i % n_active)
        for st in streams[:n_active]:
            cur.wait_stream(st)
        e1.record(cur)
        torch.cuda.synchronize(device)
        return e0.elapsed_time(e1) * 1e-3

    serial = timed(1)
    both = timed(n_ctx) if n_ctx > 1 else serial
    return both, serial, h2d, d2h, n_ctx


def time_beam_reorder(w, decs, sbs, pos, device, peak, reps=10):
    """The step next to the path in a beam-search decoder: san_beam_reorder, launches rotating
    over the replicas.  Two parent patterns: every beam takes over the whole history of its
    neighbour (parent = slot + 1 mod beam: every cached row of every self-attention plane moves),
    and seeded parents where half of the hypotheses continue themselves and the others pick a
    parent at random (rows of a hypothesis that keeps its parent do not move)."""
    import torch
    from paper_1906_11024_b200 import binding as B
    from paper_1906_11024_b200 import synth
    R = len(decs)
    sent = torch.arange(w.n_sent, dtype=torch.int32, device=device)
    lens_h = (pos + 1).astype(np.int32)
    lens = torch.from_numpy(lens_h).to(device).view(w.n_sent, w.beam).contiguous()
    max_len = int(pos.max()) + 1
    planes = w.n_layers if w.self_is_aan else len(w.self_blocks) + w.n_layers
    row_bytes = w.d_model * (4 if w.self_is_aan else w.elem_bytes)
    out = {}
    worst = ((np.arange(w.beam, dtype=np.int32) + 1) % w.beam)[None, :].repeat(w.n_sent, 0)
    seeded = synth.beam_parents(w, 0, keep_prob=0.5).reshape(w.n_sent, w.beam)
    for name, par in (("all_move", worst), ("half_keep", seeded)):
        parent = torch.from_numpy(np.ascontiguousarray(par, np.int32)).to(device)

        def all_replicas():
            for r in range(R):
                B.check(B.san_beam_reorder(decs[r].ctx, sent, parent, lens, w.n_sent, max_len), "san_beam_reorder")

        g = capture(all_replicas, device)
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize(device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            g.replay()
        e1.record()
        torch.cuda.synchronize(device)
        secs = e0.elapsed_time(e1) * 1e-3 / (reps * R)
        moves = (par != np.arange(w.beam)[None, :]).reshape(-1)
        rows = float(moves.sum()) if w.self_is_aan else float(lens_h[moves].sum())
        moved = planes * rows * row_bytes
        gbs = 2 * moved / secs / 1e9                  # every piece that moves is read once and written once
        out[name] = {"us_per_launch": secs * 1e6, "bytes_per_launch": 2 * moved, "achieved_gbs": gbs,
                     "frac_of_peak": gbs / peak, "share_of_slots_that_move": float(moves.mean())}
    out.update({"call": "san_beam_reorder", "bound": "hbm",
                "note": "all_move: every beam changes parent; half_keep: seeded parents, half of the hypotheses continue "
                        "themselves; launches of the AAN workload move only the running sums"})
    return out


def time_js_matrix(w, dec, sb, pos, device, reps=50):
    """Policy learner, device part: san_js_matrix over the self-attention weights that an
    unshared decode step wrote (one S per layer)."""
    import torch
    from paper_1906_11024_b200 import binding as B
    if w.self_is_aan or sb.S_self is None or sb.S_self.shape[0] < 2:
        return None
    M = sb.S_self.shape[0]
    lens = torch.from_numpy((pos + 1).astype(np.int32)).to(device)
    djs = torch.zeros(M, M, dtype=torch.float64, device=device)

    def one():
        B.check(B.san_js_matrix(M, sb.S_self, sb.S_self.stride(0), dec.ld_t, w.n_seqs, w.n_heads, lens, djs), "san_js_matrix")

    g = capture(one, device)
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize(device)
    secs = e0.elapsed_time(e1) * 1e-3 / reps
    nbytes = M * w.n_heads * int((pos.astype(np.int64) + 1).sum()) * 4
    return {"call": "san_js_matrix", "layers": M, "us_per_call": secs * 1e6, "bytes_per_call": nbytes,
            "achieved_gbs": nbytes / secs / 1e9,
            "note": "three launches (clear, pairs, finish) over weights that fit in L2; M(M-1)/2 pairs with two "
                    "logarithms per position: launch-bound for few layers, logarithm-bound for many, never HBM-bound"}


def time_full_block(w, device, peak, reps=5):
    """Full-sequence shared attention (encoder-side use): one san_full_block launch over the
    workload's sentences at their source lengths, a block of self_blocks[0] layers (AAN
    workload: encdec_blocks[0]).  Launches rotate over input replicas larger than L2."""
    import torch
    from paper_1906_11024_b200 import binding as B
    if w.dtype != "bf16":
        return None
    src = w.src_lens().astype(np.int64)
    cap = int(src.max())
    if cap > 512:
        return None
    pi = int((w.encdec_blocks if w.self_is_aan else w.self_blocks)[0])
    H, n = w.n_heads, w.n_sent
    per_rep = (2 + 2 * pi) * n * cap * H * 64 * 2
    R = int(min(32, max(2, math.ceil(3 * L2_BYTES / per_rep))))
    gen = torch.Generator(device=device)
    gen.manual_seed(77)
    mk = lambda *shape: torch.randn(*shape, generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)
    reps_in = [(mk(n, cap, H, 64), mk(n, cap, H, 64), mk(pi, n, cap, H, 64)) for _ in range(R)]
    out = torch.empty(pi, n, cap, H, 64, dtype=torch.bfloat16, device=device)
    lens = torch.from_numpy(src.astype(np.int32)).to(device)

    def all_replicas():
        for q, k, v in reps_in:
            B.check(B.san_full_block(B.SAN_BF16, H, pi, 0, q, k, v, lens, n, cap, cap, None, 0, out), "san_full_block")

    g = capture(all_replicas, device)
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize(device)
    secs = e0.elapsed_time(e1) * 1e-3 / (reps * R)
    rows = int(src.sum())
    nbytes = (2 + 2 * pi) * rows * H * 64 * 2                       # Q, K, pi value panels in; pi outputs out
    flops = float((2 + 2 * pi) * (src * src).sum() * H * 64)        # 2 l^2 d_h for the scores and per layer of S.V
    return {"call": "san_full_block", "layers_in_block": pi, "us_per_launch": secs * 1e6,
            "bytes_per_launch": nbytes, "achieved_gbs": nbytes / secs / 1e9, "frac_of_hbm_peak": nbytes / secs / 1e9 / peak,
            "flops_per_launch": flops, "achieved_tflops": flops / secs / 1e12,
            "bound": "tensor" if cap >= 128 else "hbm",
            "kernel": "full_block_tc5_kernel (tcgen05)" if cap >= 128 else "full_block_kernel (mma.sync)",
            "note": "length bound >= 128: 128-query tcgen05 tiles, flops count each product once; "
                    "below: sentences of 10-100 positions, bound by HBM and latency, not by the tensor pipe"}


# ------------------------------------------------------------------------- the CPU oracle arm
def oracle_sample(w, n_sent_sample):
    """Oracle state for the first sentences of the workload at the benchmarked positions."""
    from paper_1906_11024_b200 import synth
    from tests.helpers import OracleRun
    ws = synth.scaled(w, min(n_sent_sample, w.n_sent), w.name + "-sample")
    orc = OracleRun(ws)
    pos = state_positions(ws)
    ids = np.arange(ws.n_seqs, dtype=np.int32)
    if not ws.self_is_aan and pos.max() > 0:
        orc.prefill(ids, pos)
    # host inputs of one step, produced the same way the driver does it (no device involved)
    host = {}
    first_s = list(np.cumsum((0,) + tuple(ws.self_blocks))[:-1])
    first_e = list(np.cumsum((0,) + tuple(ws.encdec_blocks))[:-1])
    if ws.self_is_aan:
        host["x"] = np.stack([synth.aan_x(ws, 0, l) for l in range(ws.n_layers)])
        for t in range(int(pos.max())):          # history of the running average
            for l in range(ws.n_layers):
                orc.o.aan_step(l, ids, np.full(ws.n_seqs, t + 1), synth.aan_x(ws, 1000 + t, l))
    else:
        qkv = [synth.self_qkv(ws, 0, l) for l in range(ws.n_layers)]
        host["q"] = np.stack([qkv[l][0] for l in first_s])
        host["k"] = np.stack([qkv[l][1] for l in first_s])
        host["v"] = np.stack([qkv[l][2] for l in range(ws.n_layers)])
    host["q_enc"] = np.stack([synth.encdec_q(ws, 0, l) for l in first_e])
    host["beams"] = ids
    return ws, orc, host, ids, pos


def time_oracle(w, budget_s=12.0, n_sent_sample=8, max_steps=50, exact_steps=None, warmup=1):
    """Times the oracle as it stands.  Without exact_steps: as many steps as fit the budget."""
    ws, orc, host, ids, pos = oracle_sample(w, n_sent_sample)
    for _ in range(max(warmup, 1)):
        orc.step(host, ids, pos, want_S=False)           # touches every page once
    t0 = time.perf_counter()
    steps = 0
    if exact_steps is not None:
        for _ in range(exact_steps):
            orc.step(host, ids, pos, want_S=False)
        steps = exact_steps
    else:
        while steps < max_steps and (steps == 0 or time.perf_counter() - t0 < budget_s):
            orc.step(host, ids, pos, want_S=False)
            steps += 1
    dt = time.perf_counter() - t0
    cores = len(os.sched_getaffinity(0))
    threads = int(os.environ.get("OMP_NUM_THREADS", cores))
    return {"value": ws.n_seqs * steps / dt, "unit": UNIT, "cores": min(cores, threads), "kind": "oracle",
            "sample": f"{steps} steps of the first {ws.n_sent} sentences x beam {ws.beam} "
                      f"({ws.n_seqs} sequences) of '{w.name}' at the benchmarked cache lengths",
            "ms_per_step": dt / steps * 1e3, "steps": steps}


def whole_job(secs, units_per_rank, world, dist=None, device="cpu"):
    """Replicas only: every rank runs the same workload on its own GPU and nothing is exchanged
    on the data path.  The job's time is the slowest rank's, its throughput the units of all
    ranks over that time.  Returns (max seconds over ranks, units per second of the whole job)."""
    import torch
    t = torch.tensor([secs], dtype=torch.float64, device=device)
    if dist is not None and world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    secs_max = float(t.item())
    return secs_max, units_per_rank * world / secs_max


# ---------------------------------------------------------------------------------------- main
def config_dict(w, extra=None):
    c = {"workload": f"{w.name}: {w.n_layers} layers, d_model {w.d_model}, {w.n_heads} heads, "
                     f"{w.n_sent} sentences x beam {w.beam}, source lengths U[{w.src_lo},{w.src_hi}]",
         "self_blocks": list(w.self_blocks) if not w.self_is_aan else "AAN",
         "encdec_blocks": list(w.encdec_blocks), "storage": w.dtype, "accumulate": "f32"}
    if extra:
        c.update(extra)
    return c


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    res = time_oracle(w, n_sent_sample=2, exact_steps=max(args.steps, 1), warmup=args.warmup)
    line = {"impl": "reference", "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": res["steps"], "warmup": max(args.warmup, 1), "ms_per_step": res["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(w, {"note": "CPU oracle on a bounded sample of the workload"}),
            "cpu_baseline": {k: res[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": res["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


KERNEL_NAMES = {0: "none", 1: "decode_step_kernel (per-warp pipeline)", 2: "decode_step_team_kernel (team pipeline)",
                3: "decode_step_rows_kernel (short rows)"}


def kernel_used(dec):
    from paper_1906_11024_b200 import binding as B
    rc, which, rpu = B.san_step_kernel_used(dec.ctx)
    return {"kernel": KERNEL_NAMES.get(which, "?"), "heads_per_unit": rpu if which >= 2 else None}


def roofline_record(ab, secs_per_step, peak, peak_kind, name, traffic):
    """The step kernel against the HBM roofline.  `achieved` counts the K/V reads (and the AAN
    state) only: the roofline byte count; S, q, O and appended rows are reported beside it."""
    gbs = ab["kv"] / secs_per_step / 1e9
    return {"bound": "hbm", "kernel": name, "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
            "peak_kind": peak_kind, "frac_of_nominal_8tbs": gbs / NOMINAL_HBM_GBS,
            "bytes_per_launch": float(ab["kv"]), "us_per_launch": secs_per_step * 1e6, "launches_per_step": 1,
            "other_bytes_per_launch": {"S": ab["S"], "q_O_new_rows": ab["small"]},
            "achieved_all_bytes": ab["total"] / secs_per_step / 1e9, "traffic": traffic}


def measure(w, steps, warmup, device, peak, peak_kind, fused=True, unshared=True, shared_context=False, n_rep_cap=16):
    """One workload on this rank: the step time with sharing on (and off), the roofline record."""
    import torch
    from paper_1906_11024_b200 import synth
    pos = state_positions(w)
    ab = algorithmic_bytes(w, pos, fused)
    if shared_context:        # Eq. 5: one value plane and one output per enc-dec block
        M, Ne, d, e = w.n_layers, len(w.encdec_blocks), w.d_model, w.elem_bytes
        src = int(w.src_lens().astype(np.int64).sum())
        ab = dict(ab)
        ab["encdec_kv"] = 2 * Ne * src * d * e
        ab["kv"] = ab["self_kv"] + ab["encdec_kv"] + ab["aan"]
        ab["small"] -= (M - Ne) * w.n_seqs * d * e
        ab["total"] = ab["kv"] + ab["S"] + ab["small"]
    n_rep = int(min(n_rep_cap, max(2, math.ceil(3 * L2_BYTES / max(ab["total"], 1)))))
    decs, sbs, pos = build_replicas(w, n_rep, device, shared_context)
    secs, launches, window = time_steps(decs, sbs, steps, warmup, device, lambda: None, fused)
    err = [d.device_status()[0] for d in decs]
    assert not any(err), f"device check failed during the timed region: {err}"
    used = kernel_used(decs[0]) if fused else {"kernel": "append/weights/apply kernels", "heads_per_unit": None}
    rec = {"value": w.n_seqs * steps / secs, "unit": UNIT, "steps": steps, "ms_per_step": secs / steps * 1e3,
           "replicas": n_rep, "launches_per_step": launches, "used": used, "bytes": ab,
           "roofline": roofline_record(ab, secs / steps, peak, peak_kind, used["kernel"], ncu_traffic("fused", w.name))}
    keep = (decs, sbs, pos)
    if unshared and not shared_context:
        for d in decs:
            d.close()
        del decs, sbs, keep
        torch.cuda.empty_cache()
        wu = synth.unshared(w)
        abu = algorithmic_bytes(wu, pos, fused)
        decs_u, sbs_u, _ = build_replicas(wu, n_rep, device)
        su, lu, _ = time_steps(decs_u, sbs_u, steps, warmup, device, lambda: None, fused)
        rec["unshared"] = {"value": wu.n_seqs * steps / su, "unit": UNIT, "ms_per_step": su / steps * 1e3,
                           "kv_bytes_per_step": abu["kv"], "bytes_per_step": abu["total"],
                           "kv_gbs": abu["kv"] / (su / steps) / 1e9, "gpu_launches_per_step": lu,
                           "traffic": ncu_traffic("fused", wu.name),
                           "speedup_from_sharing": su / secs,
                           "kv_bytes_ratio_shared_over_unshared": ab["kv"] / abu["kv"]}
        keep = (decs_u, sbs_u, pos, wu)
    return rec, keep, window


def release(keep):
    import torch
    for d in keep[0]:
        d.close()
    del keep
    torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5000)
    ap.add_argument("--warmup", type=int, default=100)
    ap.add_argument("--impl", default="san", choices=["san", "reference"])
    ap.add_argument("--workload", default="long", choices=["tiny", "base", "big", "long", "aan"])
    ap.add_argument("--path", default="fused", choices=["fused", "calls"],
                    help="fused: san_decode_step, one launch per step; calls: append/weights/apply launches")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-unshared", action="store_true")
    ap.add_argument("--only", action="store_true", help="measure the named workload alone (no other workloads, no extra legs)")
    ap.add_argument("--sharing", default="on", choices=["on", "off"],
                    help="off: time the workload with every block size 1 as the main arm (for byte counts of the unshared path)")
    args = ap.parse_args()

    from paper_1906_11024_b200 import synth
    w = synth.WORKLOADS[args.workload]
    if args.sharing == "off":
        w = synth.unshared(w)
        args.no_unshared = True
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    from paper_1906_11024_b200 import build as san_build
    from paper_1906_11024_b200 import binding
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the attention path has no CPU fallback")
    san_build.build()
    binding.lib()
    device = torch.device(f"cuda:{local_rank}")
    torch.cuda.set_device(device)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        if dist is not None:
            dist.barrier()

    peak, peak_kind = measured_peak_gbs()
    fused = args.path == "fused"
    pos = state_positions(w)
    ab = algorithmic_bytes(w, pos, fused)
    n_rep = int(min(16, max(E2E_BATCHES, math.ceil(3 * L2_BYTES / max(ab["total"], 1)))))
    decs, sbs, pos = build_replicas(w, n_rep, device)

    phys = local_rank
    cvd = os.environ.get("CUDA_VISIBLE_DEVICES", "")
    if cvd:
        parts = [x.strip() for x in cvd.split(",")]
        if local_rank < len(parts) and parts[local_rank].isdigit():
            phys = int(parts[local_rank])
    sampler = ClockSampler(phys)
    sampler.start()
    secs, launches_per_step, (t0, t1) = time_steps(decs, sbs, args.steps, args.warmup, device, barrier, fused)
    clocks = sampler.stop(t0, t1)
    err = [d.device_status()[0] for d in decs]
    assert not any(err), f"device check failed during the timed region: {err}"
    used = kernel_used(decs[0]) if fused else {"kernel": "append/weights/apply kernels", "heads_per_unit": None}

    secs_max, value = whole_job(secs, w.n_seqs * args.steps, world, dist, device)

    if fused:      # one kernel per step: its launch duration is the step time of the timed region
        roof = roofline_record(ab, secs / args.steps, peak, peak_kind, "san_decode_step: " + used["kernel"], ncu_traffic(args.path, w.name))
    else:
        dom_s, dom_per_step = time_dominant_kernel(w, decs, sbs, device)
        dom_bytes = dominant_kernel_bytes(w, pos)
        roof = {"bound": "hbm", "kernel": "san_attn_apply (apply_kernel)", "achieved": dom_bytes / dom_s / 1e9, "peak": peak,
                "unit": "GB/s", "frac": dom_bytes / dom_s / 1e9 / peak, "peak_kind": peak_kind, "bytes_per_launch": dom_bytes,
                "us_per_launch": dom_s * 1e6, "launches_per_step": dom_per_step, "traffic": None}
    e2e_steps = min(args.steps, 100)
    e2e_s, e2e_serial_s, h2d, d2h, e2e_batches = time_e2e(w, decs, sbs, e2e_steps, device, fused)
    next_rows = {}
    if rank == 0 and not args.only:
        next_rows["beam_reorder"] = time_beam_reorder(w, decs, sbs, pos, device, peak)
        fb = time_full_block(w, device, peak)
        if fb is not None:
            next_rows["full_sequence"] = fb

    unshared = None
    if not args.no_unshared and rank == 0:
        for d in decs:
            d.close()
        del decs, sbs
        torch.cuda.empty_cache()
        wu = synth.unshared(w)
        abu = algorithmic_bytes(wu, pos, fused)
        decs_u, sbs_u, _ = build_replicas(wu, n_rep, device)
        su, lu, _ = time_steps(decs_u, sbs_u, args.steps, args.warmup, device, lambda: None, fused)
        unshared = {"value": wu.n_seqs * args.steps / su, "unit": UNIT, "ms_per_step": su / args.steps * 1e3,
                    "kv_bytes_per_step": abu["kv"], "bytes_per_step": abu["total"],
                    "kv_gbs": abu["kv"] / (su / args.steps) / 1e9, "gpu_launches_per_step": lu,
                    "traffic": ncu_traffic(args.path, wu.name)}
        if not args.only:
            js = time_js_matrix(wu, decs_u[0], sbs_u[0], pos, device)
            if js is not None:
                next_rows["policy_learner"] = js
        for d in decs_u:
            d.close()
        del decs_u, sbs_u
        torch.cuda.empty_cache()
    else:
        for d in decs:
            d.close()
        del decs, sbs
        torch.cuda.empty_cache()

    # ---- the other configurations, Eq. 5 and the beam sweep: fewer steps each, rank 0 only
    workloads, eq5, beams = {}, None, None
    if rank == 0 and fused and not args.only and args.sharing == "on":
        sub_steps = max(200, min(args.steps, 2000))
        for name in ("base", "big", "long", "aan"):
            if name == w.name:
                continue
            rec, keep, _ = measure(synth.WORKLOADS[name], sub_steps, max(args.warmup, 3), device, peak, peak_kind,
                                   unshared=not args.no_unshared)
            release(keep)
            workloads[name] = {k: rec[k] for k in ("value", "unit", "steps", "ms_per_step", "used", "roofline")}
            if "unshared" in rec:
                workloads[name]["unshared"] = rec["unshared"]
        workloads["tiny"] = {"note": "configuration 1 (float32, one sentence): parity only, it fits L2 and is launch-bound"}
        # Eq. 5 on the base shape: encoder-decoder attention with one value plane and one output per block
        wb = synth.WORKLOADS["base"]
        own, keep, _ = measure(wb, sub_steps, max(args.warmup, 3), device, peak, peak_kind, unshared=False)
        release(keep)
        shr, keep, _ = measure(wb, sub_steps, max(args.warmup, 3), device, peak, peak_kind, unshared=False, shared_context=True)
        release(keep)
        eq5 = {"workload": "base", "own_values_ms_per_step": own["ms_per_step"], "shared_context_ms_per_step": shr["ms_per_step"],
               "own_values_kv_bytes": own["bytes"]["kv"], "shared_context_kv_bytes": shr["bytes"]["kv"],
               "encdec_kv_bytes": {"own_values": own["bytes"]["encdec_kv"], "shared_context": shr["bytes"]["encdec_kv"]},
               "speedup": own["ms_per_step"] / shr["ms_per_step"], "roofline_frac": shr["roofline"]["frac"],
               "note": "Eq. 5: the block's lowest layer applies S to its values and the layers above reuse that output; "
                       "enc-dec K/V bytes fall from (N_e + M) to 2 N_e planes"}
        # beam sizes (Figure 5 sweeps 4..20) on the base shape
        beams = {}
        import dataclasses
        for beam in (4, 8, 12, 16, 20):
            if beam > binding.SAN_MAX_BEAM:
                continue
            wbm = dataclasses.replace(wb, beam=beam, name=f"base-beam{beam}")
            rec, keep, _ = measure(wbm, sub_steps, max(args.warmup, 3), device, peak, peak_kind, unshared=not args.no_unshared)
            release(keep)
            beams[str(beam)] = {"value": rec["value"], "ms_per_step": rec["ms_per_step"], "kv_frac": rec["roofline"]["frac"],
                                "speedup_from_sharing": rec.get("unshared", {}).get("speedup_from_sharing")}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    ms = secs_max / args.steps * 1e3
    step_gbs = ab["total"] / (secs_max / args.steps) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32" if w.dtype == "f32" else "bf16", "data": "synthetic",
        "config": config_dict(w, {"l2": f"steps rotate over {n_rep} independent replicas of the device state "
                                        f"({ab['total'] * n_rep / 1e6:.0f} MB touched per cycle, L2 is 126 MB)",
                                  "state": "each sequence at the middle of its target length"
                                           if not w.ragged_prefix else "seeded ragged prefix lengths",
                                  "mean_cache_len": float((pos + 1).mean()), "mean_src_len": float(w.src_lens().mean()),
                                  "path": "san_decode_step, one launch per step" if fused
                                          else "san_cache_append + san_attn_weights/apply per block",
                                  "kernel": used["kernel"], "heads_per_unit": used["heads_per_unit"],
                                  "multi_gpu": "replicas only: no sharding, no collective"}),
        "gpu_launches": launches_per_step * args.steps, "gpu_launches_per_step": launches_per_step,
        "hbm": {"kv_bytes_per_step": ab["kv"], "bytes_per_step": ab["total"], "achieved_gbs_all_bytes": step_gbs,
                "kv_gbs": ab["kv"] / (secs_max / args.steps) / 1e9, "peak_kind": peak_kind},
        "roofline": roof,
        "e2e": {"value": w.n_seqs * e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_s / e2e_steps * 1e3,
                "one_batch_alone_ms_per_step": e2e_serial_s / e2e_steps * 1e3,
                "batches_in_flight": e2e_batches,
                "how": "san_decode_step_host, one C-ABI call per step with pinned host buffers; a batch's step is a chain "
                       "(copy in, kernel, copy out), so several request batches (one context, stream and set of pinned "
                       "buffers each) take turns and the copies of one overlap the kernels of the others"},
        "clocks": clocks,
    }
    if workloads:
        line["workloads"] = workloads
    if eq5:
        line["eq5"] = eq5
    if beams:
        line["beam_sweep"] = beams
    if next_rows:
        line["next_rows"] = next_rows
    if unshared is not None:
        unshared["speedup_from_sharing"] = value / world / unshared["value"]
        unshared["kv_bytes_ratio_shared_over_unshared"] = ab["kv"] / unshared["kv_bytes_per_step"]
        line["unshared"] = unshared
    if world == 1 and not args.no_cpu_baseline:
        cb = time_oracle(w)
        line["cpu_baseline"] = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
