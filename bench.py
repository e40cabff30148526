"""Benchmark of the linear-attention layer's hot path on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

One step is one pass of the hot path over one batch of synthetic input.  The headline
workload is the LLaMA-2-7B-shaped prefill (B=4, H=32, d=128, T=2048, bf16, elu+1, 3 taps);
on one GPU the same run also times the other shapes (batched decode, tree verification with its
commit, long-context prefill) and reports them under "others".  --workload NAME makes another
shape the headline.  Rank 0 prints one JSON line.

With N > 1 every rank processes its own batch -- (sequence, head) units are independent, so
there is no collective on the data path -- and the value is the total over ranks divided by the
slowest rank's time.  The ranks come from torch.distributed.run (RANK / WORLD_SIZE in the
environment); started plainly with --gpus N > 1, this program starts the N ranks itself.

Timing: W warm-up steps, then R regions of exactly K steps each, every region bracketed by a
barrier and a device synchronisation on both sides and timed with CUDA events on the launching
stream; the reported time is the median region (max over ranks within each region).
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
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2406_07368_b200 import workloads as wl  # noqa: E402
from paper_2406_07368_b200 import dist as ladist   # noqa: E402

L2_BYTES = 126 * 2 ** 20
NOMINAL_HBM_GBS = 7700.0        # HGX B200 data-sheet figure, printed beside the measured copy bandwidth
REGIONS = 5                     # timed regions of K steps each; the median is reported


# ----------------------------------------------------------------------------------------
def profiled_traffic(workload: str, kernel: str | None = None):
    """DRAM bytes (read + written) per launch of a workload's dominant kernel, as counted by ncu.

    The figure is read from the summaries under profiles/ -- a line
        # bench-traffic: workload=NAME kernel=KERNEL source=PATH sha256=HEX dram_bytes_per_launch=N
    written beside each capture -- and is only returned while the kernel's source file still hashes to the value
    recorded with the capture: once the kernel has changed, the counters describe another program and the result
    is None."""
    import hashlib
    pdir = os.path.join(ROOT, "profiles")
    if not os.path.isdir(pdir):
        return None
    for fn in sorted(os.listdir(pdir)):
        if not fn.endswith((".txt", ".md")):
            continue
        for line in open(os.path.join(pdir, fn), errors="replace"):
            if not line.startswith("# bench-traffic:"):
                continue
            kv = dict(tok.split("=", 1) for tok in line.split()[2:] if "=" in tok)
            if kv.get("workload") != workload or (kernel is not None and kv.get("kernel") != kernel):
                continue
            src = os.path.join(ROOT, kv.get("source", ""))
            if not os.path.isfile(src) or hashlib.sha256(open(src, "rb").read()).hexdigest() != kv.get("sha256"):
                return None
            return float(kv["dram_bytes_per_launch"])
    return None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "sm_max_mhz": float(p.get("sm_max_mhz", 1965.0)), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sm_max_mhz": 1965.0,
            "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None
        self.t0 = self.t1 = None

    def wait_ready(self, timeout: float = 5.0):
        """nvidia-smi's start-up can stall CUDA calls for a moment: let it pass before anything is timed."""
        end = time.time() + timeout
        while self.proc is not None and not self.rows and time.time() < end:
            time.sleep(0.05)

    def mark_start(self):
        self.t0 = time.time()

    def mark_end(self):
        time.sleep(0.15)
        self.t1 = time.time()

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def __exit__(self, *a):
        if self.proc is not None:
            self.proc.terminate()
            self.thread.join(timeout=2)

    def summary(self, t0=None, t1=None):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        t0 = self.t0 if t0 is None else t0
        t1 = self.t1 if t1 is None else t1
        inside = [r for t, r in self.rows if t0 is not None and t0 <= t <= (t1 or t)]
        for r in inside or [r for _, r in self.rows]:     # samples taken during the timed region, if any fell into it
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, val in zip(names, r[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def dev(x, io, device):
    from paper_2406_07368_b200 import binding
    return torch.from_numpy(np.ascontiguousarray(x)).to(binding.TORCH_DTYPE[io]).to(device)


# ----------------------------------------------------------------------------------------
# The steps of each workload.  Each factory returns (step_fn, units_per_step, bytes_per_launch,
# launches_per_step, e2e_fn or None, description).
# ----------------------------------------------------------------------------------------
def prefill_workload(W: wl.Workload, rank: int, device):
    from paper_2406_07368_b200 import binding
    io = W.io
    q, k, v = W.prefill_inputs()
    if rank:   # another batch of the same law for every rank
        q, k, v = wl.qkv(W.seed + 1000 * rank, q.shape, W.scale, io)
    w = dev(W.weights(), "f32", device)
    ctx = binding.Context(W.H, W.d, W.W, W.phi, W.eps, io, chunk=W.chunk)
    per_set = 4 * q.size * 2                                   # q, k, v read + o written, bf16
    nsets = max(2, -(-2 * L2_BYTES // per_set) + 1) if per_set < 4 * L2_BYTES else 1
    base = [dev(x, io, device) for x in (q, k, v)]
    sets = [[x.roll(i, dims=0).contiguous() if i else x for x in base] for i in range(nsets)]
    outs = [torch.empty_like(base[0]) for _ in range(nsets)]
    st = ctx.new_state(W.B)
    ws_bytes = ctx.la_prefill_workspace_bytes(W.B, W.T)      # few chains, long sequence: lend the split workspace
    if ws_bytes:
        ctx.la_set_workspace(torch.empty(ws_bytes, dtype=torch.uint8, device=device))
    counter = [0]

    def step():
        i = counter[0] % nsets
        counter[0] += 1
        ctx.la_prefill(sets[i][0], sets[i][1], sets[i][2], w, st, init_state=False, out=outs[i])

    pinned = [torch.from_numpy(x).to(binding.TORCH_DTYPE[io]).pin_memory() for x in (q, k, v)]
    o_host = torch.empty(q.shape, dtype=binding.TORCH_DTYPE[io]).pin_memory()

    if nsets < 2:                                 # a second device buffer set for the pipelined end-to-end loop
        sets.append([torch.empty_like(x) for x in base])
        outs.append(torch.empty_like(base[0]))
    o_hosts = [o_host, torch.empty(q.shape, dtype=binding.TORCH_DTYPE[io]).pin_memory()]

    def e2e_in(b):
        for dst, src in zip(sets[b], pinned):
            dst.copy_(src, non_blocking=True)

    def e2e_compute(b):
        ctx.la_prefill(sets[b][0], sets[b][1], sets[b][2], w, st, init_state=False, out=outs[b])

    def e2e_out(b):
        o_hosts[b].copy_(outs[b], non_blocking=True)

    e2e_step = (e2e_in, e2e_compute, e2e_out)

    tokens = W.B * W.T
    units = W.B * W.H * W.T
    alg_bytes = units * 4 * W.d * 2 + W.B * W.H * (W.d * W.d + W.d) * 4
    info = {"ctx": ctx, "tokens_per_step": tokens, "alg_bytes_per_launch": alg_bytes, "launches_per_step": 1,
            "h2d": 3 * q.size * 2, "d2h": q.size * 2, "kernel": "prefill" + (" (sequence split: 3 launches)" if ws_bytes else ""),
            "flops_per_launch": units * 4 * W.d * (W.chunk + W.d),
            # causal-strict count: the masked upper triangle of every group is not counted
            "flops_strict_per_launch": units * (2 * W.d * (W.chunk + 1) + 4 * W.d * W.d),
            "period": nsets,
            "l2": f"{nsets} input sets of {per_set / 2**20:.0f} MiB rotated (each larger than L2)"}
    return step, e2e_step, info


def decode_workload(W: wl.Workload, rank: int, device):
    from paper_2406_07368_b200 import binding
    io = W.io
    ctx = binding.Context(W.H, W.d, W.W, W.phi, W.eps, io)
    w = dev(W.weights(), "f32", device)
    st = ctx.new_state(W.B)
    # state after a seeded prefill of a shorter prompt: same magnitude law, bounded set-up time
    q, k, v = W.prefill_inputs(T=256)
    ctx.la_prefill(dev(q, io, device), dev(k, io, device), dev(v, io, device), w, st)
    nrot = 8
    toks = [[dev(x, io, device) for x in W.decode_inputs(s)] for s in range(nrot)]
    out = torch.empty(W.B, W.H, W.d, dtype=binding.TORCH_DTYPE[io], device=device)
    counter = [0]

    def step():
        t = toks[counter[0] % nrot]
        counter[0] += 1
        ctx.la_decode_step(t[0], t[1], t[2], w, st, out=out)

    pinned = [x.cpu().pin_memory() for x in toks[0]]
    o_host = torch.empty(out.shape, dtype=out.dtype).pin_memory()

    outs2 = [out, torch.empty_like(out)]
    o_hosts = [o_host, torch.empty(out.shape, dtype=out.dtype).pin_memory()]

    # q, k, v of a step travel as one buffer (one copy instead of three: at this size the copies' fixed cost counts)
    pinned_qkv = torch.stack(pinned).pin_memory()
    dev_qkv = [torch.empty(pinned_qkv.shape, dtype=pinned_qkv.dtype, device=device) for _ in range(2)]

    def e2e_in(b):
        dev_qkv[b].copy_(pinned_qkv, non_blocking=True)

    def e2e_compute(b):
        ctx.la_decode_step(dev_qkv[b][0], dev_qkv[b][1], dev_qkv[b][2], w, st, out=outs2[b])

    def e2e_out(b):
        o_hosts[b].copy_(outs2[b], non_blocking=True)

    e2e_step = (e2e_in, e2e_compute, e2e_out)

    units = W.B * W.H
    el = 2
    alg = units * (8 * W.d * W.d + 2 * 4 * W.d + 4 * W.d * el + 2 * (W.W - 1) * W.d * el)
    info = {"ctx": ctx, "tokens_per_step": W.B, "alg_bytes_per_launch": alg, "launches_per_step": 1,
            "h2d": 3 * units * W.d * el, "d2h": units * W.d * el, "kernel": "decode",
            "flops_per_launch": units * 4 * W.d * W.d,
            "period": nrot,
            "setup": "state built by a seeded 256-token prompt (the workload's own prompt is 2048 tokens; the step's "
                     "cost does not depend on what the state holds)",
            "l2": f"state of {units * W.d * W.d * 4 / 2**20:.0f} MiB streamed every step (larger than L2)"}
    return step, e2e_step, info


def verify_workload(W: wl.Workload, rank: int, device):
    from paper_2406_07368_b200 import binding
    io = W.io
    ctx = binding.Context(W.H, W.d, W.W, W.phi, W.eps, io, max_nodes=W.tree_nodes, max_depth=W.max_depth)
    w = dev(W.weights(), "f32", device)
    N = W.tree_nodes
    # several independent state sets so that the rotation exceeds L2
    per_state = W.B * W.H * W.d * W.d * 4
    nsets = max(2, -(-2 * L2_BYTES // per_state) + 1)
    q, k, v = W.prefill_inputs(T=256)
    states = []
    for i in range(nsets):
        st = ctx.new_state(W.B)
        ctx.la_prefill(dev(q, io, device), dev(k, io, device), dev(v, io, device), w, st)
        states.append(st)
    nrot = 4
    drafts = [[dev(x, io, device) for x in W.draft_inputs(r)] for r in range(nrot)]
    trees = [W.trees(r) for r in range(nrot)]
    parents = [torch.from_numpy(p).to(device) for p, _ in trees]
    accepts = [torch.from_numpy(a).to(device) for _, a in trees]
    out = torch.empty(W.B, W.H, N, W.d, dtype=binding.TORCH_DTYPE[io], device=device)
    path = torch.empty(W.B, W.max_depth, dtype=torch.int32, device=device)
    clen = torch.empty(W.B, dtype=torch.int32, device=device)
    counter = [0]

    def step():
        i = counter[0]
        counter[0] += 1
        r, st = i % nrot, states[i % nsets]
        ctx.la_verify_tree(drafts[r][0], drafts[r][1], drafts[r][2], parents[r], w, st, out=out)
        ctx.la_commit(drafts[r][1], drafts[r][2], parents[r], accepts[r], st, path_out=path, commit_len=clen)

    pinned = [x.cpu().pin_memory() for x in drafts[0]]
    o_host = torch.empty(out.shape, dtype=out.dtype).pin_memory()

    outs2 = [out, torch.empty_like(out)]
    o_hosts = [o_host, torch.empty(out.shape, dtype=out.dtype).pin_memory()]

    def e2e_in(b):
        for dst, src in zip(drafts[b], pinned):
            dst.copy_(src, non_blocking=True)

    def e2e_compute(b):
        st = states[b]
        ctx.la_verify_tree(drafts[b][0], drafts[b][1], drafts[b][2], parents[b], w, st, out=outs2[b])
        ctx.la_commit(drafts[b][1], drafts[b][2], parents[b], accepts[b], st, path_out=path, commit_len=clen)

    def e2e_out(b):
        o_hosts[b].copy_(outs2[b], non_blocking=True)

    e2e_step = (e2e_in, e2e_compute, e2e_out)

    def probe(i):   # the dominant kernel alone (it does not modify the state)
        ctx.la_verify_tree(drafts[i % nrot][0], drafts[i % nrot][1], drafts[i % nrot][2], parents[i % nrot], w,
                           states[i % nsets], out=out)

    def probe_commit(i):   # the second kernel of the step alone (it advances the state, which timing does not mind)
        r = i % nrot
        ctx.la_commit(drafts[r][1], drafts[r][2], parents[r], accepts[r], states[i % nsets], path_out=path, commit_len=clen)

    # the acceptance step that sits between verify and commit in real use (the whole model runs in between, so it is
    # not part of the timed step): timed alone, as a latency figure
    toks = [[torch.from_numpy(x).to(device) for x in wl.token_batch(W.seed, r, W.B, N)] for r in range(nrot)]
    acc_out = [torch.empty(W.B, dtype=torch.int32, device=device) for _ in range(3)]

    def probe_accept(i):
        r = i % nrot
        ctx.la_accept_greedy(parents[r], toks[r][0], toks[r][1], toks[r][2], *acc_out)

    # accepted tokens per round: the depth of the accepted node, averaged over the rotation
    acc_len = float(np.mean([[wl.tree_depths(p[b])[a[b]] if a[b] >= 0 else 0 for b in range(W.B)] for p, a in trees]))
    units = W.B * W.H
    el = 2
    alg_verify = units * (4 * W.d * W.d + 4 * W.d + 4 * N * W.d * el + (W.W - 1) * W.d * el)
    info = {"ctx": ctx, "tokens_per_step": W.B * N, "alg_bytes_per_launch": alg_verify, "launches_per_step": 2,
            "h2d": 3 * units * N * W.d * el, "d2h": units * N * W.d * el, "kernel": "verify", "probe": probe,
            "second": {"kernel": "commit", "probe": probe_commit,
                       "alg_bytes_per_launch": units * (8 * W.d * W.d + 8 * W.d + acc_len * 2 * W.d * el
                                                        + 2 * (W.W - 1) * W.d * el)},
            "accepted_tokens_per_step": W.B * acc_len, "accept_probe": probe_accept,
            "flops_per_launch": units * (2 * N * W.d * W.d + 4 * N * N * W.d),
            "period": nrot * nsets // math.gcd(nrot, nsets),
            "setup": "every state set built by a seeded 256-token prompt (the workload's own prompt is 1024 tokens; the "
                     "step's cost does not depend on what the state holds)",
            "l2": f"{nsets} state sets of {per_state / 2**20:.0f} MiB rotated (together larger than 2x L2)"}
    return step, e2e_step, info


def promptgen_workload(W: wl.Workload, rank: int, device):
    """Prompt + generation: for every (P, G) pair a prefill of P tokens, then G decode steps, one sequence."""
    from paper_2406_07368_b200 import binding
    io, shapes = W.io, W.extra["shapes"]
    ctx = binding.Context(W.H, W.d, W.W, W.phi, W.eps, io, chunk=W.chunk)
    w = dev(W.weights(), "f32", device)
    tdt = binding.TORCH_DTYPE[io]
    prompts, gens, outs_p, outs_g, states = [], [], [], [], []
    for i, (P, G) in enumerate(shapes):
        q, k, v = wl.qkv(W.seed + 100 * rank + i, (W.B, W.H, P + G, W.d), W.scale, io)
        prompts.append([dev(x[:, :, :P], io, device) for x in (q, k, v)])
        # generation tokens step-major, so that every step reads one contiguous [B, H, d] slab
        gens.append([dev(np.ascontiguousarray(np.moveaxis(x[:, :, P:], 2, 0)), io, device) for x in (q, k, v)])
        outs_p.append(torch.empty(W.B, W.H, P, W.d, dtype=tdt, device=device))
        outs_g.append(torch.empty(G, W.B, W.H, W.d, dtype=tdt, device=device))
        states.append(ctx.new_state(W.B))

    def run_shape(i):
        P, G = shapes[i]
        ctx.la_prefill(prompts[i][0], prompts[i][1], prompts[i][2], w, states[i], init_state=False, out=outs_p[i])
        for g in range(G):
            ctx.la_decode_step(gens[i][0][g], gens[i][1][g], gens[i][2][g], w, states[i], out=outs_g[i][g])

    def step():
        for i in range(len(shapes)):
            run_shape(i)

    pinned = [[x.cpu().pin_memory() for x in prompts[i] + gens[i]] for i in range(len(shapes))]
    host_out = [[torch.empty(o.shape, dtype=tdt).pin_memory() for o in (outs_p[i], outs_g[i])] for i in range(len(shapes))]

    def e2e_step():
        for i in range(len(shapes)):
            for dst, src in zip(prompts[i] + gens[i], pinned[i]):
                dst.copy_(src, non_blocking=True)
            run_shape(i)
            host_out[i][0].copy_(outs_p[i], non_blocking=True)
            host_out[i][1].copy_(outs_g[i], non_blocking=True)

    tokens = W.B * sum(P + G for P, G in shapes)
    units = W.B * W.H
    el = 2
    dec_bytes = units * (8 * W.d * W.d + 2 * 4 * W.d + 4 * W.d * el + 2 * (W.W - 1) * W.d * el)
    n_launch = sum(1 + G for _, G in shapes)
    moved = 4 * tokens * W.H * W.d * el
    info = {"ctx": ctx, "tokens_per_step": tokens, "alg_bytes_per_launch": dec_bytes, "launches_per_step": n_launch,
            "h2d": 3 * tokens * W.H * W.d * el, "d2h": tokens * W.H * W.d * el, "kernel": "decode (one sequence: 32 units)",
            "probe": lambda i: ctx.la_decode_step(gens[0][0][i % 16], gens[0][1][i % 16], gens[0][2][i % 16], w, states[0],
                                                  out=outs_g[0][i % 16]),
            "flops_per_launch": units * 4 * W.d * W.d, "period": 1, "shape_probe": run_shape, "shapes": shapes,
            "l2": f"{moved / 2**20:.0f} MiB of tokens and {units * W.d * W.d * 4 / 2**20:.0f} MiB of state per shape: "
                  "L2-resident by nature of the workload (a single sequence)"}
    return step, e2e_step, info


def grouped_workload(W: wl.Workload, rank: int, device):
    """The three-branch block (la_prefill_grouped) on the prefill shape.  bf16 with d = 128 and groups of 64 or 128
    tokens run on the tensor cores (a group of 64 takes one half-filled 128-row tile); other shapes on the CUDA cores."""
    from paper_2406_07368_b200 import binding
    io = W.io
    q, k, v = W.prefill_inputs()
    if rank:
        q, k, v = wl.qkv(W.seed + 1000 * rank, q.shape, W.scale, io)
    w = dev(W.weights(), "f32", device)
    ctx = binding.Context(W.H, W.d, W.W, W.phi, W.eps, io, chunk=W.chunk)
    per_set = 4 * q.size * 2
    nsets = max(2, -(-2 * L2_BYTES // per_set) + 1)
    base = [dev(x, io, device) for x in (q, k, v)]
    sets = [[x.roll(i, dims=0).contiguous() if i else x for x in base] for i in range(nsets)]
    outs = [torch.empty_like(base[0]) for _ in range(nsets)]
    st = ctx.new_state(W.B)
    alpha, sscale = W.extra["alpha"], W.extra["softmax_scale"]
    counter = [0]

    def step():
        i = counter[0] % nsets
        counter[0] += 1
        ctx.la_prefill_grouped(sets[i][0], sets[i][1], sets[i][2], w, st, W.chunk, alpha, sscale, out=outs[i])

    pinned = [torch.from_numpy(x).to(binding.TORCH_DTYPE[io]).pin_memory() for x in (q, k, v)]
    o_host = torch.empty(q.shape, dtype=binding.TORCH_DTYPE[io]).pin_memory()

    def e2e_step():                                  # host inputs in, one call, host outputs back
        for dst, src in zip(sets[0], pinned):
            dst.copy_(src, non_blocking=True)
        ctx.la_prefill_grouped(sets[0][0], sets[0][1], sets[0][2], w, st, W.chunk, alpha, sscale, out=outs[0])
        o_host.copy_(outs[0], non_blocking=True)

    units = W.B * W.H * W.T
    flops = units * (4 * W.d * W.d + 2 * W.d * (W.chunk + 1) + 2 * W.d * W.W)   # readout + state update, scores + PV, taps
    info = {"ctx": ctx, "tokens_per_step": W.B * W.T, "alg_bytes_per_launch": units * 4 * W.d * 2, "launches_per_step": 1,
            "h2d": 3 * q.size * 2, "d2h": q.size * 2,
            "kernel": "prefill_tc in three-branch mode (groups of 64: one half-filled tile per group)",
            "flops_per_launch": flops, "period": nsets,
            "l2": f"{nsets} input sets of {per_set / 2**20:.0f} MiB rotated (each larger than L2)"}
    return step, e2e_step, info


FACTORIES = {"llama7b_prefill": prefill_workload, "grouped_block": grouped_workload, "long_prefill": prefill_workload,
             "batched_decode": decode_workload, "tree_verify": verify_workload, "prompt_gen": promptgen_workload,
             "prefill_taps32": prefill_workload, "tree_verify_taps8": verify_workload}
METRICS = {"llama7b_prefill": ("prefill_tokens_per_s_per_layer", "tokens/s"),
           "long_prefill": ("prefill_tokens_per_s_per_layer", "tokens/s"),
           "grouped_block": ("prefill_tokens_per_s_per_layer", "tokens/s"),
           "batched_decode": ("decode_tokens_per_s_per_layer", "tokens/s"),
           "tree_verify": ("verify_nodes_per_s_per_layer", "nodes/s"),
           "prefill_taps32": ("prefill_tokens_per_s_per_layer", "tokens/s"),
           "tree_verify_taps8": ("verify_nodes_per_s_per_layer", "nodes/s"),
           "prompt_gen": ("prompt_and_generation_tokens_per_s_per_layer", "tokens/s")}


# ----------------------------------------------------------------------------------------
def oracle_samples(W: wl.Workload):
    """Bounded samples of the workload for the float64 oracle: {"primary": (fn, units, text), "definition": ... }.
    The primary sample uses the oracle's fastest exact form for the mode (grouped for prefill, the recurrence for
    decode, the tree form for verify + commit); for prefill the quadratic definition is timed beside it."""
    from oracle import la_oracle as orc
    if W.name in ("llama7b_prefill", "long_prefill", "prefill_taps32"):
        T = W.T
        q, k, v = W.prefill_inputs(B=1, T=T)
        w = W.weights()
        Tq = min(W.T, 2048)
        return {"primary": (lambda: orc.prefill_chunked(q, k, v, w, W.phi, W.eps, W.chunk), T,
                            f"grouped form (groups of {W.chunk}), 1 of {W.B} sequences, all {W.H} heads, all {T} tokens"),
                "definition": (lambda: orc.prefill_quadratic(q[:, :, :Tq], k[:, :, :Tq], v[:, :, :Tq], w, W.phi, W.eps), Tq,
                               f"quadratic definition, 1 of {W.B} sequences, all {W.H} heads, first {Tq} of {W.T} tokens")}
    if W.name == "grouped_block":
        q, k, v = W.prefill_inputs(B=1, H=4)
        w = W.weights()[:4]
        return {"primary": (lambda: orc.prefill_grouped_block(q, k, v, w, W.phi, W.eps, W.chunk, W.extra["alpha"],
                                                              W.extra["softmax_scale"]), W.T * 4 / W.H,
                            f"token-by-token form, 1 of {W.B} sequences, 4 of {W.H} heads, all {W.T} tokens")}
    if W.name == "prompt_gen":
        P, G = min(W.extra["shapes"], key=lambda pg: pg[0] + pg[1])
        q, k, v = wl.qkv(W.seed, (W.B, W.H, P + G, W.d), W.scale, W.io)
        w = W.weights()

        def fn():
            _, st = orc.prefill_chunked(q[:, :, :P], k[:, :, :P], v[:, :, :P], w, W.phi, W.eps, W.chunk)
            for g in range(G):
                _, st = orc.decode_step(q[:, :, P + g], k[:, :, P + g], v[:, :, P + g], w, W.phi, W.eps, st)
        return {"primary": (fn, W.B * (P + G),
                            f"grouped prefill of {P} tokens then {G} recurrent steps: the ({P}, {G}) pair, all heads")}
    if W.name == "batched_decode":
        B = 8
        q, k, v = W.prefill_inputs(B=B, T=64)
        w = W.weights()
        _, st = orc.prefill_quadratic(q, k, v, w, W.phi, W.eps)
        qs, ks, vs = W.decode_inputs(0, B=B)
        box = [st]

        def fn():
            for _ in range(4):
                _, box[0] = orc.decode_step(qs, ks, vs, w, W.phi, W.eps, box[0])
        return {"primary": (fn, 4 * B, f"recurrent form, {B} of {W.B} sequences, all heads, 4 decode steps")}
    B = 2
    q, k, v = W.prefill_inputs(B=B, T=64)
    w = W.weights()
    _, st = orc.prefill_quadratic(q, k, v, w, W.phi, W.eps)
    qd, kd, vd = W.draft_inputs(0, B=B)
    parent, accept = W.trees(0, B=B)

    def fn():
        orc.verify_tree(qd, kd, vd, parent, w, W.phi, W.eps, st)
        orc.commit(kd, vd, parent, accept, W.phi, st, W.max_depth)
    return {"primary": (fn, B * W.tree_nodes, f"tree form, {B} of {W.B} sequences, all heads, one verify + commit round")}


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return len(os.sched_getaffinity(0))


def time_fn(fn, units, repeats: int, warmup: int = 0):
    for _ in range(warmup):
        fn()
    t0 = time.perf_counter()
    for _ in range(repeats):
        fn()
    dt = time.perf_counter() - t0
    return units * repeats / dt, dt / repeats


def l2_note(W: wl.Workload) -> str:
    """How the GPU arm keeps the 126 MB L2 from serving a step's inputs (a property of the workload's sizes)."""
    if W.name in ("llama7b_prefill", "long_prefill", "grouped_block", "prefill_taps32"):
        per_set = 4 * W.B * W.H * W.T * W.d * 2
        nsets = max(2, -(-2 * L2_BYTES // per_set) + 1) if per_set < 4 * L2_BYTES else 1
        return f"{nsets} input sets of {per_set / 2**20:.0f} MiB rotated (each larger than L2)"
    if W.name == "batched_decode":
        return f"state of {W.B * W.H * W.d * W.d * 4 / 2**20:.0f} MiB streamed every step (larger than L2)"
    if W.name in ("tree_verify", "tree_verify_taps8"):
        per_state = W.B * W.H * W.d * W.d * 4
        nsets = max(2, -(-2 * L2_BYTES // per_state) + 1)
        return f"{nsets} state sets of {per_state / 2**20:.0f} MiB rotated (together larger than 2x L2)"
    return "a single sequence: tokens and state are L2-resident by nature of the workload"


def base_config(W: wl.Workload, world: int = 1) -> dict:
    """The workload's identity: the same keys and values in both arms of the benchmark."""
    return {"workload": W.name, "B": W.B, "H": W.H, "d": W.d, "T": W.T, "chunk": W.chunk, "phi": W.phi, "eps": W.eps,
            "conv_taps": W.W, "tree_nodes": W.tree_nodes, "decode_steps": W.decode_steps, "rounds": W.rounds,
            "io": W.io, "seed": W.seed, "l2": l2_note(W), "parallelism": "replicas only" if world > 1 else "single GPU"}


def run_reference(args, W: wl.Workload):
    metric, unit = METRICS[W.name]
    fn, units, text = oracle_samples(W)["primary"]
    value, per_step = time_fn(fn, units, args.steps, args.warmup)
    cores = blas_threads()
    line = {"impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": base_config(W, int(os.environ.get("WORLD_SIZE", 1))), "sample_per_step": text,
            "cpu_baseline": {"value": value, "unit": unit, "cores": cores, "kind": "oracle", "sample": text},
            "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------
def measure(W: wl.Workload, steps: int, warmup: int, rank: int, world: int, device, clocks, use_graph: bool,
            e2e_steps: int):
    """Times one workload on this rank's GPU: R regions of `steps` steps (median reported), the dominant kernel
    alone where a step has several, and (e2e_steps > 0) the end-to-end loop with host buffers."""
    step, e2e_step, info = FACTORIES[W.name](W, rank, device)
    ctx = info["ctx"]
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    if ctx.la_last_device_status() != 0:
        raise RuntimeError(f"{W.name}: device status not OK after warm-up")

    # The same calls, recorded once into a CUDA graph of one rotation period and replayed: the steps are short
    # enough for the Python interpreter to be the bottleneck otherwise.  K steps = K // period replays, the rest eager.
    period = info["period"]

    def capture(fn):
        n0 = ctx.la_launch_count()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(period):
                fn(i)
        return g, ctx.la_launch_count() - n0

    graph, launches_per_replay = None, 0
    if use_graph and steps >= period:
        graph, launches_per_replay = capture(lambda i: step())
        graph.replay()                                     # one untimed replay
        torch.cuda.synchronize()

    def run_steps(n):
        extra = 0
        if graph is not None:
            for _ in range(n // period):
                graph.replay()
            extra = (n // period) * launches_per_replay
            n = n % period
        for _ in range(n):
            step()
        return extra

    clocks.wait_ready()
    regions, launches = [], 0
    t_start = time.time()
    for _ in range(REGIONS):
        ladist.barrier(world)
        torch.cuda.synchronize()
        launches0 = ctx.la_launch_count()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        replayed = run_steps(steps)
        ev1.record(stream)
        torch.cuda.synchronize()
        ladist.barrier(world)
        regions.append(ladist.max_over_ranks(ev0.elapsed_time(ev1), world, device))
        launches = ctx.la_launch_count() - launches0 + replayed          # per region of K steps
    time.sleep(0.15)
    t_end = time.time()
    ms = float(np.median(regions))

    # per-launch duration of one kernel alone, measured live: a short second pass on the same stream
    def time_probe(fn):
        for i in range(3):
            fn(i)
        torch.cuda.synchronize()
        pgraph = None if graph is None else capture(fn)[0]
        n_probe = min(steps, 100) if pgraph is None else period * max(1, 100 // period)
        samples = []
        for _ in range(3):
            p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            p0.record(stream)
            if pgraph is None:
                for i in range(n_probe):
                    fn(i)
            else:
                for _ in range(n_probe // period):
                    pgraph.replay()
            p1.record(stream)
            torch.cuda.synchronize()
            samples.append(p0.elapsed_time(p1) / n_probe)
        return float(np.median(samples))

    second = None
    if info["launches_per_step"] == 1 or "probe" not in info:
        kernel_ms = ms / steps
    else:
        kernel_ms = time_probe(info["probe"])
        if "second" in info:
            second = dict(info["second"])
            second["launch_ms"] = time_probe(second.pop("probe"))

    res = {"W": W, "info": info, "ctx": ctx, "regions": regions, "ms": ms, "steps": steps, "launches": int(launches),
           "kernel_ms": kernel_ms, "second": second, "graph": graph is not None, "period": period,
           "clock_window": (t_start, t_end), "value": world * info["tokens_per_step"] * steps / (ms * 1e-3)}
    if "accepted_tokens_per_step" in info:
        res["accepted_tokens_per_s"] = world * info["accepted_tokens_per_step"] * steps / (ms * 1e-3)
    if "accept_probe" in info:
        res["accept_kernel"] = {"kernel": "accept_greedy", "launch_ms": time_probe(info["accept_probe"]),
                                "note": "integer kernel, one warp per sequence: latency, not bandwidth"}
    if "shape_probe" in info:                    # latency of every (prompt, generation) pair on its own
        res["shape_ms"] = {}
        for i, (P, G) in enumerate(info["shapes"]):
            fn = info["shape_probe"]
            fn(i)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                fn(i)
            g.replay()
            torch.cuda.synchronize()
            p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            p0.record(stream)
            for _ in range(5):
                g.replay()
            p1.record(stream)
            torch.cuda.synchronize()
            res["shape_ms"][f"({P}, {G})"] = p0.elapsed_time(p1) / 5

    if e2e_steps > 0:
        # End to end: pinned host inputs copied in, result copied out, every step.  Where the workload gives the
        # three parts separately the loop is pipelined over two buffer sets: the copy-in of step i+1 and the copy-out
        # of step i-1 run on streams of their own beside the kernels of step i (PCIe is full duplex); every step
        # still pays for all of its bytes inside the timed region.
        if callable(e2e_step):
            def e2e_run(n):
                for _ in range(n):
                    e2e_step()
        else:
            e2e_in, e2e_compute, e2e_out = e2e_step
            s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

            def e2e_run(n):
                ev_in = [torch.cuda.Event() for _ in range(2)]
                ev_comp = [torch.cuda.Event() for _ in range(2)]
                ev_out = [torch.cuda.Event() for _ in range(2)]
                start = torch.cuda.Event()
                start.record(stream)
                s_in.wait_event(start)
                s_out.wait_event(start)
                for i in range(n):
                    b = i & 1
                    with torch.cuda.stream(s_in):
                        if i >= 2:
                            s_in.wait_event(ev_comp[b])        # the inputs of step i-2 have been consumed
                        e2e_in(b)
                        ev_in[b].record(s_in)
                    stream.wait_event(ev_in[b])
                    if i >= 2:
                        stream.wait_event(ev_out[b])           # the outputs of step i-2 have been copied out
                    e2e_compute(b)
                    ev_comp[b].record(stream)
                    with torch.cuda.stream(s_out):
                        s_out.wait_event(ev_comp[b])
                        e2e_out(b)
                        ev_out[b].record(s_out)
                for b in range(min(n, 2)):
                    stream.wait_event(ev_out[b])

        e2e_run(2)
        torch.cuda.synchronize()
        ladist.barrier(world)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        e2e_run(e2e_steps)
        e1.record(stream)
        torch.cuda.synchronize()
        e2e_ms = ladist.max_over_ranks(e0.elapsed_time(e1), world, device)
        res["e2e"] = {"value": world * info["tokens_per_step"] * e2e_steps / (e2e_ms * 1e-3),
                      "unit": METRICS[W.name][1], "h2d_bytes_per_step": info["h2d"], "d2h_bytes_per_step": info["d2h"],
                      "steps": e2e_steps, "pipelined": not callable(e2e_step)}
    if ctx.la_last_device_status() != 0:
        raise RuntimeError(f"{W.name}: device status not OK after the timed region")
    return res


def roofline_of(res, peaks):
    info, kernel_ms = res["info"], res["kernel_ms"]
    achieved = info["alg_bytes_per_launch"] / (kernel_ms * 1e-3) / 1e9
    tflops = info["flops_per_launch"] / (kernel_ms * 1e-3) / 1e12
    r = {"bound": "hbm", "kernel": info["kernel"], "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
         "frac": achieved / peaks["hbm_gbs"], "traffic": profiled_traffic(res["W"].name),
         "peak_source": peaks["source"], "alg_bytes_per_launch": info["alg_bytes_per_launch"], "launch_ms": kernel_ms,
         "tensor_tflops": tflops, "tensor_frac_of_sustained": tflops / peaks["bf16_tflops_sustained"],
         "frac_of_nominal_7700": achieved / NOMINAL_HBM_GBS}
    if info.get("bound") == "alu":
        # fp32 multiply-adds on the CUDA cores: 148 SMs x 128 lanes x 2 flop at the maximum SM clock
        peak = 148 * 128 * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12
        r.update({"bound": "alu", "achieved": tflops, "peak": peak, "unit": "TFLOP/s", "frac": tflops / peak,
                  "peak_source": "derived: 148 SMs x 128 fp32 lanes x 2 flop x max SM clock",
                  "hbm_gbs_algorithmic": achieved, "hbm_frac_algorithmic": achieved / peaks["hbm_gbs"]})
    if r["traffic"] is not None:                 # the same fraction from the DRAM bytes ncu counted, not the algorithmic ones
        r["achieved_from_traffic"] = r["traffic"] / (kernel_ms * 1e-3) / 1e9
        r["frac_from_traffic"] = r["achieved_from_traffic"] / peaks["hbm_gbs"]
    if "flops_strict_per_launch" in info:
        r["tensor_tflops_strict"] = info["flops_strict_per_launch"] / (kernel_ms * 1e-3) / 1e12
    if info["launches_per_step"] > 1:
        r["step_ms"] = res["ms"] / res["steps"]  # all kernels of the step; launch_ms is the dominant one alone
    if res["second"] is not None:
        second = dict(res["second"])
        a2 = second["alg_bytes_per_launch"] / (second["launch_ms"] * 1e-3) / 1e9
        second.update({"achieved": a2, "unit": "GB/s", "frac": a2 / peaks["hbm_gbs"],
                       "traffic": profiled_traffic(res["W"].name, second["kernel"])})
        r["second_kernel"] = second
    return r


def spread(res):
    per = [x / res["steps"] for x in res["regions"]]
    return {"regions": len(per), "ms_per_step_median": float(np.median(per)), "ms_per_step_min": min(per),
            "ms_per_step_max": max(per)}


def brief(res, peaks, clocks):
    """One workload as an entry of "others": device-timed step, throughput, roofline of its kernels."""
    metric, unit = METRICS[res["W"].name]
    out = {"metric": metric, "value": res["value"], "unit": unit, "steps": res["steps"],
           "ms_per_step": res["ms"] / res["steps"], "timing": spread(res), "gpu_launches": res["launches"],
           "config": base_config(res["W"]), "roofline": roofline_of(res, peaks),
           "clocks": clocks.summary(*res["clock_window"]),
           "launch": f"CUDA graph of {res['period']} steps, replayed" if res["graph"] else "one Python call per kernel"}
    for key in ("accepted_tokens_per_s", "accept_kernel", "shape_ms"):
        if key in res:
            out[key] = res[key]
    if "setup" in res["info"]:
        out["setup"] = res["info"]["setup"]
    return out


OTHERS = {"llama7b_prefill": ("batched_decode", "tree_verify", "long_prefill", "grouped_block", "prefill_taps32",
                              "tree_verify_taps8")}
DEFAULT_STEPS = {"grouped_block": 10, "llama7b_prefill": 200, "long_prefill": 50, "batched_decode": 1000, "tree_verify": 1000,
                 "prompt_gen": 20, "prefill_taps32": 100, "tree_verify_taps8": 1000}
OTHER_STEPS = {"long_prefill": 20, "batched_decode": 400, "tree_verify": 400, "grouped_block": 6, "prefill_taps32": 100,
               "tree_verify_taps8": 400}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama7b_prefill", choices=sorted(FACTORIES))
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-others", action="store_true", help="time the headline workload only")
    ap.add_argument("--no-graph", action="store_true", help="launch every step from Python instead of replaying a CUDA graph")
    args = ap.parse_args()
    W = wl.WORKLOADS[args.workload]()
    rank, world = ladist.rank_world()

    if args.impl == "reference":
        args.steps = args.steps or 3
        args.warmup = 1 if args.warmup is None else args.warmup
        if rank == 0:
            run_reference(args, W)
        return 0

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started plainly: this process becomes the launcher of one rank per GPU
        return ladist.launch_local_ranks([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], args.gpus)

    args.steps = args.steps or DEFAULT_STEPS[W.name]
    args.warmup = 5 if args.warmup is None else max(3, args.warmup)

    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    ladist.init(world, backend="nccl")

    clocks = ClockSampler(local)
    clocks.__enter__()
    try:
        res = measure(W, args.steps, args.warmup, rank, world, device, clocks, not args.no_graph, args.e2e_steps)
        peaks = measured_peaks()
        others = {}
        if world == 1 and not args.no_others:
            for name in OTHERS.get(W.name, ()):
                ctx = res.pop("ctx", None)                 # keep the headline's numbers, release its buffers
                del ctx
                torch.cuda.empty_cache()
                r2 = measure(wl.WORKLOADS[name](), OTHER_STEPS[name], args.warmup, rank, world, device, clocks,
                             not args.no_graph, 0)
                others[name] = brief(r2, peaks, clocks)
                del r2
                torch.cuda.empty_cache()
    finally:
        clocks.__exit__()

    if rank != 0:
        ladist.finish(world)
        return 0

    metric, unit = METRICS[W.name]
    info = res["info"]
    cpu = None
    if not args.no_cpu_baseline and world == 1:
        samples = oracle_samples(W)
        reps = {"grouped_block": 1, "llama7b_prefill": 8, "long_prefill": 2, "batched_decode": 3, "tree_verify": 1, "prompt_gen": 2,
                "prefill_taps32": 4, "tree_verify_taps8": 1}[W.name]
        fn, units, text = samples["primary"]
        v, per = time_fn(fn, units, reps)
        cpu = {"value": v, "unit": unit, "cores": blas_threads(), "kind": "oracle", "sample": text, "seconds": per * reps}
        if "definition" in samples:
            fn, units, text = samples["definition"]
            v2, per2 = time_fn(fn, units, 3)
            cpu["definition_form"] = {"value": v2, "unit": unit, "sample": text, "seconds": per2 * 3}
    config = base_config(W, world)
    run = {"launch": f"CUDA graph of {res['period']} steps, replayed" if res["graph"] else "one Python call per kernel",
           "timing": f"median of {REGIONS} regions of {args.steps} steps, each between barriers and device syncs",
           "l2": info["l2"]}
    if "setup" in info:
        run["setup"] = info["setup"]
    line = {"metric": metric, "value": res["value"], "unit": unit, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": res["ms"] / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if W.io == "bf16" else "f32", "data": "synthetic",
            "config": config, "run": run, "timing": spread(res), "clocks": clocks.summary(*res["clock_window"]),
            "e2e": res.get("e2e"), "gpu_launches": res["launches"], "roofline": roofline_of(res, peaks),
            "cpu_baseline": cpu}
    for key in ("accepted_tokens_per_s", "accept_kernel", "shape_ms"):
        if key in res:
            line[key] = res[key]
    if others:
        line["others"] = others
    print(json.dumps(line), flush=True)
    ladist.finish(world)
    return 0


if __name__ == "__main__":
    sys.exit(main())
