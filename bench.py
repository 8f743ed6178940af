#!/usr/bin/env python
"""Benchmark of the recurrent-layer hot path on synthetic data shaped like the paper's workloads.

One "step" is one pass of the whole hot path over one batch: for every recurrent-layer request of the
workload, single-state initialisation, exact composition, and the chunkwise scan of the request's
recompute segment from the composed state (both families when the workload has both).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg1|cfg2|cfg3|cfg4] [--impl reference]
    python bench.py --sweep        # microseconds per exact composition against K (a JSON line of its own)
    python bench.py --artifacts    # time of building the cached chunk states / transitions (a JSON line of its own)

Prints ONE JSON line (rank 0).  `value` = context tokens served per second by the step (all requests'
context tokens / step time), device-timed with inputs resident in HBM; `e2e` = the same with every
input copied host->device from pinned memory and every result copied back inside the timed region.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_11231_b200 import workloads as wl  # noqa: E402

METRIC = "effective_prefill_tokens_per_s"
UNIT = "tokens/s"
GDN_SHAPE = dict(H_k=16, H_v=32, d_k=128, d_v=128)
SSD_SHAPE = dict(H=80, P=64, N=128, G=1)
GDN_BLOCK = 64    # scan block of the tensor-core GDN kernel (tokens)
SSD_BLOCK = 128   # scan block of the tensor-core SSD kernel (tokens)


# ----------------------------------------------------------------------------- workload description

def build_requests(name: str, rank: int = 0):
    """List of requests of this rank: family, number of cached chunks K, context tokens, recompute tokens."""
    from paper_2608_11231_b200 import sharding
    return sharding.rank_requests(name, rank)


def gdn_scan_flops(tokens: int, s=GDN_SHAPE, C=GDN_BLOCK) -> float:
    """Chunkwise GDN flops: per token and value head 2*(3 d_k d_v + 2 C d_v + 2 C d_k)
    (K S, Q S, K^T U; the triangular solve applied to the right-hand side and P U; K K^T and Q K^T)."""
    per = 2.0 * (3 * s["d_k"] * s["d_v"] + 2 * C * s["d_v"] + 2 * C * s["d_k"])
    return per * s["H_v"] * tokens


def ssd_scan_flops(tokens: int, s=SSD_SHAPE, Q=SSD_BLOCK) -> float:
    """Chunkwise SSD flops: per token and head 2*(2 N P + Q P) plus C B^T once per group 2*Q*N."""
    return (2.0 * (2 * s["N"] * s["P"] + Q * s["P"]) * s["H"] + 2.0 * Q * s["N"] * s["G"]) * tokens


# DRAM bytes (read + write) per scanned token from ncu captures of one launch of each scan kernel (GDN: 8 sequences x
# 2048 tokens; Mamba-2: 16 sequences x 4096 tokens, initial and final states included); the traffic of a scan grows
# in proportion to its tokens.
NCU_DRAM_BYTES_PER_TOKEN = {"gdn.scan": (290.48e6 + 119.29e6) / 16384, "mamba2.scan": (789.18e6 + 672.45e6) / 65536}


def gdn_scan_bytes(tokens: int, s=GDN_SHAPE) -> float:
    return tokens * (2 * s["H_k"] * s["d_k"] * 2 + 2 * s["H_v"] * s["d_v"] * 2 + 2 * s["H_v"] * 4)


# ----------------------------------------------------------------------------- our arm

class Family:
    """Device-resident (and pinned-host) tensors of one recurrence family of the workload."""

    def __init__(self, fam, reqs, seed, torch, b):
        self.fam, self.reqs, self.torch, self.b = fam, reqs, torch, b
        rng = np.random.default_rng(seed)
        self.n_req = len(reqs)
        shared = any(r.get("shared_pool") for r in reqs)
        self.shared = shared
        ks = [r["K"] for r in reqs]
        self.cu_k = np.concatenate([[0], np.cumsum(ks)]).astype(np.int32)
        if shared:
            n_pool = ks[0]
            self.ids = np.concatenate([wl.request_permutation(3, i, n_pool) for i in range(self.n_req)]).astype(np.int32)
        else:
            n_pool = int(self.cu_k[-1])
            self.ids = np.arange(n_pool, dtype=np.int32)
        lens = [r["recompute"] for r in reqs]
        self.cu_seq = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
        T = int(self.cu_seq[-1])
        self.scan_tokens = T
        self.context_tokens = int(sum(r["total"] for r in reqs))
        bf = torch.bfloat16
        h = {}
        if fam == "gdn":
            s = GDN_SHAPE
            h["states"] = torch.from_numpy(wl.synthetic_states(rng, n_pool, s["H_v"], s["d_k"], s["d_v"]))
            h["trans"] = torch.from_numpy(wl.cheap_gdn_transitions(rng, n_pool, s["H_v"], s["d_k"]))
            tok = wl.gdn_tokens(rng, T, s["H_k"], s["H_v"], s["d_k"], s["d_v"], io="bf16")
            for n in ("q", "k", "v"):
                h[n] = torch.from_numpy(tok[n]).to(bf)
            h["g"], h["beta"] = torch.from_numpy(tok["g"]), torch.from_numpy(tok["beta"])
            self.family_code = b.LKV_FAMILY_GDN
            self.state_shape = (s["H_v"], s["d_k"], s["d_v"])
            self.out_shape = (T, s["H_v"], s["d_v"])
        else:
            s = SSD_SHAPE
            h["states"] = torch.from_numpy(wl.synthetic_states(rng, n_pool, s["H"], s["N"], s["P"]))
            h["trans"] = torch.from_numpy(wl.synthetic_logdecay(rng, n_pool, s["H"]))
            h["A"] = torch.from_numpy(wl.ssd_A(rng, s["H"]))
            tok = wl.ssd_tokens(rng, T, s["H"], s["P"], s["N"], s["G"], io="bf16")
            for n in ("x", "B", "C"):
                h[n] = torch.from_numpy(tok[n]).to(bf)
            h["dt"] = torch.from_numpy(tok["dt"])
            self.family_code = b.LKV_FAMILY_MAMBA2
            self.state_shape = (s["H"], s["N"], s["P"])
            self.out_shape = (T, s["H"], s["P"])
        self.host = {n: t.contiguous().pin_memory() for n, t in h.items()}
        self.dev = {n: t.cuda(non_blocking=True) for n, t in self.host.items()}
        self.S0_last = torch.empty((self.n_req,) + self.state_shape, dtype=torch.float32, device="cuda")
        self.S0 = torch.empty_like(self.S0_last)
        self.S_T = torch.empty_like(self.S0_last)
        self.out = torch.empty(self.out_shape, dtype=bf, device="cuda")
        self.host_out = torch.empty(self.out_shape, dtype=bf).pin_memory()
        self.host_S_T = torch.empty(self.S_T.shape, dtype=torch.float32).pin_memory()
        self.ws_init = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
        self.ws_scan = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
        self.h2d_bytes = sum(t.numel() * t.element_size() for t in self.host.values())
        self.d2h_bytes = self.host_out.numel() * 2 + self.host_S_T.numel() * 4
        # bytes an exact composition must move at least once: every pool state and transition that some request reads
        # (a request's first chunk contributes its state only: its transition multiplies nothing), plus S0 written
        first = set(int(self.ids[self.cu_k[r]]) for r in range(self.n_req) if ks[r] > 0)
        later = set(int(i) for r in range(self.n_req) for i in self.ids[self.cu_k[r] + 1:self.cu_k[r + 1]])
        per_state = int(np.prod(self.state_shape)) * 4
        per_trans = h["trans"][0].numel() * 4
        self.compose_bytes = len(first | later) * per_state + len(later) * per_trans + self.n_req * per_state
        self.set_bytes = self.h2d_bytes
        self.launches = 3

    def cold_copy(self):
        """A second instance over the same host data with device buffers of its own (inputs and outputs): launches
        that rotate over several of them find none of their inputs in L2."""
        import copy
        c = copy.copy(self)
        c.dev = {n: t.clone() for n, t in self.dev.items()}
        for n in ("S0_last", "S0", "S_T", "out"):
            setattr(c, n, getattr(self, n).clone())
        c.ws_init, c.ws_scan = self.ws_init.clone(), self.ws_scan.clone()
        return c

    def micro_batches(self, m):
        """The same requests as m instances over slices of this one's buffers (every request has its own pool entries and
        tokens, contiguous in request order): the end-to-end step pipelines them, so that the results of one micro-batch
        travel to the host while the inputs of the next travel to the device."""
        import copy
        if self.shared or self.n_req < m:
            return [self]
        out = []
        per_tok = ("q", "k", "v", "g", "beta", "x", "B", "C", "dt")
        for i in range(m):
            r0, r1 = self.n_req * i // m, self.n_req * (i + 1) // m
            p0, p1, t0, t1 = int(self.cu_k[r0]), int(self.cu_k[r1]), int(self.cu_seq[r0]), int(self.cu_seq[r1])
            c = copy.copy(self)
            c.n_req = r1 - r0
            c.cu_k, c.cu_seq = self.cu_k[r0:r1 + 1] - p0, self.cu_seq[r0:r1 + 1] - t0
            c.ids = np.arange(p1 - p0, dtype=np.int32)
            cut = lambda n, t: t[p0:p1] if n in ("states", "trans") else t[t0:t1] if n in per_tok else t
            c.host = {n: cut(n, t) for n, t in self.host.items()}
            c.dev = {n: cut(n, t) for n, t in self.dev.items()}
            for n in ("S0_last", "S0", "S_T", "host_S_T"):
                setattr(c, n, getattr(self, n)[r0:r1])
            c.out, c.host_out = self.out[t0:t1], self.host_out[t0:t1]
            c.ws_init, c.ws_scan = self.ws_init.clone(), self.ws_scan.clone()
            out.append(c)
        return out

    def upload(self):
        for n, t in self.host.items():
            self.dev[n].copy_(t, non_blocking=True)

    def download(self):
        self.host_out.copy_(self.out, non_blocking=True)
        self.host_S_T.copy_(self.S_T, non_blocking=True)

    def init_last(self):
        b, d = self.b, self.dev
        b.lkv_init_state_batched(d["states"], None, self.ids, self.cu_k, self.n_req, b.LKV_INIT_LAST, None,
                                 self.S0_last, family=self.family_code, workspace_t=self.ws_init)

    def init_exact(self):
        b, d = self.b, self.dev
        b.lkv_init_state_batched(d["states"], d["trans"], self.ids, self.cu_k, self.n_req, b.LKV_INIT_EXACT, None,
                                 self.S0, family=self.family_code, workspace_t=self.ws_init)

    def scan(self):
        b, d = self.b, self.dev
        if self.fam == "gdn":
            b.lkv_gdn_fwd(d["q"], d["k"], d["v"], d["g"], d["beta"], self.S0, self.out, self.S_T,
                          cu_seqlens=self.cu_seq, workspace_t=self.ws_scan)
        else:
            b.lkv_ssd_fwd(d["x"], d["dt"], d["A"], d["B"], d["C"], self.S0, self.out, self.S_T,
                          cu_seqlens=self.cu_seq, workspace_t=self.ws_scan)

    def step(self):
        self.init_last()
        self.init_exact()
        self.scan()

    def make_full_prefill(self, tokens: int):
        """One request's whole context as one sequence (device-generated stand-in tokens, timing only): the scan of
        it from the empty state is the full-prefill reference that the initialisers + recompute scan replace."""
        torch, bf = self.torch, self.torch.bfloat16
        gen = torch.Generator(device="cuda").manual_seed(5)
        rn = lambda *shape: torch.randn(shape, generator=gen, device="cuda")
        if self.fam == "gdn":
            s = GDN_SHAPE
            nrm = torch.nn.functional.normalize
            self.full = dict(q=nrm(rn(tokens, s["H_k"], s["d_k"]), dim=-1).to(bf), k=nrm(rn(tokens, s["H_k"], s["d_k"]), dim=-1).to(bf),
                             v=rn(tokens, s["H_v"], s["d_v"]).to(bf), g=-0.1 * torch.nn.functional.softplus(rn(tokens, s["H_v"])),
                             beta=torch.sigmoid(rn(tokens, s["H_v"])))
            self.full_ST = torch.empty((1,) + self.state_shape, dtype=torch.float32, device="cuda")
            self.full_out = torch.empty((tokens, s["H_v"], s["d_v"]), dtype=bf, device="cuda")
        else:
            s = SSD_SHAPE
            self.full = dict(x=rn(tokens, s["H"], s["P"]).to(bf), dt=torch.nn.functional.softplus(-2.0 + 0.5 * rn(tokens, s["H"])),
                             B=(rn(tokens, s["G"], s["N"]) / s["N"] ** 0.5).to(bf), C=(rn(tokens, s["G"], s["N"]) / s["N"] ** 0.5).to(bf))
            self.full_ST = torch.empty((1,) + self.state_shape, dtype=torch.float32, device="cuda")
            self.full_out = torch.empty((tokens, s["H"], s["P"]), dtype=bf, device="cuda")
        self.full_tokens = tokens

    def full_prefill_segmented(self):
        """The same full prefill with the sequence cut into segments scanned in parallel (GDN; the library picks the count)."""
        b, d = self.b, self.full
        if getattr(self, "seg_scratch", None) is None:
            s = GDN_SHAPE
            self.seg_scratch = self.torch.empty(64 * s["H_v"] * s["d_k"] * s["d_v"] * 4, dtype=self.torch.uint8, device="cuda")
        b.lkv_gdn_fwd_segmented(d["q"], d["k"], d["v"], d["g"], d["beta"], None, self.full_out, self.full_ST, n_segments=0,
                                scratch=self.seg_scratch, workspace_t=self.ws_scan)

    def full_prefill(self):
        b, d = self.b, self.full
        if self.fam == "gdn":
            b.lkv_gdn_fwd(d["q"], d["k"], d["v"], d["g"], d["beta"], None, self.full_out, self.full_ST, workspace_t=self.ws_scan)
        else:
            b.lkv_ssd_fwd(d["x"], d["dt"], self.dev["A"], d["B"], d["C"], None, self.full_out, self.full_ST,
                          workspace_t=self.ws_scan)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons every 200 ms while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        sm = [float(r[0]) for r in self.rows if r and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) > 1 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) > 3 + i and r[3 + i] == "Active" for r in self.rows)]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def cpu_baseline_sample(pairs: int = 8, T: int = 12288):
    """The oracle as it stands, timed on this machine's cores on a bounded sample of the workload:
    `pairs` times, exact composition of one GDN request (K = 16) plus a T-token GDN scan, all 32 value
    heads, and the same for one Mamba-2 request (K = 16, T tokens, 80 heads)."""
    import oracle
    rng = np.random.default_rng(99)
    s, m = GDN_SHAPE, SSD_SHAPE
    K = 16
    tok = wl.gdn_tokens(rng, T, s["H_k"], s["H_v"], s["d_k"], s["d_v"])
    states = wl.synthetic_states(rng, K, s["H_v"], s["d_k"], s["d_v"])
    trans = wl.cheap_gdn_transitions(rng, K, s["H_v"], s["d_k"])
    mt = wl.ssd_tokens(rng, T, m["H"], m["P"], m["N"], m["G"])
    A = wl.ssd_A(rng, m["H"])
    mstates = wl.synthetic_states(rng, K, m["H"], m["N"], m["P"])
    lam = wl.synthetic_logdecay(rng, K, m["H"])
    oracle.num_threads()
    t0 = time.perf_counter()
    for _ in range(pairs):
        S0 = oracle.init_exact_gdn(states, trans)
        oracle.gdn_seq(tok["q"], tok["k"], tok["v"], tok["g"], tok["beta"], S0)
        M0 = oracle.init_exact_mamba(mstates, lam)
        oracle.ssd_seq(mt["x"], mt["dt"], A, mt["B"], mt["C"], M0)
    dt = time.perf_counter() - t0
    # context covered by the sample at the workload's recompute ratio (0.2): each request's
    # T recomputed tokens stand for T / 0.2 context tokens
    context = pairs * 2 * T / 0.2
    return dict(value=context / dt, unit=UNIT, cores=oracle.num_threads(), kind="oracle",
                sample=f"{pairs} GDN + {pairs} Mamba-2 requests, K={K} exact composition + {T}-token scan each "
                       f"(= {int(context)} context tokens at r=0.2), {dt:.2f} s"), dt


def run_reference(args):
    """--impl reference: the fp64 oracle on the host cores, each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    pairs = 2
    for _ in range(args.warmup if args.warmup < 2 else 1):
        cpu_baseline_sample(pairs)
    times, base = [], None
    for _ in range(args.steps):
        base, dt = cpu_baseline_sample(pairs)
        times.append(dt)
    context = pairs * 2 * 12288 / 0.2
    t = sum(times) / len(times)
    value = context / t
    base["value"] = value
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=1e3 * t, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic", config={"workload": args.workload, "sample": base["sample"]},
                cpu_baseline=base, e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line))


L2_BYTES = 126e6
SMALL_KERNEL_US = 100.0   # below this a single launch between two events is dominated by the 2.048 us event resolution
                          # (on these boxes) and the launch gap: such kernels are timed many launches at a time instead


class Timer:
    """Device timing helpers of one rank (CUDA events on the current stream, max over ranks)."""

    def __init__(self, torch, dist, world):
        from paper_2608_11231_b200 import sharding
        self.torch, self.dist, self.world, self.sharding = torch, dist, world, sharding
        self.flush_buf = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")

    def barrier(self):
        self.torch.cuda.synchronize()
        if self.world > 1:
            self.dist.barrier()
            self.torch.cuda.synchronize()

    def max_over_ranks(self, x: float) -> float:
        return self.sharding.job_step_ms(x, self.dist if self.world > 1 else None, "cuda")

    def graph_of(self, fn):
        """Capture fn (launches only, no allocation) into a CUDA graph so that host overhead of the
        Python binding does not enter device timings of microsecond-scale kernels."""
        torch = self.torch
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        return g

    def back_to_back(self, replay, steps):
        torch = self.torch
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.barrier()
        ev0.record()
        for _ in range(steps):
            replay()
        ev1.record()
        self.barrier()
        return self.max_over_ranks(ev0.elapsed_time(ev1) / steps)  # ms per step

    def flushed(self, replay, steps):
        """Each iteration timed alone, L2 flushed (untimed) before it.  Returns the list of ms."""
        torch = self.torch
        ts = []
        self.barrier()
        for _ in range(steps):
            self.flush_buf.zero_()
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record()
            replay()
            ev1.record()
            ev1.synchronize()
            ts.append(ev0.elapsed_time(ev1))
        self.barrier()
        return ts

    def kernel_us(self, fns, set_bytes, steps):
        """Device time of one launch of a kernel, cold inputs.  fns: the same call over several sets of buffers.

        A launch longer than SMALL_KERNEL_US is timed alone between two events after an L2 flush (median, p90 over
        `steps`).  A shorter one is timed R launches at a time inside one graph between one event pair, the launches
        rotating over n sets of buffers whose total size exceeds L2 (so every launch finds its inputs in HBM), and the
        time divided by R; median and p90 over 9 such replays."""
        g = self.graph_of(fns[0])
        ts = sorted(1e3 * t for t in self.flushed(g.replay, steps))
        single = dict(us=statistics.median(ts), p90_us=ts[min(len(ts) - 1, int(0.9 * len(ts)))],
                      method="one launch per event pair, L2 flushed before it")
        if single["us"] >= SMALL_KERNEL_US or len(fns) < 2:
            return single
        n = len(fns)
        R = max(24, n)

        def many():
            for i in range(R):
                fns[i % n]()
        gm = self.graph_of(many)
        per = []
        for _ in range(9):
            t = self.flushed(gm.replay, 1)[0]
            per.append(1e3 * t / R)
        per.sort()
        return dict(us=statistics.median(per), p90_us=per[min(len(per) - 1, int(0.9 * len(per)))],
                    method=f"{R} launches per event pair rotating over {n} buffer sets "
                           f"({n * set_bytes / 1e6:.0f} MB in total, L2 is 126 MB), time / {R}",
                    one_launch_flushed_us=single["us"], event_resolution_us=2.048)


def n_cold_sets(set_bytes: float) -> int:
    """Buffer sets needed for their total to exceed L2 with margin: at least 4, at most 48."""
    return int(min(48, max(4, -(-1.5 * L2_BYTES // max(set_bytes, 1.0)))))


def host_us_per_call(fn, torch, calls=50):
    """Host time of one call of the Python binding + C entry point (argument checks, tensor maps, launch), measured
    while the stream is kept short of work: what a caller pays on its own thread per launch."""
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(calls):
        fn()
    dt = time.perf_counter() - t0
    torch.cuda.synchronize()
    return 1e6 * dt / calls


def measure_workload(name, rank, world, args, torch, b, dist, timer, peaks, with_e2e=True):
    """All device timings of one workload on this rank: whole step, every kernel alone, the full-prefill reference."""
    reqs = build_requests(name, rank)
    fams = []
    for fam in ("mamba2", "gdn"):
        sub = [r for r in reqs if r["family"] == fam]
        if sub:
            fams.append(Family(fam, sub, seed=100 + rank * 10 + len(fams), torch=torch, b=b))
    torch.cuda.synchronize()
    context_tokens = sum(f.context_tokens for f in fams)
    scan_tokens = sum(f.scan_tokens for f in fams)
    total_input_bytes = sum(f.h2d_bytes for f in fams)
    cold_by_size = total_input_bytes > 4 * L2_BYTES        # inputs far larger than the 126 MB L2
    steps = args.steps

    fam_streams = [torch.cuda.Stream() for _ in fams[1:]]

    def step():
        # the families are independent: the second one runs on a stream of its own (a fork and a join inside the
        # step, captured into the graph like everything else), so that its CTAs fill the tail of the first one's kernels
        cur = torch.cuda.current_stream()
        for f, st in zip(fams[1:], fam_streams):
            st.wait_stream(cur)
            with torch.cuda.stream(st):
                f.step()
        fams[0].step()
        for st in fam_streams:
            cur.wait_stream(st)

    for _ in range(max(args.warmup, 3)):
        step()
    g_step = timer.graph_of(step)
    for _ in range(max(args.warmup, 3)):
        g_step.replay()
    if cold_by_size:
        ms = timer.back_to_back(g_step.replay, steps)
    else:
        ts = timer.flushed(g_step.replay, steps)
        ms = timer.max_over_ranks(sum(ts) / len(ts))

    # per-kernel device times, each kernel alone
    parts = {}
    for f in fams:
        sets = [f]
        if not cold_by_size:
            sets += [f.cold_copy() for _ in range(n_cold_sets(f.set_bytes) - 1)]
        for kname in ("init_last", "init_exact", "scan"):
            r = timer.kernel_us([getattr(x, kname) for x in sets], f.set_bytes, max(steps, 7))
            r["us"] = 1e3 * timer.max_over_ranks(1e-3 * r["us"])
            parts[f"{f.fam}.{kname}"] = r
        del sets
    host_us = {}
    if rank == 0:
        for f in fams:
            host_us[f"{f.fam}.init_exact"] = host_us_per_call(f.init_exact, torch)
            host_us[f"{f.fam}.scan"] = host_us_per_call(f.scan, torch, calls=20)

    ms_e2e, e2e_steps = None, 0
    if with_e2e:
        # the requests of a step are independent: they go through in micro-batches (four per family), one stream each, so
        # that the device->host copies of one overlap the host->device copies of the next
        e2e_units = [u for f in fams for u in f.micro_batches(4)]
        e2e_streams = [torch.cuda.Stream() for _ in e2e_units]

        def step_e2e():
            cur = torch.cuda.current_stream()
            for f, st in zip(e2e_units, e2e_streams):
                st.wait_stream(cur)
                with torch.cuda.stream(st):
                    f.upload()
                    f.step()
                    f.download()
            for st in e2e_streams:
                cur.wait_stream(st)
        e2e_steps = max(1, min(steps, 3))
        step_e2e()
        ms_e2e = timer.back_to_back(step_e2e, e2e_steps)

    # full-prefill reference (single-family configurations): one request's whole context scanned from the empty state
    full = {}
    if name in ("cfg1", "cfg2", "cfg3"):
        for f in fams:
            f.make_full_prefill(f.reqs[0]["total"])
            g = timer.graph_of(f.full_prefill)
            t = 1e-3 * statistics.median(1e3 * x for x in timer.flushed(g.replay, max(steps, 5)))
            # the same request served from the cache: its share of the batched init calls plus its recompute scan
            t_cached = 1e-3 * (parts[f"{f.fam}.init_exact"]["us"] + parts[f"{f.fam}.scan"]["us"]) / f.n_req
            full[f.fam] = dict(tokens=f.full_tokens, us=1e3 * t, tokens_per_s=f.full_tokens / (t * 1e-3),
                               cached_path_us_per_request=1e3 * t_cached, cached_over_full=t_cached / t)
            if f.fam == "gdn":
                # the same prefill as a sequence-parallel scan (lkv_gdn_fwd_segmented, segment count chosen by the library)
                g2 = timer.graph_of(f.full_prefill_segmented)
                t2 = 1e-3 * statistics.median(1e3 * x for x in timer.flushed(g2.replay, max(steps, 5)))
                full[f.fam]["segmented_us"] = 1e3 * t2
                full[f.fam]["segments"] = max(1, min((148 // GDN_SHAPE["H_v"] + 3) // 2, f.full_tokens // 512))
                f.seg_scratch = None
            del f.full, f.full_out

    detail = {}
    for f in fams:
        us = {k: parts[f"{f.fam}.{k}"]["us"] for k in ("init_last", "init_exact", "scan")}
        flops = gdn_scan_flops(f.scan_tokens) if f.fam == "gdn" else ssd_scan_flops(f.scan_tokens)
        tf = flops / (us["scan"] * 1e-6) / 1e12
        tpeak = peaks["bf16_tflops_sustained"] if us["scan"] > 50e3 else peaks["bf16_tflops"]
        gbs = f.compose_bytes / (us["init_exact"] * 1e-6) / 1e9
        detail[f.fam] = dict(
            requests=f.n_req, context_tokens=f.context_tokens, scan_tokens=f.scan_tokens,
            init_last_us=us["init_last"], init_exact_us=us["init_exact"], scan_us=us["scan"],
            init_exact_p90_us=parts[f"{f.fam}.init_exact"]["p90_us"], scan_p90_us=parts[f"{f.fam}.scan"]["p90_us"],
            timing={k: parts[f"{f.fam}.{k}"]["method"] for k in ("init_exact", "scan")},
            scan_tokens_per_s=f.scan_tokens / (us["scan"] * 1e-6), scan_tflops=tf, scan_frac_of_tensor_peak=tf / tpeak,
            compose_bytes=f.compose_bytes, compose_gbs=gbs, compose_frac_of_hbm=gbs / peaks["hbm_gbs"])
        if host_us:
            detail[f.fam]["host_us_per_call"] = dict(init_exact=round(host_us[f"{f.fam}.init_exact"], 1),
                                                     scan=round(host_us[f"{f.fam}.scan"], 1))
    return dict(name=name, reqs=reqs, fams=fams, ms=ms, ms_e2e=ms_e2e, e2e_steps=e2e_steps, parts=parts, full=full,
                detail=detail, context_tokens=context_tokens, scan_tokens=scan_tokens, cold_by_size=cold_by_size)


def l2_note(cold_by_size):
    return ("inputs far larger than L2, steps timed back to back" if cold_by_size else
            "L2 flushed (512 MiB write, untimed) before every timed step")


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2608_11231_b200 import binding as b
    from paper_2608_11231_b200 import sharding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    b.load()
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            peaks = json.load(fh)
        peak_src = "measured"
    except OSError:
        peaks = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
        peak_src = "fallback"
    timer = Timer(torch, dist, world)

    # clocks are sampled from the warm-up to the end of the end-to-end steps: the GPU is busy throughout
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    m = measure_workload(args.workload, rank, world, args, torch, b, dist, timer, peaks)
    clocks = sampler.stop() if rank == 0 else None
    ms, ms_e2e, parts, fams = m["ms"], m["ms_e2e"], m["parts"], m["fams"]
    job_context_tokens, job_scan_tokens = m["context_tokens"], m["scan_tokens"]
    if world > 1:
        job_context_tokens = sharding.job_total(m["context_tokens"], dist, "cuda")
        job_scan_tokens = sharding.job_total(m["scan_tokens"], dist, "cuda")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # dominant kernel: the one with the largest share of the step
    dom = max(parts, key=lambda k: parts[k]["us"])
    fam_name, kern = dom.split(".")
    f = next(x for x in fams if x.fam == fam_name)
    dom_ms = 1e-3 * parts[dom]["us"]
    if kern == "scan":
        flops = gdn_scan_flops(f.scan_tokens) if fam_name == "gdn" else ssd_scan_flops(f.scan_tokens)
        achieved = flops / (dom_ms * 1e-3) / 1e12
        peak = peaks["bf16_tflops_sustained"] if dom_ms > 50.0 else peaks["bf16_tflops"]
        per_token = NCU_DRAM_BYTES_PER_TOKEN.get(dom)
        roof = dict(bound="tensor", achieved=achieved, peak=peak, unit="TFLOP/s", frac=achieved / peak,
                    traffic=None if per_token is None else per_token * f.scan_tokens,
                    traffic_source="ncu dram bytes of a smaller launch of the same kernel, scaled by tokens", kernel=dom,
                    peak_source=peak_src)
    else:
        achieved = f.compose_bytes / (dom_ms * 1e-3) / 1e9
        roof = dict(bound="hbm", achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s",
                    frac=achieved / peaks["hbm_gbs"], traffic=None, kernel=dom, peak_source=peak_src)

    RUN = dict(requests=len(m["reqs"]), context_tokens=m["context_tokens"], scan_tokens=m["scan_tokens"],
               cold_by_size=m["cold_by_size"], h2d=sum(x.h2d_bytes for x in fams), d2h=sum(x.d2h_bytes for x in fams),
               e2e_steps=m["e2e_steps"], launches=sum(x.launches for x in fams), detail=m["detail"], full=m["full"])

    # the other single-GPU configurations, same protocol (a one-GPU run of the default workload only)
    configs = {}
    if world == 1 and args.workload == "cfg4" and not args.no_configs:
        del m, fams, f
        torch.cuda.empty_cache()
        for name in ("cfg1", "cfg2", "cfg3"):
            c = measure_workload(name, 0, 1, args, torch, b, dist, timer, peaks, with_e2e=False)
            configs[name] = dict(ms_per_step=c["ms"], value=c["context_tokens"] / (c["ms"] * 1e-3), unit=UNIT,
                                 requests=len(c["reqs"]), context_tokens=c["context_tokens"],
                                 scan_tokens=c["scan_tokens"], l2=l2_note(c["cold_by_size"]), kernels=c["detail"],
                                 full_prefill=c["full"])
            del c
            torch.cuda.empty_cache()

    base, _ = cpu_baseline_sample() if world == 1 else (None, None)
    if base is not None:
        # the same oracle on one thread, on a quarter-size sample (about as long as the all-core run)
        import oracle
        n_all = oracle.num_threads()
        oracle.set_num_threads(1)
        try:
            one, _ = cpu_baseline_sample(pairs=1, T=3072)
        finally:
            oracle.set_num_threads(n_all)
        base["one_thread"] = dict(value=one["value"], sample=one["sample"])
    line = dict(
        metric=METRIC, value=job_context_tokens / (ms * 1e-3), unit=UNIT, n_gpus=world, steps=args.steps,
        warmup=max(args.warmup, 3), ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None,
        dtype="bf16", data="synthetic",
        config=dict(workload=args.workload, requests=RUN["requests"], context_tokens=RUN["context_tokens"],
                    scan_tokens=RUN["scan_tokens"], l2=l2_note(RUN["cold_by_size"]),
                    timing="CUDA-graph replay, CUDA events", sharding="requests across ranks, no collective"),
        e2e=dict(value=job_context_tokens / (ms_e2e * 1e-3), unit=UNIT,
                 h2d_bytes_per_step=RUN["h2d"], d2h_bytes_per_step=RUN["d2h"],
                 ms_per_step=ms_e2e, steps=RUN["e2e_steps"]),
        gpu_launches=RUN["launches"] * args.steps,
        scan_tokens_per_s=job_scan_tokens / (ms * 1e-3),
        roofline=roof, kernels=RUN["detail"], clocks=clocks)
    if RUN["full"]:
        line["full_prefill"] = RUN["full"]
    if configs:
        line["configs"] = configs
    if base is not None:
        line["cpu_baseline"] = base
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_sweep(args):
    """--sweep: microseconds per exact composition against K, both families, batch 1 and batch 8 (every request
    with its own pool entries), cold inputs (Timer.kernel_us).  Prints one JSON line of its own."""
    import torch

    from paper_2608_11231_b200 import binding as b
    torch.cuda.set_device(0)
    b.load()
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            hbm = json.load(fh)["hbm_gbs"]
    except OSError:
        hbm = 6650.0
    timer = Timer(torch, None, 1)
    gen = torch.Generator(device="cuda").manual_seed(7)
    rows = []
    for fam in ("mamba2", "gdn"):
        if fam == "gdn":
            H, dk, dv, code = GDN_SHAPE["H_v"], GDN_SHAPE["d_k"], GDN_SHAPE["d_v"], b.LKV_FAMILY_GDN
        else:
            H, dk, dv, code = SSD_SHAPE["H"], SSD_SHAPE["N"], SSD_SHAPE["P"], b.LKV_FAMILY_MAMBA2
        for n_req in (1, 8):
            for K in (1, 2, 4, 8, 16, 32, 64):
                n_pool = n_req * K
                ids = np.arange(n_pool, dtype=np.int32)
                cu_k = (np.arange(n_req + 1) * K).astype(np.int32)
                tr_bytes = n_pool * H * (dk * dk if fam == "gdn" else 1) * 4
                set_bytes = (n_pool + n_req) * H * dk * dv * 4 + tr_bytes
                fns, keep = [], []
                for _ in range(n_cold_sets(set_bytes)):
                    states = torch.randn((n_pool, H, dk, dv), generator=gen, device="cuda")
                    if fam == "gdn":
                        trans = torch.randn((n_pool, H, dk, dk), generator=gen, device="cuda") * (0.45 / dk ** 0.5)
                    else:
                        trans = -2.0 * torch.rand((n_pool, H), generator=gen, device="cuda")
                    S0 = torch.empty((n_req, H, dk, dv), device="cuda")
                    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
                    keep.append((states, trans, S0, ws))
                    fns.append(lambda t=keep[-1]: b.lkv_init_state_batched(t[0], t[1], ids, cu_k, n_req, b.LKV_INIT_EXACT,
                                                                           None, t[2], family=code, workspace_t=t[3]))
                r = timer.kernel_us(fns, set_bytes, max(args.steps, 7))
                nbytes = set_bytes
                if fam == "gdn":   # the first chunk's transition is never read
                    nbytes -= n_req * H * dk * dk * 4
                rows.append(dict(family=fam, requests=n_req, K=K, us=round(r["us"], 2), p90_us=round(r["p90_us"], 2),
                                 gbs=round(nbytes / r["us"] / 1e3, 1), frac_of_hbm=round(nbytes / r["us"] / 1e3 / hbm, 3),
                                 launches_per_event_pair=1 if "one launch" in r["method"] else max(24, len(fns)),
                                 buffer_sets=len(fns)))
                del fns, keep
                torch.cuda.empty_cache()
    # the online fold (transitions applied from the cached key / gate streams, one scan per chunk) beside the
    # composition over materialised transitions: one request, K chunks of 1024 tokens, GDN benchmark shapes
    fold = []
    sg = GDN_SHAPE
    for K in (4, 16):
        L = 1024
        T = K * L
        rn = lambda *shape: torch.randn(shape, generator=gen, device="cuda")
        kk = torch.nn.functional.normalize(rn(T, sg["H_k"], sg["d_k"]), dim=-1).to(torch.bfloat16)
        gg = -0.1 * torch.nn.functional.softplus(rn(T, sg["H_v"]))
        bb = torch.sigmoid(rn(T, sg["H_v"]))
        states = rn(K, sg["H_v"], sg["d_k"], sg["d_v"])
        cu = (np.arange(K + 1) * L).astype(np.int32)
        ws = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
        trans = b.lkv_gdn_chunk_transition(kk, gg, bb, cu_seqlens=cu, workspace_t=ws)
        S0 = torch.empty((sg["H_v"], sg["d_k"], sg["d_v"]), device="cuda")
        r_fold = timer.kernel_us([lambda: b.lkv_init_state_fold(states, kk, gg, bb, cu, K, None, S0, workspace_t=ws)], 0, 7)
        r_mat = timer.kernel_us([lambda: b.lkv_init_state(states, trans, K, b.LKV_INIT_EXACT, S0, family=b.LKV_FAMILY_GDN,
                                                          workspace_t=ws)], 0, 7)
        fold.append(dict(K=K, chunk_len=L, fold_us=round(r_fold["us"], 1), materialised_us=round(r_mat["us"], 1),
                         stream_bytes=int(T * (sg["H_k"] * sg["d_k"] * 2 + 2 * sg["H_v"] * 4)),
                         transition_bytes=int((K - 1) * sg["H_v"] * sg["d_k"] * sg["d_k"] * 4),
                         timing="one call per event pair, L2 flushed before it"))
    print(json.dumps(dict(sweep="compose_us_vs_K", fold_vs_materialised=fold, timing="kernels under 100 us: 24 or more launches per CUDA-event pair "
                          "inside one graph, rotating over buffer sets whose total exceeds L2, time divided by the "
                          "launches, median and p90 of 9 replays; longer ones: one launch per event pair after an L2 "
                          "flush, median and p90", rows=rows)))


def run_artifacts(args):
    """--artifacts: time of building the cached artefacts of a batch of cache chunks (64 chunks x 1024 tokens per
    family, benchmark shapes): final-state-only scans from the empty state for S_local, and the chunk transitions /
    log-decays.  Prints one JSON line of its own."""
    import torch

    from paper_2608_11231_b200 import binding as b
    torch.cuda.set_device(0)
    b.load()
    n_chunks, L = 64, 1024
    T = n_chunks * L
    cu = (np.arange(n_chunks + 1) * L).astype(np.int32)
    gen = torch.Generator(device="cuda").manual_seed(11)
    bf = torch.bfloat16
    rn = lambda *shape: torch.randn(shape, generator=gen, device="cuda")
    s, m = GDN_SHAPE, SSD_SHAPE
    k = torch.nn.functional.normalize(rn(T, s["H_k"], s["d_k"]), dim=-1).to(bf)
    q = torch.nn.functional.normalize(rn(T, s["H_k"], s["d_k"]), dim=-1).to(bf)
    v = rn(T, s["H_v"], s["d_v"]).to(bf)
    g = -0.1 * torch.nn.functional.softplus(rn(T, s["H_v"]))
    beta = torch.sigmoid(rn(T, s["H_v"]))
    x = rn(T, m["H"], m["P"]).to(bf)
    dt = torch.nn.functional.softplus(-2.0 + 0.5 * rn(T, m["H"]))
    A = -torch.exp(2.0 * torch.rand(m["H"], generator=gen, device="cuda"))
    Bm = (rn(T, m["G"], m["N"]) / m["N"] ** 0.5).to(bf)
    Cm = (rn(T, m["G"], m["N"]) / m["N"] ** 0.5).to(bf)
    ws = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    st_g = torch.empty((n_chunks, s["H_v"], s["d_k"], s["d_v"]), device="cuda")
    tr_g = torch.empty((n_chunks, s["H_v"], s["d_k"], s["d_k"]), device="cuda")
    st_m = torch.empty((n_chunks, m["H"], m["N"], m["P"]), device="cuda")
    lam = torch.empty((n_chunks, m["H"]), device="cuda")
    calls = {
        "gdn_states": lambda: b.lkv_gdn_fwd(q, k, v, g, beta, None, None, st_g, cu_seqlens=cu, want_outputs=False, workspace_t=ws),
        "gdn_transitions": lambda: b.lkv_gdn_chunk_transition(k, g, beta, tr_g, cu_seqlens=cu, workspace_t=ws),
        "gdn_states_and_transitions_one_launch": lambda: b.lkv_gdn_chunk_artifacts(k, v, g, beta, st_g, tr_g, cu_seqlens=cu,
                                                                                   workspace_t=ws),
        "mamba_states": lambda: b.lkv_ssd_fwd(x, dt, A, Bm, Cm, None, None, st_m, cu_seqlens=cu, want_outputs=False, workspace_t=ws),
        "mamba_logdecays": lambda: b.lkv_mamba_chunk_logdecay(dt, A, lam, cu_seqlens=cu, workspace_t=ws),
    }
    out = {}
    for name, fn in calls.items():
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(max(args.steps, 5)):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            e1.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3)
        us = statistics.median(ts)
        out[name] = dict(us=round(us, 1), tokens_per_s=round(T / us * 1e6))
    print(json.dumps(dict(artifacts="chunk_prefill", chunks=n_chunks, chunk_len=L, timing="CUDA events around one call, "
                          "inputs (about 1.1 GB per family) larger than L2, median", calls=out)))


def run_dry(args):
    """--dry-run: every rank on CPU (gloo); the step is a stand-in that sleeps (rank + 1) ms.  Same request sharding,
    same max-over-ranks time and whole-job token count as the GPU path; rank 0 prints the line."""
    import torch.distributed as dist

    from paper_2608_11231_b200 import sharding
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
    reqs = build_requests(args.workload, rank)
    tokens = sum(r["total"] for r in reqs)
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time.sleep(1e-3 * (rank + 1))
    local_ms = 1e3 * (time.perf_counter() - t0) / args.steps
    d = dist if world > 1 else None
    ms = sharding.job_step_ms(local_ms, d)
    total = sharding.job_total(tokens, d)
    if rank == 0:
        print(json.dumps(dict(metric=METRIC, value=total / (ms * 1e-3), unit=UNIT, n_gpus=world, steps=args.steps,
                              warmup=args.warmup, ms_per_step=ms, higher_is_better=True, scaling="weak",
                              vs_baseline=None, dtype="none", data="none (stand-in step on CPU)",
                              config=dict(workload=args.workload, requests=len(reqs), context_tokens=total,
                                          dry_run=True), gpu_launches=0)))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_profile_case(args):
    """--profile-case NAME: three launches of one kernel on a small fixed case (inputs larger than L2, a few GB at most)
    and nothing else -- the command that ncu captures for the summaries under profiles/."""
    import torch

    from paper_2608_11231_b200 import binding as b
    torch.cuda.set_device(0)
    b.load()
    gen = torch.Generator(device="cuda").manual_seed(3)
    rn = lambda *shape: torch.randn(shape, generator=gen, device="cuda")
    bf = torch.bfloat16
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    name = args.profile_case
    if name == "gdn_scan":
        s, n_seq, L = GDN_SHAPE, 8, 2048
        T = n_seq * L
        nrm = torch.nn.functional.normalize
        q, k = nrm(rn(T, s["H_k"], s["d_k"]), dim=-1).to(bf), nrm(rn(T, s["H_k"], s["d_k"]), dim=-1).to(bf)
        v, g, beta = rn(T, s["H_v"], s["d_v"]).to(bf), -0.1 * torch.nn.functional.softplus(rn(T, s["H_v"])), torch.sigmoid(rn(T, s["H_v"]))
        S0 = rn(n_seq, s["H_v"], s["d_k"], s["d_v"])
        o, ST = torch.empty_like(v), torch.empty_like(S0)
        cu = (np.arange(n_seq + 1) * L).astype(np.int32)
        fn = lambda: b.lkv_gdn_fwd(q, k, v, g, beta, S0, o, ST, cu_seqlens=cu, workspace_t=ws)
        work = dict(tokens=T, flops=gdn_scan_flops(T))
    elif name == "ssd_scan":
        s, n_seq, L = SSD_SHAPE, 16, 4096
        T = n_seq * L
        x = rn(T, s["H"], s["P"]).to(bf)
        dt = torch.nn.functional.softplus(-2.0 + 0.5 * rn(T, s["H"]))
        A = -torch.exp(2.0 * torch.rand(s["H"], generator=gen, device="cuda"))
        Bm, Cm = (rn(T, s["G"], s["N"]) / s["N"] ** 0.5).to(bf), (rn(T, s["G"], s["N"]) / s["N"] ** 0.5).to(bf)
        S0 = rn(n_seq, s["H"], s["N"], s["P"])
        y, ST = torch.empty_like(x), torch.empty_like(S0)
        cu = (np.arange(n_seq + 1) * L).astype(np.int32)
        fn = lambda: b.lkv_ssd_fwd(x, dt, A, Bm, Cm, S0, y, ST, cu_seqlens=cu, workspace_t=ws)
        work = dict(tokens=T, flops=ssd_scan_flops(T))
    elif name in ("gdn_compose", "mamba_compose"):
        n_req, K = (32, 8) if name == "gdn_compose" else (32, 16)
        if name == "gdn_compose":
            H, dk, dv, code = GDN_SHAPE["H_v"], GDN_SHAPE["d_k"], GDN_SHAPE["d_v"], b.LKV_FAMILY_GDN
            trans = rn(n_req * K, H, dk, dk) * (0.45 / dk ** 0.5)
        else:
            H, dk, dv, code = SSD_SHAPE["H"], SSD_SHAPE["N"], SSD_SHAPE["P"], b.LKV_FAMILY_MAMBA2
            trans = -2.0 * torch.rand((n_req * K, H), generator=gen, device="cuda")
        states = rn(n_req * K, H, dk, dv)
        S0 = torch.empty((n_req, H, dk, dv), device="cuda")
        ids, cu_k = np.arange(n_req * K, dtype=np.int32), (np.arange(n_req + 1) * K).astype(np.int32)
        fn = lambda: b.lkv_init_state_batched(states, trans, ids, cu_k, n_req, b.LKV_INIT_EXACT, None, S0, family=code, workspace_t=ws)
        nbytes = (states.numel() + S0.numel()) * 4 + (trans.numel() - (n_req * H * dk * dk if name == "gdn_compose" else 0)) * 4
        work = dict(requests=n_req, K=K, bytes=nbytes)
    else:
        raise SystemExit("unknown profile case")
    ts = []
    for _ in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        e1.synchronize()
        ts.append(1e3 * e0.elapsed_time(e1))
    assert b.lkv_device_status(ws) == b.LKV_OK
    print(json.dumps(dict(profile_case=name, us_per_call=[round(t, 1) for t in ts], **work)))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg4", choices=["cfg1", "cfg2", "cfg3", "cfg4"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sweep", action="store_true", help="composition time against K instead of the step benchmark")
    ap.add_argument("--artifacts", action="store_true", help="time of building chunk states and transitions")
    ap.add_argument("--profile-case", default=None, choices=["gdn_scan", "ssd_scan", "gdn_compose", "mamba_compose"],
                    help="three launches of one kernel on a small fixed case, for an ncu capture")
    ap.add_argument("--no-configs", action="store_true", help="leave the cfg1-cfg3 object out of the default line")
    ap.add_argument("--dry-run", action="store_true",
                    help="ranks on CPU over gloo with a stand-in step: exercises the launch, sharding and timing "
                         "reduction of --gpus N where there are no GPUs")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as a plain script: become the launcher of N ranks of this same command line, one per GPU
        from paper_2608_11231_b200 import sharding
        sys.exit(sharding.launch_ranks(os.path.abspath(__file__), sys.argv[1:], args.gpus))
    if args.dry_run:
        run_dry(args)
        return
    if args.profile_case:
        run_profile_case(args)
        return
    if args.artifacts:
        run_artifacts(args)
    elif args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
