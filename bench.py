#!/usr/bin/env python
"""Benchmark of the IsoQuant hot path: one step = quantize-append of one new K/V row per sequence and KV
head, the fused decode over the packed cache, and the split merge with the inverse rotation.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Prints ONE JSON line. Metric: packed-KV bytes the decode consumes per second (codes + fp32 scales of K
and V, all KV heads, all sequences), whole job. `--impl reference` times the fp64 CPU oracle on a bounded
sample of the same workload.
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

WORKLOADS = {
    # name: (B, ctx, H_q, H_kv, d) -- the batched serving sweep; lengths ragged in [0.5, 1.0] x ctx
    "config5_B32_ctx32768": (32, 32768, 64, 8, 128),
    "config5_B8_ctx32768": (8, 32768, 64, 8, 128),
    "config5_B1_ctx32768": (1, 32768, 64, 8, 128),
    "config5_B32_ctx4096": (32, 4096, 64, 8, 128),
    "config5_B8_ctx4096": (8, 4096, 64, 8, 128),
    "config5_B1_ctx4096": (1, 4096, 64, 8, 128),
    # one sequence of a million rows: the same shape far beyond the paper's 32 K (0.8 GB of packed cache, 4 GB as fp16)
    "config5_B1_ctx1048576": (1, 1048576, 64, 8, 128),
    # the wide-head shape of config 3 (d = 256, 16 query / 8 KV heads) as a ragged batch that exceeds L2
    "d256_B32_ctx16384": (32, 16384, 16, 8, 256),
    # single-sequence shapes (configs 3 and 4) as a stack of 48 per-layer caches of full length, every layer with its own
    # three launches of batch 1: the caches of the stack exceed L2 together, a step is one pass over the layers
    "config3_48layers": (48, 16384, 16, 8, 256),
    "config4_48layers": (48, 32768, 32, 8, 128),
}
PER_SEQUENCE_LAUNCHES = {"config3_48layers", "config4_48layers"}
DEFAULT_WORKLOAD = "config5_B32_ctx32768"
T_CAP_MARGIN = 2048  # rows of head-room so that every sequence can take the benchmark's appends

# DRAM traffic of one decode launch, from two ncu captures of the decode kernel (summarised under profiles/): a
# one-pass capture of the two DRAM byte counters on the full B = 32 launch (dram__bytes_read.sum = 614.22 MB for
# 612.32 MB of algorithmic packed-KV bytes; dram__bytes_write.sum = 7.8 and 11.0 MB for 2.13 MB of partial results,
# S = 2 slots) and the multi-pass capture at B = 8 (182.60 MB for 182.01 MB; 5.69 MB for 1.33 MB of partials, S = 5).
# Both give reads = 1.003 x the algorithmic bytes and writes = 4.3 - 4.4 x the partial results (the rest of the
# writes are dirty lines of the kernels before it leaving L2). Reads scale with the rows processed, writes with the
# partial results. The bench line's roofline.traffic is this MODEL applied to the workload it runs, and says so.
NCU_READ_PER_ALGORITHMIC_BYTE = 614.22 / 612.32
NCU_WRITE_PER_PARTIAL_BYTE = 0.5 * (7.76 + 11.02) / 2.13


GRAPH_EVENT_STRIDE = 4


def decode_traffic_bytes(algorithmic_bytes: float, B: int, H_q: int, S: int, d: int) -> int:
    partial_bytes = B * H_q * S * (d + 2) * 4
    return int(NCU_READ_PER_ALGORITHMIC_BYTE * algorithmic_bytes + NCU_WRITE_PER_PARTIAL_BYTE * partial_bytes)


def bytes_per_row(d: int) -> int:
    return 2 * (BITS * d // 8) + 2 * (2 if SCALES_F16 else 4)   # K and V codes + scales, per cached row per KV head


def measured_peak_hbm():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
    except Exception:
        return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clocks, power and throttle reasons through NVML (read-only) every few ms while the timed region runs."""

    def __init__(self, gpu_index: int, period_s: float = 0.004):
        self.gpu, self.period = gpu_index, period_s
        self.samples, self.reasons, self.stop_flag, self.thread, self.err = [], set(), False, None, None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            idx = self.gpu
            if vis:
                try:
                    idx = int(vis.split(",")[self.gpu])
                except ValueError:
                    idx = self.gpu
            self.h = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.nv = pynvml
            self.smax = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception as e:  # noqa: BLE001
            self.err = repr(e)
            return
        self.thread = threading.Thread(target=self._run, daemon=True)
        self.thread.start()

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": nv.nvmlClocksEventReasonHwSlowdown, "hw_thermal_slowdown": nv.nvmlClocksEventReasonHwThermalSlowdown,
                 "sw_thermal_slowdown": nv.nvmlClocksEventReasonSwThermalSlowdown, "sw_power_cap": nv.nvmlClocksEventReasonSwPowerCap}
        while not self.stop_flag:
            try:
                self.samples.append((nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM), nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception as e:  # noqa: BLE001
                self.err = repr(e)
                break
            time.sleep(self.period)

    def stop(self):
        self.stop_flag = True
        if self.thread is not None:
            self.thread.join(timeout=2)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "error": self.err}
        sm = [c for c, _ in self.samples]
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": self.smax, "reasons": sorted(self.reasons), "samples": len(sm),
                "power_w_max": round(max(p for _, p in self.samples), 1)}


def init_distributed(world: int, local_rank: int, backend: str = "nccl") -> None:
    """One process per GPU; rendezvous on 127.0.0.1 unless the launcher says otherwise. The data path has no
    collective: the group is used for the barrier around the timed region and the max-over-ranks time."""
    if world <= 1:
        return
    import torch.distributed as dist
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29531")
    if backend == "nccl":
        import torch
        torch.cuda.set_device(local_rank)
    dist.init_process_group(backend)


def max_over_ranks(ms: float, world: int, device=None) -> float:
    """The slowest rank's time: every multi-GPU number is reported against it."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    tt = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def aggregate_gbs(bytes_per_rank: float, ms: float, world: int) -> float:
    """Whole-job throughput of `world` replicas that each moved bytes_per_rank in ms (weak scaling)."""
    return world * bytes_per_rank / (ms * 1e-3) / 1e9


SCALES_F16 = False  # binary16 scale arrays: 100 instead of 104 bytes per cached row and KV head
PAGE_ROWS = 0       # > 0: the cache is a pool of pages of this many rows behind a block table in scrambled order
BITS = 3            # bits per code (Algorithm 1's b); the paper's and the benchmark's configurations are 3-bit
CODEBOOK = "int8"   # "int8": Lloyd-Max levels on an 8-bit grid (integer tensor-core decode path); "fp16": exact fp16 levels


def build_state(name: str, device, rank: int):
    """Synthetic cache for one rank: seeded K/V generated on the GPU in chunks and bulk-quantized (untimed)."""
    import torch

    import paper_2608_08081_b200 as iq
    import workloads

    B, ctx, H_q, H_kv, d = WORKLOADS[name]
    gen = workloads.config5_device(B, ctx, device, H_q, H_kv, d, full_lengths=name in PER_SEQUENCE_LAUNCHES)
    t_cap = ctx + T_CAP_MARGIN
    shape = iq.Shape(B, H_q, H_kv, d, t_cap, bits=BITS)
    cb = iq.iq_lloyd_max_codebook(d, BITS, CODEBOOK)
    rot = torch.empty(iq.iq_rotation_floats(d, H_kv), dtype=torch.float32, device=device)
    iq.iq_make_rotation(d, H_kv, 0, np.ascontiguousarray(gen["quats"]), rot)
    if PAGE_ROWS:
        assert t_cap % PAGE_ROWS == 0, "--page-rows must divide the capacity (ctx + 2048)"
        n_tab = t_cap // PAGE_ROWS
        perm = np.random.Generator(np.random.Philox(77 + rank)).permutation(B * n_tab).astype(np.int32)
        cache = iq.new_paged_cache(shape, B * n_tab, PAGE_ROWS, torch.from_numpy(perm.reshape(B, n_tab)).to(device), device,
                                   scales_dtype=torch.float16 if SCALES_F16 else torch.float32)
    else:
        cache = iq.new_cache(shape, device, scales_dtype=torch.float16 if SCALES_F16 else torch.float32)
    status = torch.zeros(4, dtype=torch.int32, device=device)
    lens_np = gen["lens"].astype(np.int32)
    qa_ms, qa_rows = 0.0, 0
    for b0, k, v in gen["chunks"]():
        nb = k.shape[0]
        sub = iq.Shape(nb, H_q, H_kv, d, t_cap, bits=BITS)
        if PAGE_ROWS:   # the pool is shared; the chunk's sequences are rows b0 .. b0 + nb of the block table
            view = iq.Cache(cache.k_codes, cache.k_scales, cache.v_codes, cache.v_scales, cache.block_table[b0:b0 + nb], PAGE_ROWS)
        else:
            view = iq.Cache(cache.k_codes[b0:b0 + nb], cache.k_scales[b0:b0 + nb], cache.v_codes[b0:b0 + nb], cache.v_scales[b0:b0 + nb])
        pos = torch.zeros(nb, dtype=torch.int32, device=device)
        nn = torch.from_numpy(lens_np[b0:b0 + nb]).to(device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        iq.iq_quantize_append(sub, rot, cb, k, v, pos, nn, ctx, view, status)   # bulk compression at the prefill boundary
        e1.record()
        torch.cuda.synchronize()
        if b0 > 0:   # the first chunk warms up
            qa_ms += e0.elapsed_time(e1)
            qa_rows += int(lens_np[b0:b0 + nb].astype(np.int64).sum()) * H_kv * 2
        del k, v
    qa = None
    if qa_rows:
        bytes_per_row = 2 * d + BITS * d // 8 + 4   # fp16 in + packed codes + fp32 scale out
        peak, _ = measured_peak_hbm()
        gbs = qa_rows * bytes_per_row / (qa_ms * 1e-3) / 1e9
        qa = {"rows_per_s": round(qa_rows / (qa_ms * 1e-3), 1), "gb_per_s": round(gbs, 1), "frac_of_hbm_peak": round(gbs / peak, 4),
              "rows": qa_rows, "bytes_per_row": bytes_per_row, "what": "bulk iq_quantize_append of the prefill (K and V rows), CUDA events"}
    return dict(iq=iq, shape=shape, cb=cb, rot=rot, cache=cache, status=status, lens_np=lens_np, q0=gen["q"], quats=gen["quats"],
                B=B, ctx=ctx, H_q=H_q, H_kv=H_kv, d=d, t_cap=t_cap, quantize_append=qa)


def step_inputs(st, n_steps: int, device, seed: int):
    """Pre-drawn per-step inputs (same law as the cache rows): q [n][B][H_q][d], k/v [n][B][1][H_kv][d], fp16."""
    import torch

    g = torch.Generator(device=device)
    g.manual_seed(seed)
    B, H_q, H_kv, d = st["B"], st["H_q"], st["H_kv"], st["d"]
    q = torch.randn((n_steps, B, H_q, d), generator=g, device=device).to(torch.float16)
    k = torch.randn((n_steps, B, 1, H_kv, d), generator=g, device=device).to(torch.float16)
    v = torch.randn((n_steps, B, 1, H_kv, d), generator=g, device=device).to(torch.float16)
    return q, k, v


class StepRunner:
    """One workload on one GPU: its packed cache, the per-step inputs, the launches of a step, and a CUDA graph of K
    steps whose decode launches are bracketed by event-record nodes."""

    def __init__(self, name: str, device, rank: int, K: int, W: int, splits: int = 0):
        import torch

        self.torch = torch
        self.name, self.device, self.K, self.W = name, device, K, W
        self.st = st = build_state(name, device, rank)
        iq = self.iq = st["iq"]
        self.B, self.H_q, self.H_kv, self.d = st["B"], st["H_q"], st["H_kv"], st["d"]
        # Launch groups: the whole batch in one set of launches, or (stack-of-layers workloads) one set per sequence.
        self.per_seq = name in PER_SEQUENCE_LAUNCHES
        self.gshape = iq.Shape(1, self.H_q, self.H_kv, self.d, st["t_cap"], bits=BITS) if self.per_seq else st["shape"]
        self.S = splits or iq.iq_suggest_splits(self.gshape, st["ctx"])
        self.ws = iq.DecodeWorkspace(st["shape"], self.S, want_argmax=False, device=device)
        # Row i of this table holds the sequence lengths before step i: the step appends at lens_tab[i] and attends to
        # lens_tab[i + 1] rows (the serving engine knows the lengths; no kernel is spent on incrementing them).
        lens0 = torch.from_numpy(st["lens_np"]).to(device)
        self.lens_tab = (lens0[None, :] + torch.arange(K + W + 4, device=device, dtype=torch.int32)[:, None]).contiguous()
        self.q_all, self.k_all, self.v_all = step_inputs(st, K + W, device, 99 + rank)
        B = self.B
        self.groups = [slice(b, b + 1) for b in range(B)] if self.per_seq else [slice(0, B)]
        cache = st["cache"]
        if PAGE_ROWS:
            self.gcache = [iq.Cache(cache.k_codes, cache.k_scales, cache.v_codes, cache.v_scales, cache.block_table[g], PAGE_ROWS) for g in self.groups]
        else:
            self.gcache = [iq.Cache(cache.k_codes[g], cache.k_scales[g], cache.v_codes[g], cache.v_scales[g]) for g in self.groups]
        self.n_groups = len(self.groups)
        # Small launch groups take the one-call step whose decode launch also appends (iq_decode_step_fused: two launches);
        # a group whose decode launch is bracketed by event records takes the three separate calls, so that the records
        # can sit between them. For larger groups the one-call step enqueues the same three launches anyway.
        gB = 1 if self.per_seq else B
        self.one_call = BITS == 3 and gB * self.H_kv * (1 + self.H_q // self.H_kv) <= 180
        self.step_ws = torch.empty(max(iq.iq_decode_step_workspace_bytes(self.gshape, self.S), 16), dtype=torch.uint8, device=device) if self.one_call else None
        self.launch_count = 0   # kernels launched by launches() since the counter was last cleared
        self.graph, self.graph_evs, self.graph_error = None, None, None
        self.side = torch.cuda.Stream(device=device)   # carries the event records that bracket decode launches

    def _stamp(self, event):
        """Records `event` on the side stream at the point the launching stream has reached, WITHOUT putting anything
        between the kernels of the launching stream: under graph capture the record becomes a sibling node that depends
        on the kernel before it, and the next kernel keeps its direct (programmatic) dependency on that kernel. An event
        node placed between two kernels would serialise them and add about 5 us to the launch it brackets."""
        torch = self.torch
        main = torch.cuda.current_stream()
        here = torch.cuda.Event()
        here.record(main)
        self.side.wait_event(here)
        event.record(self.side)

    def launches(self, i, q, k, v, ev=None, out=None):
        """The step's launches on device inputs q [B][H_q][d], k, v [B][1][H_kv][d]: append, decode, combine per group;
        ev = (group, event pair) brackets that group's decode launch."""
        iq, st, ws, S, torch = self.iq, self.st, self.ws, self.S, self.torch
        for j, g in enumerate(self.groups):
            if self.one_call and not (ev is not None and ev[0] == j):
                iq.iq_decode_step_fused(self.gshape, st["rot"], st["cb"], q[g], k[g][:, 0], v[g][:, 0], self.gcache[j], self.lens_tab[i][g], S,
                                        self.step_ws, (ws.out if out is None else out)[g], ws.lse[g], None, ws.status)
                self.launch_count += 2
                continue
            self.launch_count += 3
            iq.iq_quantize_append(self.gshape, st["rot"], st["cb"], k[g], v[g], self.lens_tab[i][g], None, 1, self.gcache[j], st["status"])
            if ev is not None and ev[0] == j:
                self._stamp(ev[1][0])   # fires when the append kernel has completed
            iq.iq_decode_attention(self.gshape, st["rot"], st["cb"], q[g], self.gcache[j], self.lens_tab[i + 1][g], S, ws.part_acc[g], ws.part_ml[g], None, ws.status)
            if ev is not None and ev[0] == j:
                self._stamp(ev[1][1])   # fires when the decode kernel has completed
            iq.iq_combine_splits(self.gshape, st["rot"], S, ws.part_acc[g], ws.part_ml[g], None, (ws.out if out is None else out)[g], ws.lse[g], None)

    def decode_alone(self, n: int = 20, replays: int = 7):
        """The decode launch by itself: a CUDA graph of n decode launches (no append, no merge, no event nodes), replayed;
        returns the median time per launch in ms, or None without a graph. Consecutive launches overlap their set-up with
        the tail of the one before (programmatic dependent launch), as they do behind the append kernel in a step."""
        iq, st, ws, S, torch = self.iq, self.st, self.ws, self.S, self.torch
        i = self.W   # lengths of the first timed step

        def launches():
            for _ in range(n):
                for j, g in enumerate(self.groups):
                    iq.iq_decode_attention(self.gshape, st["rot"], st["cb"], self.q_all[i][g], self.gcache[j], self.lens_tab[i + 1][g], S,
                                           ws.part_acc[g], ws.part_ml[g], None, ws.status)
        try:
            launches()
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                launches()
            graph.replay()
            torch.cuda.synchronize()
        except Exception:
            return None
        ts = []
        for _ in range(replays):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            graph.replay()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) / (n * self.n_groups))
        del graph
        return float(np.median(ts))

    def one_step(self, i, ev=None):
        self.launches(i, self.q_all[i], self.k_all[i], self.v_all[i], None if ev is None else (i % self.n_groups, ev))

    def warm_up(self):
        for i in range(self.W):
            self.one_step(i)
        self.torch.cuda.synchronize()

    def capture(self):
        """The K timed steps captured once into a CUDA graph: the three launches of a step then follow each other on the
        device as they do under a serving engine's decode graph, instead of waiting for the host's three binding calls.
        Every GRAPH_EVENT_STRIDE-th decode launch is bracketed by two event-record nodes that hang off the kernels beside
        it (see _stamp): the first fires when the append kernel before the decode launch has completed, the second when
        the decode kernel has, so their difference is the time the launch adds to the step's critical path."""
        torch, K, W = self.torch, self.K, self.W
        try:
            self.graph_evs = [(torch.cuda.Event(enable_timing=True, external=True), torch.cuda.Event(enable_timing=True, external=True))
                              for _ in range((K + GRAPH_EVENT_STRIDE - 1) // GRAPH_EVENT_STRIDE)]
            self.graph = torch.cuda.CUDAGraph()
            self.launch_count = 0
            with torch.cuda.graph(self.graph):
                self.side.wait_stream(torch.cuda.current_stream())     # the side stream joins the capture
                for i in range(K):
                    self.one_step(W + i, self.graph_evs[i // GRAPH_EVENT_STRIDE] if i % GRAPH_EVENT_STRIDE == 0 else None)
                torch.cuda.current_stream().wait_stream(self.side)     # and is joined back before the capture ends
            self.graph_launches = self.launch_count                    # kernels in one replay
            self.graph.replay()                                        # untimed: first replay of a new graph
            torch.cuda.synchronize()
        except Exception as e:  # noqa: BLE001 -- reported in the JSON line; the host-launched loop is timed instead
            self.graph, self.graph_error = None, f"{type(e).__name__}: {e}"[:200]
            torch.cuda.synchronize()

    def timed_pass(self, run_k_steps, evs, barrier=None):
        """One call of run_k_steps (exactly K steps) between two events on the launching stream, a synchronize on both
        sides; the event pairs in evs bracket decode launches inside it."""
        torch = self.torch
        stream = torch.cuda.current_stream()
        torch.cuda.synchronize()
        if barrier is not None:
            barrier()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        run_k_steps()
        t1.record(stream)
        torch.cuda.synchronize()
        return t0.elapsed_time(t1), [a.elapsed_time(b) for a, b in evs]

    def timed_region(self, min_region_s: float, max_replays: int = 100000, barrier=None):
        """The timed region: the K-step graph replayed R times, each replay timed on its own (events and a synchronize
        on both sides), until the replays add up to min_region_s. With no graph: the host-launched K steps, R times.
        Returns (per-replay ms, decode-launch ms of every bracketed launch)."""
        K = self.K
        if self.graph is not None:
            run, evs = self.graph.replay, self.graph_evs
        else:
            eager_evs = [(self.torch.cuda.Event(enable_timing=True), self.torch.cuda.Event(enable_timing=True)) for _ in range(K)]

            def run():
                for i in range(K):
                    self.one_step(self.W + i, eager_evs[i])
            evs = eager_evs
        per_replay, dec = [], []
        while True:
            ms, d = self.timed_pass(run, evs, barrier)
            per_replay.append(ms)
            dec.extend(d)
            if len(per_replay) >= max_replays or (sum(per_replay) >= 1e3 * min_region_s and len(dec) >= 50):
                break
        return per_replay, dec

    def rows_at_first_timed_step(self) -> int:
        return int(self.st["lens_np"].astype(np.int64).sum()) + self.B * self.W

    def bytes_of_steps(self):
        rows = self.rows_at_first_timed_step()
        return [(rows + self.B * (i + 1)) * self.H_kv * bytes_per_row(self.d) for i in range(self.K)]

    def bracketed_launch_bytes(self):
        """Algorithmic bytes of the bracketed decode launches of one pass: one launch per bracketed step, over
        1 / n_groups of the step's rows."""
        b = self.bytes_of_steps()
        return [x / self.n_groups for x in (b[::GRAPH_EVENT_STRIDE] if self.graph is not None else b)]


def point_summary(name: str, device, rank: int, K: int = 20, W: int = 3, min_region_s: float = 0.1):
    """A short measurement of one workload: step time and bracketed decode-launch time under graph replay."""
    import torch

    peak, _ = measured_peak_hbm()
    r = StepRunner(name, device, rank, K, W)
    r.warm_up()
    r.capture()
    per_replay, dec = r.timed_region(min_region_s, max_replays=2000)
    assert int(r.ws.status[0].item()) == 0 and int(r.st["status"][0].item()) == 0, "device status flags set"
    ms_step = float(np.mean(per_replay)) / K
    step_bytes = float(np.mean(r.bytes_of_steps()))
    launch_bytes = float(np.mean(r.bracketed_launch_bytes()))
    dec_ms = float(np.mean(dec))
    out = {"workload": name, "batch": r.B, "ctx": r.st["ctx"], "num_splits": r.S, "launch_groups": r.n_groups,
           "ms_per_step": round(ms_step, 5), "step_gb_per_s": round(step_bytes / (ms_step * 1e-3) / 1e9, 1),
           "decode_tokens_per_s": round(r.B / (ms_step * 1e-3), 1),
           "decode_launch_ms": round(dec_ms, 5), "decode_gb_per_s": round(launch_bytes / (dec_ms * 1e-3) / 1e9, 1),
           "decode_frac_of_hbm_peak": round(launch_bytes / (dec_ms * 1e-3) / 1e9 / peak, 4),
           "algorithmic_bytes_per_step": int(step_bytes), "replays": len(per_replay), "decode_launches_timed": len(dec)}
    if r.graph_error:
        out["graph_error"] = r.graph_error
    del r
    torch.cuda.empty_cache()
    return out


SWEEP_POINTS = ["config5_B1_ctx4096", "config5_B8_ctx4096", "config5_B32_ctx4096",
                "config5_B1_ctx32768", "config5_B8_ctx32768", "config5_B32_ctx32768"]
TARGET_FRAC_OF_PEAK = 0.70   # the stated target: fused decode over a 32K-token packed cache at >= 70 % of the HBM peak


def run_ours(args, rank: int, world: int, local_rank: int):
    import torch
    import torch.distributed as dist

    global CODEBOOK, BITS
    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    K, W = args.steps, args.warmup
    r = StepRunner(args.workload, device, rank, K, W, args.splits)
    st, iq, ws = r.st, r.iq, r.ws
    shape, cb, rot, cache = st["shape"], st["cb"], st["rot"], st["cache"]
    B, H_q, H_kv, d, S, n_groups = r.B, r.H_q, r.H_kv, r.d, r.S, r.n_groups
    stream = torch.cuda.current_stream()
    r.warm_up()
    if not args.no_graph:
        r.capture()
    barrier = dist.barrier if world > 1 else None

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    # the host-launched loop once (reported beside the graph replay; it is the timed region with --no-graph)
    eager_evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]

    def eager_k_steps():
        for i in range(K):
            r.one_step(W + i, eager_evs[i])

    r.launch_count = 0
    eager_ms, eager_dec_ms = r.timed_pass(eager_k_steps, eager_evs, barrier)
    eager_launches = r.launch_count   # kernels of one pass of the K host-launched steps
    # the timed region: the K steps R times, until it lasts args.min_region seconds (whatever --steps is)
    per_replay, dec_ms = r.timed_region(args.min_region, barrier=barrier)
    clocks = sampler.stop() if rank == 0 else None
    alone_ms = r.decode_alone() if not args.no_graph else None
    assert int(ws.status[0].item()) == 0 and int(st["status"][0].item()) == 0, "device status flags set"
    R = len(per_replay)
    bytes_steps = r.bytes_of_steps()
    ms_total = max_over_ranks(float(sum(per_replay)), world, device)
    eager_ms = max_over_ranks(eager_ms, world, device)
    rows = r.rows_at_first_timed_step()

    # ---- end to end through the C-ABI binding with host buffers: H2D of the step inputs and D2H of the output inside the timed region
    # the step's host inputs (q, new k, new v) sit in one pinned staging buffer per step and travel in one copy
    nq, nk = B * H_q * d, B * H_kv * d
    q_all, k_all, v_all, lens_tab = r.q_all, r.k_all, r.v_all, r.lens_tab
    hin = torch.cat([q_all[:W + K].reshape(W + K, nq), k_all[:W + K].reshape(W + K, nk), v_all[:W + K].reshape(W + K, nk)], dim=1).cpu().pin_memory()
    din = torch.empty(nq + 2 * nk, dtype=torch.float16, device=device)
    dq = din[:nq].view(B, H_q, d); dk = din[nq:nq + nk].view(B, 1, H_kv, d); dv = din[nq + nk:].view(B, 1, H_kv, d)
    out16 = torch.empty((B, H_q, d), dtype=torch.float16, device=device)   # the result travels as binary16, like q, k and v
    hout = torch.empty((B, H_q, d), dtype=torch.float16).pin_memory()

    stepper = None if r.per_seq else iq.HostStepper(shape, rot, cb, hin, din, lens_tab, cache, ws, out16, hout)   # every argument marshalled once

    def e2e_step(i):
        if r.per_seq:   # a stack of layers: the copies once, the launches per layer
            din.copy_(hin[i], non_blocking=True)
            r.launches(i, dq, dk, dv, out=out16)
            hout.copy_(out16, non_blocking=True)
            torch.cuda.synchronize()
        else:           # the library's host-buffer call: copy in, append, decode, combine, copy out, wait
            stepper.step(i)

    n_e2e = K
    n_e2e_warm = min(3, W)   # the e2e leg re-appends over the same rows (it restarts from row 0 of the length table)
    for i in range(n_e2e_warm):
        e2e_step(i)
    rows_e2e = int(st["lens_np"].astype(np.int64).sum()) + B * n_e2e_warm
    e2e_bytes_pass = sum((rows_e2e + B * (i + 1)) * H_kv * bytes_per_row(d) for i in range(n_e2e))
    e2e_total_ms, e2e_passes = 0.0, 0
    while e2e_total_ms < 1e3 * min(args.min_region, 0.25) and e2e_passes < 200:   # the same K steps, repeated like the timed region
        if world > 1:
            dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for i in range(n_e2e):
            e2e_step(n_e2e_warm + i)
        e1.record(stream)
        torch.cuda.synchronize()
        e2e_total_ms += e0.elapsed_time(e1)
        e2e_passes += 1
    e2e_ms = max_over_ranks(e2e_total_ms, world, device)

    if rank != 0:
        return None
    peak, peak_src = measured_peak_hbm()
    ms_step = ms_total / (K * R)
    value = aggregate_gbs(sum(bytes_steps) * R, ms_total, world)
    dec_avg_ms = sum(dec_ms) / len(dec_ms)
    timed_launch_bytes = r.bracketed_launch_bytes()        # per pass; every pass brackets the same launches
    launch_bytes = sum(timed_launch_bytes) / len(timed_launch_bytes)
    achieved = launch_bytes / (dec_avg_ms * 1e-3) / 1e9
    step_ms_replays = [m / K for m in per_replay]
    out = {
        "metric": "fused decode packed-KV GB/s",
        "value": round(value, 1),
        "unit": "GB/s",
        "n_gpus": world,
        "steps": K,
        "warmup": W,
        "replays": R,
        "ms_per_step": round(ms_step, 4),
        "ms_per_step_median": round(float(np.median(step_ms_replays)), 4),
        "ms_per_step_cv": round(float(np.std(step_ms_replays) / np.mean(step_ms_replays)), 4),
        "higher_is_better": True,
        "scaling": "weak",
        "vs_baseline": None,
        "dtype": (f"u{BITS} codes, int8 tensor-core operands, int32 accumulate" if CODEBOOK == "int8"
                  else "u3 codes, f16 tensor-core operands, f32 accumulate"),
        "data": "synthetic",
        "config": {"workload": args.workload, "batch": B, "ctx": st["ctx"], "n_q_heads": H_q, "n_kv_heads": H_kv, "head_dim": d,
                   "t_cap": st["t_cap"], "lengths": "ctx" if r.per_seq else "ragged, floor(ctx*U[0.5,1.0])",
                   "launch_groups": n_groups, "ms_per_launch_group": round(ms_step / n_groups, 5), "cached_rows_per_kv_head": rows,
                   "num_splits": S, "bytes_per_row_per_kv_head": bytes_per_row(d), "l2": "inputs_larger_than_l2",
                   "step": ("one-call step (iq_decode_step_fused: the decode launch also appends the new rows, then the merge; two launches), every %d-th step's bracketed group by the three separate calls" % GRAPH_EVENT_STRIDE
                            if r.one_call else "quantize-append 1 row/seq + fused decode + combine"), "codebook": CODEBOOK, "scales": "fp16" if SCALES_F16 else "fp32", "cache": (f"paged, {PAGE_ROWS} rows per page, scrambled" if PAGE_ROWS else "contiguous"), "parallelism": f"replicas x{world}",
                   "timed_region": ((f"{R} replays of a CUDA graph holding the K steps" if r.graph is not None else f"the K steps launched from the host, {R} times")
                                    + ", each replay between its own events and synchronizes; the replays' times are summed")},
        "decode_tokens_per_s": round(world * B / (ms_step * 1e-3), 1),
        "frac_of_8TBs": round(value / world / 8000.0, 4),
        "roofline": {"bound": "hbm", "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s", "frac": round(achieved / peak, 4),
                     "target_frac": TARGET_FRAC_OF_PEAK, "gap_to_target": round(TARGET_FRAC_OF_PEAK - achieved / peak, 4),
                     "traffic": decode_traffic_bytes(launch_bytes, B // n_groups, H_q, S, d),
                     "traffic_source": "MODELLED from ncu DRAM byte counters of one decode launch (config 5, B = 32, ctx = 32768; reads 1.003 x the algorithmic bytes, writes 4.4 x the partial results), scaled to this workload by rows processed (reads) and partial results (writes); not measured in this run",
                     "kernel": "decode_kernel", "peak_source": peak_src,
                     "avg_launch_ms": round(dec_avg_ms, 4), "median_launch_ms": round(float(np.median(dec_ms)), 4),
                     "launch_ms_cv": round(float(np.std(dec_ms) / np.mean(dec_ms)), 4), "launches_timed": len(dec_ms),
                     "timing": ("CUDA event-record nodes beside every %d-th decode launch of the replayed graph: from the completion of the kernel before it to its own completion (sibling nodes: the kernels keep their direct dependencies)" % GRAPH_EVENT_STRIDE
                                if r.graph is not None else "CUDA events on a side stream beside every decode launch: from the completion of the kernel before it to its own completion"),
                     "algorithmic_bytes_per_launch": int(launch_bytes),
                     "launch_alone": (None if not alone_ms else {
                         "ms": round(alone_ms, 4), "gb_per_s": round(launch_bytes / (alone_ms * 1e-3) / 1e9, 1),
                         "frac": round(launch_bytes / (alone_ms * 1e-3) / 1e9 / peak, 4),
                         "what": "the same decode launch in a CUDA graph of 20 decode launches and nothing else (median of 7 replays, outside the timed region): what the event nodes and the neighbouring small kernels add to the bracketed figure above is the difference"})},
        "e2e": {"value": round(aggregate_gbs(e2e_bytes_pass * e2e_passes, e2e_ms, world), 1), "unit": "GB/s",
                "h2d_bytes_per_step": int(B * (H_q + 2 * H_kv) * d * 2), "d2h_bytes_per_step": int(B * H_q * d * 2),
                "ms_per_step": round(e2e_ms / max(n_e2e * e2e_passes, 1), 4), "steps": n_e2e * e2e_passes,
                "note": "packed cache is device-resident state; per-step inputs (q, new k/v) come from pinned host memory in one copy, the output (binary16) returns to pinned host memory, one synchronize per step; iq_decode_step_host through a stepper that marshals its arguments once"},
        "host_launched": {"value": round(aggregate_gbs(sum(bytes_steps), eager_ms, world), 1), "unit": "GB/s",
                          "ms_per_step": round(eager_ms / K, 4), "decode_launch_ms": round(sum(eager_dec_ms) / K, 4),
                          "note": "the same K steps launched call by call from the host (three binding calls per step), one pass"},
        "quantize_append": st["quantize_append"],
        # counted as they are enqueued: per step and launch group quantize_append_few_kernel, decode_kernel, combine_kernel, or
        # (one-call step of a small group) the decode kernel that also appends, and combine_kernel
        "gpu_launches": (r.graph_launches if r.graph is not None else eager_launches) * R,
        "clocks": clocks,
    }
    if clocks and clocks.get("sm_mhz"):
        out["clocks"]["ms_per_step_x_sm_mhz"] = round(ms_step * clocks["sm_mhz"], 2)   # clock-normalised step time
    if r.graph_error:
        out["graph_error"] = r.graph_error
    if not args.no_materialised and world == 1 and not r.per_seq:
        out["reconstruct_then_compute"] = materialised_baseline(st, lens_tab[W + K], q_all[W + K - 1], ws, S, peak)
    if not args.no_cpu_baseline and world == 1 and not PAGE_ROWS and not SCALES_F16:
        out["cpu_baseline"] = cpu_baseline(st, lens_tab[n_e2e_warm + n_e2e], q_all[W + K - 1])
    # ---- the other points of the serving sweep and the fp16-codebook path, each measured briefly in the same run
    if not args.no_sweep and world == 1 and args.workload == DEFAULT_WORKLOAD and not PAGE_ROWS and not SCALES_F16:
        main = {"workload": args.workload, "batch": B, "ctx": st["ctx"], "num_splits": S, "launch_groups": n_groups,
                "ms_per_step": round(ms_step, 5), "step_gb_per_s": round(value, 1), "decode_tokens_per_s": out["decode_tokens_per_s"],
                "decode_launch_ms": round(dec_avg_ms, 5), "decode_gb_per_s": round(achieved, 1), "decode_frac_of_hbm_peak": round(achieved / peak, 4),
                "algorithmic_bytes_per_step": int(np.mean(bytes_steps)), "replays": R, "decode_launches_timed": len(dec_ms)}
        del r, st, ws, cache, q_all, k_all, v_all, lens_tab, hin, din, dq, dk, dv
        torch.cuda.empty_cache()
        main_cb = CODEBOOK
        out["sweep"] = {"what": "config 5: batch {1, 8, 32} x ctx {4096, 32768}, ragged lengths; step = append + decode + combine under graph replay, decode launch between event nodes",
                        "points": [main if n == args.workload else point_summary(n, device, rank) for n in SWEEP_POINTS]}
        CODEBOOK = "fp16" if main_cb == "int8" else "int8"
        try:
            o = point_summary(args.workload, device, rank)
            o["codebook"] = CODEBOOK
            out["decode_fp16_codebook" if CODEBOOK == "fp16" else "decode_int8_codebook"] = o
        finally:
            CODEBOOK = main_cb
        # the other bit widths of Algorithm 1 on the same workload (cache rebuilt at that width; the paper's setting is 3 bits)
        out["other_bit_widths"] = {}
        for b in (2, 4):
            BITS = b
            try:
                o = point_summary(args.workload, device, rank)
                o["bits"] = b
                o["bytes_per_row_per_kv_head"] = bytes_per_row(d)
                out["other_bit_widths"][str(b)] = o
            finally:
                BITS = 3
    return out


def materialised_baseline(st, lens_dev, q, ws, S, peak):
    """The execution model the fused path replaces, on the same packed cache and the same step: iq_reconstruct_rows
    writes the whole cache back as fp16 K/V, a library attention kernel (flash_attn) attends to them. Reported beside
    the fused step, not part of it."""
    import torch

    iq, shape, cb, rot, cache = st["iq"], st["shape"], st["cb"], st["rot"], st["cache"]
    B, H_q, H_kv, d, T = st["B"], st["H_q"], st["H_kv"], st["d"], st["t_cap"]
    lens_dev = lens_dev.contiguous()
    rows = int(lens_dev.sum().item())
    res = {"what": "iq_reconstruct_rows (packed cache -> fp16 K/V, every cached row) + flash_attn_with_kvcache on the fp16 tensors; CUDA events",
           "fp16_kv_bytes": rows * H_kv * d * 2 * 2}
    try:
        k = torch.empty((B, T, H_kv, d), dtype=torch.float16, device=lens_dev.device)
        v = torch.empty_like(k)
    except torch.OutOfMemoryError as e:
        res["unavailable"] = f"fp16 K/V do not fit: {e}"[:160]
        return res

    def timed(f, reps):
        f()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            f()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    rec_ms = timed(lambda: iq.iq_reconstruct_rows(shape, rot, cb, cache, lens_dev, k, v), 3)
    rec_bytes = rows * H_kv * (bytes_per_row(d) + 2 * d * 2)           # packed rows in, fp16 K and V rows out
    res["reconstruct_ms"] = round(rec_ms, 4)
    res["reconstruct_gb_per_s"] = round(rec_bytes / (rec_ms * 1e-3) / 1e9, 1)
    res["fp16_attention_ms_at_hbm_peak"] = round(res["fp16_kv_bytes"] / (peak * 1e9) * 1e3, 4)   # a perfect fp16 kernel
    iq.decode_step(shape, rot, cb, q, cache, lens_dev, ws)             # the fused path on the same query and lengths
    try:
        from flash_attn import flash_attn_with_kvcache

        q4 = q.reshape(B, 1, H_q, d)
        att_ms = timed(lambda: flash_attn_with_kvcache(q4, k, v, cache_seqlens=lens_dev), 10)
        o = flash_attn_with_kvcache(q4, k, v, cache_seqlens=lens_dev).reshape(B, H_q, d).float()
        res["fp16_attention_ms"] = round(att_ms, 4)
        res["fp16_attention_kernel"] = "flash_attn.flash_attn_with_kvcache"
        res["max_abs_diff_vs_fused"] = float((o - ws.out.float()).abs().max().item())   # fp16 K/V rounding shifts the logits
        res["max_abs_out"] = float(ws.out.float().abs().max().item())
        res["ms_per_step"] = round(rec_ms + att_ms, 4)
    except Exception as e:  # noqa: BLE001 -- the library kernel is optional; the reconstruction time stands on its own
        res["fp16_attention_ms"] = None
        res["fp16_attention_error"] = f"{type(e).__name__}: {e}"[:160]
    del k, v
    return res


def cpu_baseline(st, lens, q_last, target_s: float = 12.0):
    """The fp64 oracle, as it stands, timed on this machine's host cores on a bounded sample of the same workload: the
    decode of the whole batch's cache (a copy of the device cache), repeated until about `target_s` seconds of CPU
    work have been spent."""
    import oracle

    nb = st["B"]
    cache = {k: getattr(st["cache"], k)[:nb].cpu().numpy() for k in ("k_codes", "k_scales", "v_codes", "v_scales")}
    ln = lens[:nb].cpu().numpy().astype(np.int32)
    q = q_last[:nb].cpu().numpy()
    lv = np.array(st["cb"].levels, np.float32)
    nbytes = int(ln.astype(np.int64).sum()) * st["H_kv"] * bytes_per_row(st["d"])
    total, reps = 0.0, 0
    while reps < 1 or (total < target_s and reps < 16):
        t0 = time.perf_counter()
        oracle.decode_attention(st["quats"], lv, q, cache, ln, st["H_kv"])
        total += time.perf_counter() - t0
        reps += 1
    res = {"value": round(reps * nbytes / total / 1e9, 4), "unit": "GB/s", "cores": oracle.num_threads(), "kind": "oracle",
           "sample": f"{reps} x decode of all {nb} sequences (all {st['H_q']} query heads, {nbytes / 1e6:.0f} MB of packed cache), "
                     f"{total:.1f} s"}
    # the same oracle on one thread, on the first sequence alone
    threads = oracle.num_threads()
    oracle.set_num_threads(1)
    try:
        one = {k: v[:1] for k, v in cache.items()}
        t0 = time.perf_counter()
        oracle.decode_attention(st["quats"], lv, q[:1], one, ln[:1], st["H_kv"])
        t1 = time.perf_counter() - t0
        res["value_1_thread"] = round(int(ln[0]) * st["H_kv"] * bytes_per_row(st["d"]) / t1 / 1e9, 4)
    finally:
        oracle.set_num_threads(threads)
    return res


def run_reference(args, rank: int, world: int):
    """Reference arm: the oracle on host cores, on a bounded sample of the same workload, generated on the host."""
    if rank != 0:
        return None
    import oracle
    import workloads
    from oracle import lloyd_max

    B, ctx, H_q, H_kv, d = WORKLOADS[args.workload]
    lens_all = workloads.config5_lengths(B, ctx)
    nb = 1
    T = int(lens_all[0])
    g = np.random.Generator(np.random.Philox(workloads.stream_seed(5, 0) + 7))
    lv, th = lloyd_max.int8_codebook(d, 1 << BITS) if CODEBOOK == "int8" else lloyd_max.fp16_codebook(d, 1 << BITS)
    quats = workloads.quaternion_pairs(workloads.rng(5, workloads.QUAT_STREAM), H_kv, d)
    P = oracle.row_bytes(d, BITS)
    cache = oracle.new_cache(nb, H_kv, d, workloads.cap128(T + args.warmup + args.steps + 1), BITS)
    # the sample's cache content: uniformly random codes and Gaussian-row-like scales (the decode cost does not depend on values)
    cache["k_codes"][:] = g.integers(0, 256, cache["k_codes"].shape, dtype=np.uint8)
    cache["v_codes"][:] = g.integers(0, 256, cache["v_codes"].shape, dtype=np.uint8)
    cache["k_scales"][:] = np.sqrt(d) * (1 + 0.05 * g.standard_normal(cache["k_scales"].shape))
    cache["v_scales"][:] = np.sqrt(d) * (1 + 0.05 * g.standard_normal(cache["v_scales"].shape))
    times = []
    lens = np.array([T], np.int32)
    for i in range(args.warmup + args.steps):
        k1 = workloads.to_fp16(g.standard_normal((nb, 1, H_kv, d)))
        v1 = workloads.to_fp16(g.standard_normal((nb, 1, H_kv, d)))
        q1 = workloads.to_fp16(g.standard_normal((nb, H_q, d)))
        t0 = time.perf_counter()
        oracle.quantize_append(quats, th, k1, v1, lens, None, cache)
        lens = lens + 1
        oracle.decode_attention(quats, lv, q1, cache, lens, H_kv)
        dt = time.perf_counter() - t0
        if i >= args.warmup:
            times.append((dt, int(lens[0]) * H_kv * bytes_per_row(d)))
    tot_t = sum(t for t, _ in times)
    tot_b = sum(b for _, b in times)
    val = round(tot_b / tot_t / 1e9, 4)
    sample = f"each step: quantize-append + decode of 1 of {B} sequences ({T} rows x {H_kv} KV heads, {H_q} query heads)"
    return {"impl": "reference", "metric": "fused decode packed-KV GB/s", "value": val, "unit": "GB/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(1e3 * tot_t / max(len(times), 1), 3),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "sample": sample},
            "cpu_baseline": {"value": val, "unit": "GB/s", "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--splits", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-materialised", action="store_true", help="skip the reconstruct-then-compute comparison")
    ap.add_argument("--scales", default="fp32", choices=["fp32", "fp16"], help="precision of the stored row norms")
    ap.add_argument("--page-rows", type=int, default=0, help="paged cache: rows per page (multiple of 128 dividing ctx + 2048), pages in scrambled order")
    ap.add_argument("--no-graph", action="store_true", help="time the host-launched loop instead of a CUDA-graph replay of the K steps")
    ap.add_argument("--min-region", type=float, default=0.5, help="seconds the timed region must last: the K steps are repeated until it does")
    ap.add_argument("--no-sweep", action="store_true", help="skip the other config-5 points and the other codebook's decode path")
    ap.add_argument("--codebook", default="int8", choices=["int8", "fp16"])
    ap.add_argument("--bits", type=int, default=3, choices=[2, 3, 4], help="bits per code (the headline configuration is 3)")
    args = ap.parse_args()
    global CODEBOOK, PAGE_ROWS, SCALES_F16, BITS
    BITS = args.bits
    SCALES_F16 = args.scales == "fp16"
    CODEBOOK = args.codebook
    PAGE_ROWS = args.page_rows
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        out = run_reference(args, rank, world)
        if out is not None:
            print(json.dumps(out), flush=True)
        return
    if args.steps + args.warmup + 8 > T_CAP_MARGIN:
        raise SystemExit(f"--steps + --warmup must stay below {T_CAP_MARGIN - 8}")
    init_distributed(world, local_rank, "nccl")
    out = run_ours(args, rank, world, local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()
    if out is not None:
        print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
