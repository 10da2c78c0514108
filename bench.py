#!/usr/bin/env python
"""Benchmark of the chunked-prefill attention path (libpdd) on B200.

One "step" is one pass of the whole hot path over one synthetic prompt: every prefill
chunk and the received-token append (KV append + causal attention + window column sums),
then importance reduction and top-k keep mask.  The default workload is the largest
single-GPU configuration, the long prompt: 32 query / 8 KV heads, head_dim 128,
32768-token prompt in chunks of 2048 plus 256 received tokens, 1 % outlier keys, keep
ratio 0.2.  The same line carries an `also` list with the other configurations (the
Llama-7B-shaped 4096-token layer, the 16 ragged sequences, and the 28-layer stack with its
projection GEMMs done by torch and timed apart).  Short workloads repeat the pass inside a
step so that the timed region spans enough clock samples whatever --steps is.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--workload c4|c2|c5|c3|c1|c3l|c4s|c4w] [--window last|all] [--no-also]

Prints ONE JSON line (rank 0).  `value` is tokens/s with inputs resident in HBM; `e2e`
is the same metric through the C ABI with pinned-host inputs copied inside the timed
region and the keep mask read back.  `roofline` covers the attention kernel (tensor
bound): algorithmic flops (4*d per unmasked query-key pair per head) over its
event-timed duration, against the measured dense bf16 peak.  `cpu_baseline` times the
CPU checker, as it stands, on a bounded sample of the same workload.
With N > 1 every rank runs an independent replica on its own GPU (the path does not
shard); value is the aggregate over ranks, time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2508_09035_b200 import workloads as wl  # noqa: E402

NOMINAL_BF16_TFLOPS = 2250.0
# One ncu capture of the attention kernel (dram__bytes_read.sum + dram__bytes_write.sum of one
# launch) on the small long-prompt case: the 2048-row chunk at pos0 = 6144 of an 8192-token
# prompt.  DRAM traffic of this kernel grows in proportion to its algorithmic bytes (q + out +
# one read of the sequence's K and V per call), so `roofline.traffic` scales the capture to the
# mean launch of the timed workload.  The capture belongs to one version of the kernel source:
# if csrc/attn_tc.cuh has changed since (first 12 hex digits of its sha256), traffic is null.
FWD_ATTN_TRAFFIC_CAPTURE = dict(dram_bytes=69.590e6, algorithmic_bytes=67.109e6,
                                source_sha256="65d70472c945")
TARGET_TIMED_MS = 120.0          # a timed region at least this long (>= 20 clock samples at 4 ms)
FALLBACK_BF16_TFLOPS = 1590.0
FALLBACK_HBM_GBS = 6650.0


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(bf16=float(d["bf16_tflops"]), bf16_sustained=float(d.get("bf16_tflops_sustained", 0)),
                    hbm=float(d["hbm_gbs"]), source="measured")
    return dict(bf16=FALLBACK_BF16_TFLOPS, bf16_sustained=1400.0, hbm=FALLBACK_HBM_GBS,
                source="fallback")


def get_workload(name: str, window: str) -> wl.Workload:
    if name == "c1":
        return wl.config_c1(window)
    if name == "c2":
        return wl.config_c2(window)
    if name == "c4":
        return wl.config_c4(window)
    if name == "c5":
        return wl.config_c5(window)
    if name == "c3":
        raise SystemExit("c3 is the layer stack: it has its own runner (StackRunner)")
    if name == "c3l":
        # One layer of config 3's attention stack (12 query / 2 KV heads, 8192-token prompt in
        # chunks of 1024, 128 received tokens after every chunk, every prompt row in the
        # observation window) on N(0,1) q/k/v standing in for the projected activations.
        calls, kind = wl.make_calls(8192, 1024, 0, "all", interleave_received=128)
        q, k, v = wl.normal_qkv(wl.rng_for(2), int(kind.shape[0]), 12, 2, 128)
        return wl.Workload("c3_one_layer_l8192", 12, 2, 128, 64, 0.5,
                           [wl.Sequence(q, k, v, kind, calls)], 1024, 1.0 / float(np.sqrt(128)),
                           "one layer of the 28-layer stack: 12/2 heads, d=128, 8192-token prompt in "
                           "chunks of 1024 with 128 received tokens after each chunk")
    if name == "c4s":       # config 4 recipe cut to 8192 tokens: a small case for profiling
        return wl.config_c4(window, n_prompt=8192, chunk=2048, n_received=256)
    if name == "c4w":       # config 4 under a 4096-key sliding window (the device model's attention)
        import dataclasses
        base = wl.config_c4(window)
        return dataclasses.replace(base, name=base.name + "_w4096", sliding_window=4096,
                                   description=base.description + ", sliding window 4096")
    raise SystemExit("unknown workload %s" % name)


class ClockSampler(threading.Thread):
    """Samples SM clock, power and throttle reasons while the timed region runs.

    Reads NVML in-process every few milliseconds (the timed region of a short run is only
    milliseconds long); falls back to an nvidia-smi loop if NVML cannot be loaded.  Only
    reads: no clock, power or mode setting is touched.  mark() brackets the timed region;
    the summary uses the samples inside it (all samples if none fell inside)."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    REASON_BITS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40),
                   ("sw_thermal_slowdown", 0x20), ("sw_power_cap", 0x4))

    def __init__(self, gpu_index: int, uuid: str = ""):
        super().__init__(daemon=True)
        self.gpu_index, self.uuid = gpu_index, uuid
        self.rows, self.times = [], []
        self.proc = None
        self.marks = []
        self._stop = threading.Event()
        self.source = "none"

    def mark(self):
        self.marks.append(time.perf_counter())

    def _run_nvml(self) -> bool:
        try:
            import pynvml
            pynvml.nvmlInit()
            if self.uuid:
                h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + self.uuid).encode())
            else:
                h = pynvml.nvmlDeviceGetHandleByIndex(self.gpu_index)
            mx = pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM)
        except Exception:
            return False
        self.source = "nvml"
        act = lambda bit, mask: "Active" if mask & bit else "Not Active"
        while not self._stop.is_set():
            try:
                sm = pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)
                pw = pynvml.nvmlDeviceGetPowerUsage(h) / 1000.0
                try:
                    mask = pynvml.nvmlDeviceGetCurrentClocksEventReasons(h)
                except Exception:
                    mask = pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                self.times.append(time.perf_counter())
                self.rows.append([str(sm), str(mx), "%.1f" % pw, hex(mask)] +
                                 [act(bit, mask) for _, bit in self.REASON_BITS])
            except Exception:
                pass
            time.sleep(0.004)
        return True

    def run(self):
        if self._run_nvml():
            return
        try:
            self.source = "nvidia-smi"
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            for line in self.proc.stdout:
                self.times.append(time.perf_counter())
                self.rows.append([x.strip() for x in line.split(",")])
        except Exception:
            pass

    def stop(self):
        self._stop.set()
        if self.proc is not None:
            self.proc.terminate()
        rows = self.rows
        if len(self.marks) >= 2 and len(self.times) == len(rows):
            inside = [r for r, t in zip(rows, self.times) if self.marks[0] <= t <= self.marks[-1]]
            rows = inside or rows
        sm, mx, reasons = [], [], set()
        for r in rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except Exception:
                continue
            for (n, _), v in zip(self.REASON_BITS, r[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        return dict(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)),
                    reasons=sorted(reasons), samples=len(sm), source=self.source)


def dist_setup(n_gpus: int):
    """Rank, world size and a barrier/max-reduce pair.  One process per GPU."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        backend = "nccl" if __import__("torch").cuda.is_available() else "gloo"
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if not dist.is_initialized():
            dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world, local


def aggregate_over_ranks(ms_local: float, units_local: float, world: int, device=None):
    """Whole-job figures for independent replicas: time = max over ranks, units = sum."""
    if world == 1:
        return ms_local, units_local
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms_local], dtype=torch.float64, device=device or "cpu")
    u = torch.tensor([units_local], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def to_bf16_tensor(x: np.ndarray, pin: bool = False):
    import torch
    bits = wl.bf16_bits(x).view(np.int16)
    t = torch.from_numpy(bits.copy())
    if pin:
        t = t.pin_memory()
    return t.view(torch.bfloat16)


def grouped_calls(w: wl.Workload):
    """The workload's calls as batched library calls: prompt chunk t of every sequence that
    still has one goes into one call (split by window flag), then one call with all blocks of
    received tokens.  A single sequence keeps its calls in their own order."""
    if len(w.seqs) == 1:
        return [(c.kind, c.window, [(0, c)]) for c in w.seqs[0].calls]
    out = []
    prompt_calls = [[c for c in s.calls if c.kind == wl.PROMPT] for s in w.seqs]
    for t in range(max(len(pc) for pc in prompt_calls)):
        group = [(si, pc[t]) for si, pc in enumerate(prompt_calls) if t < len(pc)]
        for win in (False, True):
            sub = [(si, c) for si, c in group if c.window == win]
            if sub:
                out.append((wl.PROMPT, win, sub))
    group = [(si, c) for si, s in enumerate(w.seqs) for c in s.calls if c.kind == wl.RECEIVED]
    if group:
        out.append((wl.RECEIVED, False, group))
    return out


class Runner:
    """Holds device-resident and pinned-host copies of the workload's calls and replays them
    through the C ABI with pre-marshalled arguments (the per-call Python work is one ctypes
    call).  Several sequences are driven by batched calls."""

    def __init__(self, w: wl.Workload, device):
        import ctypes
        import torch
        from paper_2508_09035_b200 import binding as B
        self.torch, self.B, self.w, self.device = torch, B, w, device
        self.lib = B.lib()
        self.n_seqs = len(w.seqs)
        groups = grouped_calls(w)
        max_rows = max(sum(c.length for _, c in g) for _, _, g in groups)
        self.total_tokens = sum(s.n_tokens for s in w.seqs)
        self.kv = B.KVCache(w.n_q_heads, w.n_kv_heads, w.head_dim, page_tokens=w.page_tokens,
                            max_seqs=self.n_seqs, max_tokens_total=self.total_tokens,
                            max_tokens_per_seq=max(s.n_tokens for s in w.seqs),
                            max_rows_per_call=max_rows,
                            softmax_scale=w.softmax_scale, device=device,
                            sliding_window=w.sliding_window)
        self.out = torch.empty((max_rows, w.n_q_heads, w.head_dim), dtype=torch.bfloat16,
                               device=device)
        # Per call: q|k|v rows of the call (all its sequences, packed) back to back, once
        # resident on the device and once in pinned host memory with a device staging buffer
        # for the end-to-end arm.  The attention output of every call lands in one buffer.
        self.calls = []
        self.h2d_bytes = 0
        for kind, window, group in groups:
            parts = [torch.cat([to_bf16_tensor(getattr(w.seqs[si], name)[c.pos0:c.pos0 + c.length])
                                .reshape(-1) for si, c in group]) for name in ("q", "k", "v")]
            host = torch.cat(parts).pin_memory()
            dev = host.to(device)
            stage = torch.empty_like(dev)
            nq, nk = parts[0].numel(), parts[1].numel()
            batch, keep = B.make_batch([si for si, _ in group], [c.pos0 for _, c in group],
                                       [c.length for _, c in group])
            fn = self.lib.pdd_prefill_chunk if kind == wl.PROMPT else self.lib.pdd_append_received

            def ptrs(t):
                p = t.data_ptr()
                return p, p + 2 * nq, p + 2 * (nq + nk)
            self.calls.append(dict(fn=fn, batch=batch, keep=keep, host=host, dev=dev, stage=stage,
                                   dev_ptrs=ptrs(dev), stage_ptrs=ptrs(stage),
                                   out_ptr=self.out.data_ptr(),
                                   flags=B.PDD_WINDOW if window else 0,
                                   bref=ctypes.byref(batch)))
            self.h2d_bytes += host.numel() * 2
        # scores, kinds and keep mask of all sequences packed back to back
        self.offsets = [0]
        for s in w.seqs:
            self.offsets.append(self.offsets[-1] + s.n_tokens)
        n = self.total_tokens
        self.score = torch.zeros(n, dtype=torch.float32, device=device)
        self.kinds = torch.from_numpy(np.concatenate([s.kind for s in w.seqs])).to(device)
        self.keep = torch.empty(n, dtype=torch.uint8, device=device)
        self.n_kept = torch.zeros(self.n_seqs, dtype=torch.int32, device=device)
        self.keep_host = torch.empty(n, dtype=torch.uint8).pin_memory()
        self.n_kept_host = torch.zeros(self.n_seqs, dtype=torch.int32).pin_memory()
        self.flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=device)
        self.d2h_bytes = n + 4 * self.n_seqs
        self.stream = self.kv.stream
        self.seq_ids = (ctypes.c_int32 * self.n_seqs)(*range(self.n_seqs))
        self.topk_args = ((ctypes.c_int64 * (self.n_seqs + 1))(*self.offsets),
                          (ctypes.c_int64 * self.n_seqs)(*([0] * self.n_seqs)),
                          (ctypes.c_int64 * self.n_seqs)(*[s.n_tokens for s in w.seqs]))
        # End-to-end arm: host-to-device copies run on a stream of their own, one event per
        # call, so that the copy of call i+1 overlaps the kernels of call i.
        self.topk_events = None
        self.copy_stream = torch.cuda.Stream(device=device)
        self.copied = [torch.cuda.Event() for _ in self.calls]
        self.step_begin = torch.cuda.Event()

    def flush_l2(self):
        self.flush_buf.fill_(1)

    def backlog(self, ms: float = 1.0):
        """Keeps the GPU busy for about `ms` so that the host can run ahead of it; the
        following launches then execute back to back and event pairs around them measure
        device time rather than launch latency."""
        self.torch.cuda._sleep(int(ms * 1.9e6))

    def step(self, e2e: bool = False):
        """One pass of the hot path.  e2e: each call's inputs come from pinned host memory
        (one copy per call) and the keep mask is read back."""
        B, lib, h, st, w = self.B, self.lib, self.kv.h, self.stream, self.w
        torch = self.torch
        rc = 0
        for si in range(self.n_seqs):
            rc |= lib.pdd_kv_reset(h, si, st)
        if e2e:
            # The copies start inside the timed region (after this point of the compute
            # stream, which also orders them after the previous step's use of the staging
            # buffers) and every call waits for its own inputs only.
            self.step_begin.record()
            self.copy_stream.wait_event(self.step_begin)
            with torch.cuda.stream(self.copy_stream):
                for c, ev in zip(self.calls, self.copied):
                    c["stage"].copy_(c["host"], non_blocking=True)
                    ev.record()
        for i, c in enumerate(self.calls):
            if e2e:
                torch.cuda.current_stream().wait_event(self.copied[i])
                q, k, v = c["stage_ptrs"]
            else:
                q, k, v = c["dev_ptrs"]
            rc |= c["fn"](h, c["bref"], q, k, v, c["out_ptr"], c["flags"], st)
        if self.n_seqs == 1:
            # one sequence: importance reduction and selection through one call
            rc |= lib.pdd_importance_topk(h, 0, B.PDD_POOL_NONE, 1, self.score.data_ptr(), 0, 0,
                                          self.total_tokens, float(w.keep_ratio),
                                          self.keep.data_ptr(), self.n_kept.data_ptr(), st)
        else:
            rc |= lib.pdd_token_importance_batched(h, self.n_seqs, self.seq_ids, B.PDD_POOL_NONE, 1,
                                                   self.score.data_ptr(), self.topk_args[0], 0, st)
            if self.topk_events is not None:  # the handle-free top-k is not in the library's trace
                ev = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                ev[0].record()
            rc |= lib.pdd_refine_topk_batched(self.score.data_ptr(), self.kinds.data_ptr(),
                                              self.n_seqs, self.topk_args[0], self.topk_args[1],
                                              self.topk_args[2], float(w.keep_ratio),
                                              self.keep.data_ptr(), self.n_kept.data_ptr(), st)
            if self.topk_events is not None:
                ev[1].record()
                self.topk_events.append(ev)
        if rc:
            raise RuntimeError("libpdd call failed: %s" % lib.pdd_last_error_detail().decode())
        if e2e:
            self.keep_host.copy_(self.keep, non_blocking=True)
            self.n_kept_host.copy_(self.n_kept, non_blocking=True)

    def timed(self, steps: int, e2e: bool) -> float:
        """Sum of per-step device times (ms); L2 is flushed between steps, outside the
        event pairs."""
        torch = self.torch
        evs = []
        for _ in range(steps):
            self.flush_l2()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            self.step(e2e)
            b.record()
            evs.append((a, b))
        torch.cuda.synchronize(self.device)
        return float(sum(a.elapsed_time(b) for a, b in evs))


def kernel_table(trace, trace_steps: int, w: wl.Workload, peaks) -> dict:
    """Per-kernel launches and event-timed milliseconds of the traced passes; for the kernels
    that only move data, also the algorithmic bytes of one pass over their time (GB/s) and the
    fraction of the measured copy bandwidth.  Those kernels run a few microseconds per launch,
    so their figures are launch- and latency-bound, not bandwidth-bound."""
    n_tokens = sum(s.n_tokens for s in w.seqs)
    row_kv = 2 * w.n_kv_heads * w.head_dim * 2            # K and V bytes of one position
    per_pass = {
        # read the call's k, v rows and write them into the cache; one kind byte per position
        "kv_append": 2 * n_tokens * row_kv + n_tokens,
        # read fp32 column sums of every head, write one fp32 score per position
        "importance_reduce": 4 * n_tokens * (w.n_q_heads + 1),
        # scores (fp32) read once into shared memory; kind (1 byte) read by the counting pass,
        # the three radix passes and the mask pass; the mask pass writes one byte
        "radix_topk": n_tokens * (4 + 5 + 1),
    }
    out = {}
    for k, (c, ms) in trace.items():
        e = dict(launches=c, total_ms=ms)
        if k in per_pass and ms > 0:
            gbs = per_pass[k] * trace_steps / (ms * 1e-3) / 1e9
            e.update(algorithmic_bytes_per_pass=per_pass[k], achieved_gbs=gbs,
                     frac_of_hbm_peak=gbs / peaks["hbm"])
        out[k] = e
    return out


def oracle_sample(w: wl.Workload, stride: int):
    """Time the CPU checker on every `stride`-th query row (all heads) of the workload plus
    the full importance/top-k tail.  Evenly spaced rows cost the same on average as all
    rows, so rows/second estimates whole-prompt tokens/second."""
    from oracle import pdd_oracle as orc
    sw = w.sliding_window
    n_rows, dt = 0, 0.0
    for si, s in enumerate(w.seqs):
        rows = np.arange(stride - 1, s.n_tokens, stride)
        if len(rows) == 0:
            continue
        q64, k64, v64 = (a.astype(np.float64) for a in (s.q, s.k, s.v))
        if si == 0:
            orc.attention_rows(q64, k64, v64, w.softmax_scale, rows[:1], sw)    # load the library
        t0 = time.perf_counter()
        orc.attention_rows(q64, k64, v64, w.softmax_scale, rows, sw)
        win = np.zeros(s.n_tokens, dtype=np.uint8)
        for c in s.calls:
            if c.window:
                win[c.pos0:c.pos0 + c.length] = 1
        sub = np.zeros_like(win)
        sub[rows] = win[rows]
        cs = orc.colsum(q64, k64, w.softmax_scale, sub, sw)
        score = orc.importance([cs])
        orc.refine_topk(score, s.kind, 0, s.n_tokens, w.keep_ratio)
        dt += time.perf_counter() - t0
        n_rows += len(rows)
    return n_rows, dt, orc.threads()


def run_reference(args, rank: int, world: int):
    """The CPU checker as the reference arm: rank 0 only, bounded sample per step."""
    if rank != 0:
        return
    w = get_workload(args.workload, args.window)
    stride = args.ref_stride or max(8, w.n_tokens // 256)
    for _ in range(args.warmup):
        oracle_sample(w, stride * 8)
    t_total, rows_total, cores = 0.0, 0, 1
    for _ in range(args.steps):
        n, dt, cores = oracle_sample(w, stride)
        t_total += dt
        rows_total += n
    value = rows_total / t_total
    sample = "every %d-th query row, all heads, %d rows per step" % (stride, rows_total // args.steps)
    line = dict(metric="prefill_tokens_per_s", value=value, unit="tokens/s", impl="reference",
                n_gpus=args.gpus, steps=args.steps, warmup=args.warmup,
                ms_per_step=1e3 * t_total / args.steps, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=w.name, description=w.description, window=args.window,
                            keep_ratio=w.keep_ratio, passes_per_step=1, parallelism="1 gpu"),
                cpu_baseline=dict(value=value, unit="tokens/s", cores=cores, kind="oracle",
                                  sample=sample),
                e2e=dict(value=value, unit="tokens/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line), flush=True)


def attention_source_tag() -> str:
    import hashlib
    path = os.path.join(ROOT, "paper_2508_09035_b200", "csrc", "attn_tc.cuh")
    try:
        return hashlib.sha256(open(path, "rb").read()).hexdigest()[:12]
    except OSError:
        return ""


def attention_bytes_per_launch(w: wl.Workload) -> float:
    """Algorithmic HBM bytes of the mean attention launch of a workload: q and out of the
    call's rows plus one read of K and V of every sequence of the call up to its new length."""
    per_row_q = w.n_q_heads * w.head_dim * 2
    per_pos_kv = 2 * w.n_kv_heads * w.head_dim * 2
    groups = grouped_calls(w)
    total = 0
    for _, _, group in groups:
        for _, c in group:
            total += 2 * c.length * per_row_q + (c.pos0 + c.length) * per_pos_kv
    return total / max(len(groups), 1)


def scaled_traffic(w: wl.Workload):
    cap = FWD_ATTN_TRAFFIC_CAPTURE
    if not cap["dram_bytes"] or cap["source_sha256"] != attention_source_tag():
        return None
    return cap["dram_bytes"] * attention_bytes_per_launch(w) / cap["algorithmic_bytes"]


class StackRunner:
    """Config 3: the 28-layer decoder attention stack.  Per call and layer:
    x -> RMSNorm -> Wq, Wk, Wv (torch bf16 GEMMs) -> libpdd attention call -> Wo -> residual;
    one pdd_kv handle per layer; importance accumulated over the layers, then one top-k.
    The projections are glue, not part of the attention path: they are timed apart (the same
    torch ops without the library calls) and counted in tokens/s only."""

    def __init__(self, st: wl.LayerStack, device):
        import ctypes
        import torch
        from paper_2508_09035_b200 import binding as B
        self.torch, self.B, self.st, self.device = torch, B, st, device
        self.lib = B.lib()
        T = len(st.token_ids)
        self.total_tokens = T
        hq, hkv, d = st.n_q_heads, st.n_kv_heads, st.head_dim
        self.max_rows = max(c.length for c in st.calls)
        self.caches = [B.KVCache(hq, hkv, d, page_tokens=128, max_seqs=1, max_tokens_total=T,
                                 max_tokens_per_seq=T, max_rows_per_call=self.max_rows,
                                 device=device) for _ in range(st.n_layers)]
        self.W = [{n: to_bf16_tensor(st.weight(l, n)).to(device) for n in "qkvo"}
                  for l in range(st.n_layers)]
        self.x_host = to_bf16_tensor(st.embedding_rows(st.token_ids), pin=True)
        self.x_dev = self.x_host.to(device)
        self.x_stage = torch.empty_like(self.x_dev)
        self.out = torch.zeros((self.max_rows, hq, d), dtype=torch.bfloat16, device=device)
        self.calls = []
        for c in st.calls:
            batch, keep = B.make_batch([0], [c.pos0], [c.length])
            fn = self.lib.pdd_prefill_chunk if c.kind == wl.PROMPT else self.lib.pdd_append_received
            self.calls.append(dict(fn=fn, batch=batch, keep=keep, bref=ctypes.byref(batch),
                                   pos0=c.pos0, length=c.length,
                                   flags=B.PDD_WINDOW if c.window else 0))
        self.score = torch.zeros(T, dtype=torch.float32, device=device)
        self.kinds = torch.from_numpy(st.kind.copy()).to(device)
        self.keep = torch.empty(T, dtype=torch.uint8, device=device)
        self.n_kept = torch.zeros(1, dtype=torch.int32, device=device)
        self.keep_host = torch.empty(T, dtype=torch.uint8).pin_memory()
        self.n_kept_host = torch.zeros(1, dtype=torch.int32).pin_memory()
        self.flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=device)
        self.h2d_bytes = self.x_host.numel() * 2
        self.d2h_bytes = T + 4
        self.stream = self.caches[0].stream
        self.n_seqs = 1

    def flush_l2(self):
        self.flush_buf.fill_(1)

    @staticmethod
    def _rmsnorm(torch, x):
        return torch.nn.functional.rms_norm(x, (x.shape[-1],), eps=1e-6)      # unit gain

    def step(self, e2e: bool = False, attention: bool = True):
        """One pass of the stack.  attention=False runs the glue alone (same torch ops, the
        library calls left out) to time the projections."""
        torch, B, lib, st = self.torch, self.B, self.lib, self.st
        hq, hkv, d = st.n_q_heads, st.n_kv_heads, st.head_dim
        rc = 0
        if attention:
            for cch in self.caches:
                rc |= lib.pdd_kv_reset(cch.h, 0, self.stream)
        if e2e:
            self.x_stage.copy_(self.x_host, non_blocking=True)
        x_all = self.x_stage if e2e else self.x_dev
        for c in self.calls:
            x = x_all[c["pos0"]:c["pos0"] + c["length"]]
            out = self.out[:c["length"]]
            for l, cch in enumerate(self.caches):
                h_in = self._rmsnorm(torch, x)
                W = self.W[l]
                q = h_in @ W["q"]
                k = h_in @ W["k"]
                v = h_in @ W["v"]
                if attention:
                    rc |= c["fn"](cch.h, c["bref"], q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                  out.data_ptr(), c["flags"], self.stream)
                x = torch.addmm(x, out.view(-1, hq * d), W["o"])
        if attention:
            for l, cch in enumerate(self.caches):
                rc |= lib.pdd_token_importance(cch.h, 0, B.PDD_POOL_NONE, 1, self.score.data_ptr(),
                                               1 if l > 0 else 0, self.stream)
            rc |= lib.pdd_refine_topk(self.score.data_ptr(), self.kinds.data_ptr(),
                                      self.total_tokens, 0, self.total_tokens,
                                      float(st.keep_ratio), self.keep.data_ptr(),
                                      self.n_kept.data_ptr(), self.stream)
            if rc:
                raise RuntimeError("libpdd call failed: %s" % lib.pdd_last_error_detail().decode())
            if e2e:
                self.keep_host.copy_(self.keep, non_blocking=True)
                self.n_kept_host.copy_(self.n_kept, non_blocking=True)

    def timed(self, steps: int, e2e: bool, passes: int = 1, attention: bool = True) -> float:
        torch = self.torch
        evs = []
        for _ in range(steps * passes):
            self.flush_l2()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            self.step(e2e, attention)
            b.record()
            evs.append((a, b))
        torch.cuda.synchronize(self.device)
        return float(sum(a.elapsed_time(b) for a, b in evs))

    def status(self) -> int:
        return max(c.status() for c in self.caches)

    def trace(self, on: bool):
        for c in self.caches:
            c.trace(on)

    def trace_read(self) -> dict:
        agg = {}
        for c in self.caches:
            for k, (n, ms) in c.trace_read().items():
                a = agg.get(k, (0, 0.0))
                agg[k] = (a[0] + n, a[1] + ms)
        return agg

    def attention_flops(self) -> int:
        T = self.total_tokens
        return 4 * self.st.head_dim * self.st.n_q_heads * (T * (T + 1) // 2) * self.st.n_layers


def measure(name: str, window: str, steps: int, warmup: int, device, local: int, peaks,
            world: int = 1, barrier=None, schedule: int = 0) -> dict:
    """Times one workload: HBM-resident passes, end-to-end passes, then a traced pass for the
    per-kernel figures.  Returns the fields of a bench line (or of an `also` entry)."""
    import torch
    stack = name == "c3"
    if stack:
        st = wl.config_c3()
        runner = StackRunner(st, device)
        tokens, wname = runner.total_tokens, "c3_stack_%dl_l8192" % st.n_layers
        description = ("%d-layer decoder attention stack, 12/2 heads, d=128, hidden 1536, 8192-token "
                       "prompt in chunks of 1024 with 128 received tokens after each chunk, every "
                       "prompt row in the observation window; RMSNorm + Wq/Wk/Wv/Wo by torch" % st.n_layers)
        keep_ratio, flops, w = st.keep_ratio, runner.attention_flops(), None
    else:
        w = get_workload(name, window)
        runner = Runner(w, device)
        if schedule:
            runner.kv.set_schedule(schedule)     # pins one way of cutting the attention work
        tokens, wname, description = w.n_tokens, w.name, w.description
        keep_ratio, flops = w.keep_ratio, w.attention_flops()
    barrier = barrier or (lambda: torch.cuda.synchronize(device))

    for _ in range(warmup):
        runner.step(False)
        runner.step(True)
    torch.cuda.synchronize(device)
    # how many passes make one step: short workloads repeat the pass so that the timed region
    # is long enough for the clock record
    t0 = time.perf_counter()
    runner.step(False)
    torch.cuda.synchronize(device)
    est_ms = max((time.perf_counter() - t0) * 1e3, 1e-3)
    passes = max(1, int(np.ceil(TARGET_TIMED_MS / (est_ms * steps))))
    sampler = ClockSampler(local, str(getattr(torch.cuda.get_device_properties(device), "uuid", "")))
    sampler.start()
    barrier()
    sampler.mark()
    ms_dev = runner.timed(steps, False, passes) if stack else runner.timed(steps * passes, e2e=False)
    barrier()
    ms_e2e = runner.timed(steps, True, passes) if stack else runner.timed(steps * passes, e2e=True)
    barrier()
    sampler.mark()
    clocks = sampler.stop()
    status = runner.status() if stack else runner.kv.status()
    assert status == 0, "device-side error word set"
    n_kept = int(runner.n_kept_host.sum().item())
    glue_ms = None
    if stack:
        glue_ms = runner.timed(min(steps, 2), False, 1, attention=False) / min(steps, 2)

    # per-kernel timing pass (events around every launch; not part of the numbers above)
    trace_steps = min(steps * passes, 2 if stack else 5)
    if stack:
        runner.trace(True)
        for _ in range(trace_steps):
            runner.flush_l2()
            torch.cuda._sleep(int(1.9e6))
            runner.step(False)
            torch.cuda.synchronize(device)
        trace = runner.trace_read()
        runner.trace(False)
    else:
        runner.kv.trace(True)
        runner.topk_events = []
        for _ in range(trace_steps):
            runner.flush_l2()
            runner.backlog(1.0)
            runner.step(False)
            torch.cuda.synchronize(device)
        trace = runner.kv.trace_read()
        runner.kv.trace(False)
        if runner.topk_events:
            trace["radix_topk"] = (len(runner.topk_events),
                                   float(sum(a.elapsed_time(b) for a, b in runner.topk_events)))
        runner.topk_events = None
    launches_per_pass = sum(c for c, _ in trace.values()) // trace_steps
    attn_name = "fwd_attn" if "fwd_attn" in trace else sorted(
        (k for k in trace if k.startswith("attn")), key=lambda k: -trace[k][1])[0]
    attn_cnt, attn_ms = trace[attn_name]
    flops_per_launch = flops / (attn_cnt / trace_steps)
    attn_tflops = flops_per_launch / (attn_ms / attn_cnt * 1e-3) / 1e12
    comb_ms = trace.get("attn_combine", (0, 0.0))[1]
    attn_with_combine = flops * trace_steps / ((attn_ms + comb_ms) * 1e-3) / 1e12

    n_passes = steps * passes
    ms_dev_all, units = aggregate_over_ranks(ms_dev, tokens * n_passes, world, device)
    ms_e2e_all, _ = aggregate_over_ranks(ms_e2e, tokens * n_passes, world, device)
    res = dict(
        workload=wname, description=description, tokens_per_pass=tokens, passes_per_step=passes,
        value=units / (ms_dev_all * 1e-3), ms_per_step=ms_dev_all / steps,
        ms_per_pass=ms_dev_all / n_passes,
        e2e=dict(value=units / (ms_e2e_all * 1e-3), unit="tokens/s",
                 h2d_bytes_per_step=runner.h2d_bytes * passes,
                 d2h_bytes_per_step=runner.d2h_bytes * passes, ms_per_step=ms_e2e_all / steps),
        attention_tflops=attn_tflops, attention_tflops_with_combine=attn_with_combine,
        frac_of_measured_peak=attn_tflops / peaks["bf16"],
        frac_of_nominal_peak=attn_tflops / NOMINAL_BF16_TFLOPS,
        launches_per_pass=int(launches_per_pass), clocks=clocks, n_kept=n_kept,
        keep_ratio=keep_ratio, attn_kernel=attn_name,
        kernels=(kernel_table(trace, trace_steps, w, peaks) if w is not None else
                 {k: dict(launches=c, total_ms=ms) for k, (c, ms) in trace.items()}),
        traffic=scaled_traffic(w) if w is not None else None,
        _workload=w)
    if stack:
        res["projection_glue_ms_per_pass"] = glue_ms
        res["attention_path_ms_per_pass"] = max(ms_dev_all / n_passes - glue_ms, 0.0)
    del runner
    torch.cuda.empty_cache()
    return res


ALSO_WORKLOADS = (("c2", 20), ("c5", 4), ("c3", 2))     # name, steps (each step repeats short passes)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4")
    ap.add_argument("--window", default="last", choices=["last", "all"])
    ap.add_argument("--ref-stride", type=int, default=0)
    ap.add_argument("--cpu-baseline-stride", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-also", action="store_true")
    ap.add_argument("--schedule", type=int, default=0, choices=[0, 1, 2, 3, 4],
                    help="pin how the attention kernel's work is cut (0: the library's cost model)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3

    if args.impl == "reference":
        rank = int(os.environ.get("RANK", "0"))
        run_reference(args, rank, int(os.environ.get("WORLD_SIZE", "1")))
        return

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    rank, world, local = dist_setup(args.gpus)
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    peaks = load_peaks()

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize(device)

    m = measure(args.workload, args.window, args.steps, args.warmup, device, local, peaks, world,
                barrier, args.schedule)
    also = []
    if not args.no_also and world == 1:
        for name, k in ALSO_WORKLOADS:
            if name == args.workload:
                continue
            a = measure(name, args.window, k, 3, device, local, peaks)
            also.append(dict(
                workload=a["workload"], value=a["value"], unit="tokens/s",
                ms_per_step=a["ms_per_step"], ms_per_pass=a["ms_per_pass"],
                passes_per_step=a["passes_per_step"], steps=k,
                e2e_value=a["e2e"]["value"], attention_tflops=a["attention_tflops"],
                attention_tflops_with_combine=a["attention_tflops_with_combine"],
                frac=a["frac_of_measured_peak"], frac_of_nominal_peak=a["frac_of_nominal_peak"],
                launches_per_pass=a["launches_per_pass"], clocks=a["clocks"],
                **({"projection_glue_ms_per_pass": a["projection_glue_ms_per_pass"],
                    "attention_path_ms_per_pass": a["attention_path_ms_per_pass"]}
                   if "projection_glue_ms_per_pass" in a else {})))
    if rank != 0:
        return
    w = m["_workload"]
    line = dict(
        metric="prefill_tokens_per_s", value=m["value"], unit="tokens/s", n_gpus=world,
        steps=args.steps, warmup=args.warmup, ms_per_step=m["ms_per_step"],
        higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16", data="synthetic",
        config=dict(workload=m["workload"], description=m["description"], window=args.window,
                    keep_ratio=m["keep_ratio"], passes_per_step=m["passes_per_step"],
                    l2="flushed between passes (256 MiB write)",
                    e2e_copies="pinned host -> device per call on a copy stream, overlapped with "
                               "the previous call's kernels; keep mask read back; the attention "
                               "output stays on the device (the next layer reads it there)",
                    parallelism="replicas only" if world > 1 else "1 gpu", n_kept=m["n_kept"],
                    **({"attention_schedule": args.schedule} if args.schedule else {})),
        attention_tflops=m["attention_tflops"],
        attention_tflops_with_combine=m["attention_tflops_with_combine"],
        attention_frac_of_nominal_peak=m["frac_of_nominal_peak"],
        e2e=m["e2e"],
        gpu_launches=int(m["launches_per_pass"] * m["passes_per_step"] * args.steps),
        clocks=m["clocks"],
        kernels=m["kernels"],
        roofline=dict(bound="tensor", kernel=m["attn_kernel"], achieved=m["attention_tflops"],
                      peak=peaks["bf16"], unit="TFLOP/s", frac=m["frac_of_measured_peak"],
                      peak_source=peaks["source"] + " burst bf16 (kernel timed alone per launch)",
                      frac_of_sustained_peak=(m["attention_tflops"] / peaks["bf16_sustained"]
                                              if peaks["bf16_sustained"] else None),
                      traffic=m["traffic"],
                      traffic_unit="bytes per launch (dram read + write of one ncu capture of this "
                                   "kernel, scaled by algorithmic bytes to the mean launch)"),
        also=also,
    )
    if m.get("projection_glue_ms_per_pass") is not None:
        line["projection_glue_ms_per_pass"] = m["projection_glue_ms_per_pass"]
    if not args.no_cpu_baseline and w is not None:
        # a bounded sample: whole prompt for the short workloads, every n-th row for the long ones
        tokens = w.n_tokens
        stride = args.cpu_baseline_stride or (1 if tokens <= 8192 else tokens // 2048)
        n, dt, cores = oracle_sample(w, stride)
        line["cpu_baseline"] = dict(value=n / dt, unit="tokens/s", cores=cores, kind="oracle",
                                    sample="every %d-th query row, all heads (%d rows, %.1f s)"
                                           % (stride, n, dt))
    print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
