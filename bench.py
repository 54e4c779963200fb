"""Benchmark of the ADORE decode path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..4] [--impl ours|reference]

A step is one pass of the whole hot path for one new token per sequence: for every layer the
top-K attention over the slot cache (with weight emission and the in-place admit), once per
step the controller + selection, and for every layer the rebuild projection + RoPE + scatter.
Inputs are synthetic (seeded Gaussians of the workload's shapes) and resident in HBM when the
timed region starts; the `e2e` number repeats the steps through the host-buffer entry point.
The K timed steps are replayed (the cache put back to the same state outside the events) until
their device time adds up to about a second; `value` is the median over those repeats. The
default run (config 3) also carries a short run of config 4, the largest one, in `largest_config`.
One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

METRIC = "decode tokens/s (= batch x decode steps/s) at batch B, cache C"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, taken from the committed ncu summary
# named beside it (one capture of the kernel as it stands; None once the kernel has changed since). For the rebuild GEMM
# the capture saw fewer rows than the timed launches: the weight bytes are fixed, the rest (row reads, cache-row
# writes) is scaled by the rows processed.
NCU_TRAFFIC_BYTES = {
    ("rebuild projection", "cfg3_llama7b_b64_c512_rebuild20pct"):
        {"bytes": 278.7e6 + 144.0e6, "rows": 9950.0, "profile": "profiles/rebuild_tc_pair_kernel_cfg3.md"},
    ("rebuild projection", "cfg2_llama7b_b16_c256"):
        {"bytes": 68.2e6 + 1.1e6, "rows": 128.0, "profile": "profiles/rebuild_tc_split_kernel_cfg2.md"},
    ("attention kernel", "cfg3_llama7b_b64_c512_rebuild20pct"):
        {"bytes": 359.1e6 + 6.7e6, "rows": None, "profile": "profiles/attention_tma_kernel_cfg3.md"},
    # config 4's per-layer launch, captured on a one-layer cache of the same shape (the sweep point C=1024, B=32)
    ("attention kernel", "cfg4_llama7b_L32_b32_c1024"):
        {"bytes": 403.4e6 + 4.6e6, "rows": None, "profile": "profiles/attention_tma_kernel_cfg4_shape.md"},
    ("attention kernel", "cfg5_sweep_c1024_b32"):
        {"bytes": 403.4e6 + 4.6e6, "rows": None, "profile": "profiles/attention_tma_kernel_cfg4_shape.md"},
}


def ncu_traffic(kernel, cfg, rows):
    """(bytes per launch or None, the profile the figure comes from or None)"""
    t = NCU_TRAFFIC_BYTES.get((kernel, cfg.name))
    if t is None:
        return None, None
    if t["rows"] is None:
        return t["bytes"], t["profile"]
    fixed = 2 * cfg.n_heads * cfg.head_dim * cfg.hidden * cfg.elem_bytes
    return fixed + (t["bytes"] - fixed) * rows / t["rows"], t["profile"]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def default_steps(cfg: wl.WorkloadConfig):
    return {1: 80, 2: 150, 3: 300, 4: 40}.get(cfg_index(cfg), 40)


def sweep_point(capacity: int, batch: int) -> wl.WorkloadConfig:
    for cap, b, cfg in wl.sweep_points():
        if cap == capacity and b == batch:
            return cfg
    raise SystemExit(f"no sweep point C={capacity} B={batch}")


def run_sweep(args):
    """Capacity x batch sweep: every point in its own process (a fresh context per point)."""
    for cap, b, cfg in wl.sweep_points():
        cmd = [sys.executable, os.path.abspath(__file__), "--config", "5", "--capacity", str(cap), "--batch", str(b),
               "--no-cpu-baseline", "--no-e2e", "--warmup", str(args.warmup), "--min-timed-ms", "300"]
        if args.steps is not None:
            cmd += ["--steps", str(args.steps)]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            print(json.dumps({"workload": cfg.name, "error": res.stderr.strip().splitlines()[-1:]}), flush=True)
            continue
        d = json.loads(res.stdout.strip().splitlines()[-1])
        st = d["stages"]
        print(json.dumps({"workload": cfg.name, "capacity": cap, "batch": b, "steps_per_s": d["steps_per_s"],
                          "tokens_per_s": d["value"], "ms_per_step": d["ms_per_step"],
                          "attention_hbm_frac": st["attention"]["frac"],
                          "attention_plus_selection_hbm_frac": {
                              k: (st["attention_plus_selection"].get(k) or {}).get("frac")
                              for k in ("stages_added", "overlapped", "overlapped_without_controller_tail")},
                          "rebuild": {k: st.get("rebuild", {}).get(k) for k in ("bound", "frac", "rows_per_launch", "ms_per_launch")},
                          "clocks": d["clocks"]}), flush=True)


def cfg_index(cfg):
    for k, v in wl.CONFIGS.items():
        if v.name == cfg.name:
            return k
    return 0


# ------------------------------------------------------------------------------------------------
# distributed plumbing (replicas: sequences are independent, no data-path collective)
# ------------------------------------------------------------------------------------------------
def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def max_over_ranks(value: float, world: int, device) -> float:
    """Largest `value` over all ranks (the slowest rank defines the job's time)."""
    if world == 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(batch_per_rank: int, steps: int, world: int, ms_max: float) -> float:
    return batch_per_rank * world * steps / (ms_max * 1e-3)


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    """nvidia-smi in the background, one sample every 20 ms; window() gives the median SM clock and the throttle reasons
    seen between two time.time() stamps."""
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_index: int):
        self.path = tempfile.mktemp(prefix="adore_clocks_", suffix=".csv")
        self.proc = None
        self.rows = None
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "20", "-i", str(gpu_index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def close(self):
        """Stops the sampler and reads what it wrote: (time, sm MHz, max MHz, power W, [reason flags])."""
        import datetime
        self.rows = []
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        try:
            for line in open(self.path):
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    self.rows.append((ts, float(parts[1]), float(parts[2]), float(parts[3]),
                                      [v.lower().startswith("active") for v in parts[5:9]]))
                except ValueError:
                    continue
            os.unlink(self.path)
        except Exception:
            pass

    def window(self, t_begin: float, t_end: float, what: str):
        if self.rows is None:
            self.close()
        sel = [r for r in self.rows if t_begin - 0.01 <= r[0] <= t_end + 0.01]
        out = {"sm_mhz": None, "sm_max_mhz": None, "power_w": None, "reasons": [], "samples": len(sel), "window": what}
        if sel:
            reasons = sorted({n for r in sel for n, on in zip(self.NAMES, r[4]) if on})
            out.update(sm_mhz=float(np.median([r[1] for r in sel])), sm_max_mhz=sel[-1][2],
                       power_w=float(np.median([r[3] for r in sel])), reasons=reasons)
        return out


# ------------------------------------------------------------------------------------------------
# device-side synthetic workload
# ------------------------------------------------------------------------------------------------
class DeviceRun:
    """Cache + pre-generated per-step inputs on the GPU for `total_steps` decode steps."""

    def __init__(self, cfg: wl.WorkloadConfig, total_steps: int, rank: int, order: str = "attend-first",
                 score_source: str = "controller"):
        import torch
        from paper_2407_02328_b200 import adore as lib
        self.torch, self.lib, self.cfg = torch, lib, cfg
        self.order = order
        c = cfg
        assert total_steps <= c.steps, f"{total_steps} steps asked, the workload has {c.steps}"
        self.dt = torch.float32 if c.dtype == "f32" else torch.bfloat16
        dev = torch.device("cuda")
        g = torch.Generator(device=dev)
        g.manual_seed(c.seed * 1000 + rank)
        B, L, H, dh, d = c.batch, c.n_layers, c.n_heads, c.head_dim, c.hidden
        N = H * dh
        self.stream = torch.cuda.current_stream().cuda_stream
        self.handle = lib.adore_cache_create(
            lib.make_config(batch=B, n_layers=L, n_heads=H, head_dim=dh, hidden=d, capacity=c.capacity,
                            rebuild_max=c.rebuild_max, topk=c.topk, max_tokens=c.max_tokens,
                            ctrl_hidden=c.ctrl_hidden, dtype=c.dtype, rebuild_mode=c.rebuild_mode,
                            rope_theta=c.rope_theta, pos_scale=c.pos_scale,
                            flags={"attention": lib.ADORE_FLAG_SCORE_FROM_ATTENTION,
                                   "controller-relative": lib.ADORE_FLAG_RELATIVE_POSITION}.get(score_source, 0)),
            wl.controller_weights(c), self.stream)

        def randn(*shape, std=1.0):
            return (torch.randn(*shape, generator=g, device=dev, dtype=torch.float32) * std)

        def rows(*shape):
            x = randn(*shape)
            if c.per_layer_inputs:
                x = x * torch.rsqrt(x.pow(2).mean(-1, keepdim=True) + 1e-5)
            return x.to(self.dt)

        def prompt_rows():          # [B, prompt, d], drawn 256 tokens at a time to bound the fp32 temporary
            out = torch.empty((B, c.prompt, d), dtype=self.dt, device=dev)
            for t0 in range(0, c.prompt, 256):
                t1 = min(c.prompt, t0 + 256)
                out[:, t0:t1] = rows(B, t1 - t0, d)
            return out

        if c.identity_projection:
            eye = torch.eye(N, device=dev, dtype=self.dt)
            self.w_kv = [torch.cat([eye, eye], 0).contiguous() for _ in range(L)]
        else:
            self.w_kv = [randn(2 * N, d, std=0.02).to(self.dt).contiguous() for _ in range(L)]
        self.w_q = [randn(N, d, std=0.02).to(self.dt).contiguous() for _ in range(L)]
        for l in range(L):
            lib.adore_cache_set_projection(self.handle, l, self.w_kv[l])
        # prompt
        self.tables = None
        if c.per_layer_inputs:
            self.tables = [torch.zeros((B, c.max_tokens, d), dtype=self.dt, device=dev) for _ in range(L)]
        self.prompt_ms = 0.0        # device time of the prompt's bulk load (controller scan, selection, fill of every layer)
        if c.prompt:
            xp = prompt_rows()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            lib.adore_cache_append_tokens(self.handle, xp, c.prompt)
            lib.adore_cache_join(self.handle)
            e1.record()
            torch.cuda.synchronize()
            self.prompt_ms = e0.elapsed_time(e1)
            if c.per_layer_inputs:
                self.tables[0][:, : c.prompt] = xp
                for l in range(1, L):
                    self.tables[l][:, : c.prompt] = prompt_rows()
                    e0.record()
                    lib.adore_cache_fill_layer(self.handle, l, self.tables[l])
                    lib.adore_cache_join(self.handle)
                    e1.record()
                    torch.cuda.synchronize()
                    self.prompt_ms += e0.elapsed_time(e1)
            del xp
        # per-step inputs
        S = self.S = total_steps
        n_x = L if c.per_layer_inputs else 1
        self.x = rows(S, n_x, B, d).contiguous()
        self.q = torch.empty((S, L, B, H, dh), dtype=self.dt, device=dev)
        self.k = torch.empty_like(self.q)
        self.v = torch.empty_like(self.q)
        for s in range(S):
            n = c.prompt + s
            for l in range(L):
                xl = self.x[s, l if c.per_layer_inputs else 0].float()
                kv = xl @ self.w_kv[l].float().t()
                self.k[s, l] = self._rope(kv[:, :N].reshape(B, H, dh), n).to(self.dt)
                self.v[s, l] = kv[:, N:].reshape(B, H, dh).to(self.dt)
                if c.identity_projection:
                    self.q[s, l] = randn(B, H, dh).to(self.dt)
                else:
                    self.q[s, l] = (c.q_scale * self._rope((xl @ self.w_q[l].float().t()).reshape(B, H, dh), n)).to(self.dt)
                if c.per_layer_inputs:
                    self.tables[l][:, n] = self.x[s, l]
        self.r_in = 0
        self.lists = self.counts = None
        if c.rebuild_mode == "explicit":
            mean = c.max_tokens * c.rebuild_p
            self.r_in = int(min(c.max_tokens, math.ceil(mean + 6 * math.sqrt(mean) + 8)))
            self.lists = torch.full((S, B, self.r_in), -1, dtype=torch.int32, device=dev)
            self.counts = torch.zeros((S, B), dtype=torch.int32, device=dev)
            for s in range(S):
                n = c.prompt + s
                if n == 0:
                    continue
                flag = torch.rand((B, n), generator=g, device=dev) < c.rebuild_p
                key = torch.where(flag, torch.arange(n, device=dev).expand(B, n), torch.full((B, n), 1 << 30, device=dev))
                srt = key.sort(dim=1).values[:, : self.r_in]
                cnt = flag.sum(1).clamp(max=self.r_in).to(torch.int32)
                w = srt.shape[1]
                self.lists[s, :, :w] = torch.where(srt < (1 << 30), srt, torch.full_like(srt, -1)).to(torch.int32)
                self.counts[s] = cnt
        self.out = torch.empty((B, H, dh), dtype=self.dt, device=dev)
        self.weights = torch.empty((B, H, c.capacity + 1), dtype=torch.float32, device=dev)
        self.next = 0
        # device addresses of every step's inputs, taken once: the timed loop then only passes integers
        ptrs = lambda a: [[a[s, l].data_ptr() for l in range(a.shape[1])] for s in range(a.shape[0])]
        self.pq, self.pk, self.pv = ptrs(self.q), ptrs(self.k), ptrs(self.v)
        self.px = [self.x[s, 0].data_ptr() for s in range(self.x.shape[0])]
        self.pl = None if self.lists is None else [self.lists[s].data_ptr() for s in range(self.lists.shape[0])]
        self.pc = None if self.counts is None else [self.counts[s].data_ptr() for s in range(self.counts.shape[0])]
        self.pt = None if self.tables is None else [t.data_ptr() for t in self.tables]
        self.pout, self.pw = self.out.data_ptr(), self.weights.data_ptr()
        if order == "rebuild-first":
            # R_max + 1 query rows per sequence (Section 2.3); the same random rows serve every step
            R1 = c.rebuild_max + 1
            self.q_rows = torch.randn((B, H, R1, dh), generator=g, device=dev, dtype=torch.float32).to(self.dt)
            self.out_rows = torch.empty((B, H, R1, dh), dtype=self.dt, device=dev)
            self.pqr, self.por = self.q_rows.data_ptr(), self.out_rows.data_ptr()
        lib.adore_cache_sync_status(self.handle)

    def _rope(self, y, n):
        c, torch = self.cfg, self.torch
        if c.rope_theta == 0.0:
            return y
        j = torch.arange(c.head_dim // 2, device=y.device, dtype=torch.float64)
        ang = (n * torch.pow(torch.tensor(c.rope_theta, dtype=torch.float64, device=y.device), -2.0 * j / c.head_dim))
        cs, sn = torch.cos(ang).float(), torch.sin(ang).float()
        a, b = y[..., 0::2], y[..., 1::2]
        out = torch.empty_like(y)
        out[..., 0::2] = a * cs - b * sn
        out[..., 1::2] = a * sn + b * cs
        return out

    def step(self):
        lib, c, s = self.lib, self.cfg, self.next
        pl = None if self.pl is None else self.pl[s]
        pc = None if self.pc is None else self.pc[s]
        if self.order == "rebuild-first":
            lib.adore_step_begin(self.handle, self.px[s], pl, pc, self.r_in)
            for l in range(c.n_layers):
                lib.adore_rebuild(self.handle, l, self.pt[l] if (self.pt is not None and l > 0) else None)
                lib.adore_attend_rows(self.handle, l, self.pqr, self.pk[s][l], self.pv[s][l], self.por, None)
            self.next += 1
            return
        for l in range(c.n_layers):
            lib.adore_decode_step(self.handle, l, self.pq[s][l], self.pk[s][l], self.pv[s][l], self.px[s], pl, pc, self.r_in,
                                  self.pout, self.pw)
            lib.adore_rebuild(self.handle, l, self.pt[l] if (self.pt is not None and l > 0) else None)
        self.next += 1

    def make_host_inputs(self, first: int, count: int):
        """Pinned host copies of the inputs of steps first..first+count-1 (for the end-to-end pass)."""
        t = self.torch
        sl = slice(first, first + count)
        pin = lambda a: a.cpu().pin_memory()
        self.h = dict(q=pin(self.q[sl]), k=pin(self.k[sl]), v=pin(self.v[sl]), x=pin(self.x[sl]),
                      lists=None if self.lists is None else pin(self.lists[sl]),
                      counts=None if self.counts is None else pin(self.counts[sl]),
                      out=t.empty((self.cfg.n_layers,) + tuple(self.out.shape), dtype=self.dt).pin_memory())
        self.h_first = first
        # host addresses taken once: the timed loop passes integers only
        h = self.h
        self.hp = dict(q=[[h["q"][i, l].data_ptr() for l in range(h["q"].shape[1])] for i in range(count)],
                       k=[[h["k"][i, l].data_ptr() for l in range(h["k"].shape[1])] for i in range(count)],
                       v=[[h["v"][i, l].data_ptr() for l in range(h["v"].shape[1])] for i in range(count)],
                       x=[h["x"][i, 0].data_ptr() for i in range(count)],
                       lists=None if h["lists"] is None else [h["lists"][i].data_ptr() for i in range(count)],
                       counts=None if h["counts"] is None else [h["counts"][i].data_ptr() for i in range(count)],
                       out=[h["out"][l].data_ptr() for l in range(self.cfg.n_layers)])

    def step_host(self):
        lib, c, s = self.lib, self.cfg, self.next
        i, hp = s - self.h_first, self.hp
        pl = None if hp["lists"] is None else hp["lists"][i]
        pc = None if hp["counts"] is None else hp["counts"][i]
        # the calls of all layers are queued back to back (each layer has its own `out` buffer on the host), then the
        # host waits once for the step's results
        for l in range(c.n_layers):
            lib.adore_decode_rebuild_host_queued(self.handle, l, hp["q"][i][l], hp["k"][i][l], hp["v"][i][l], hp["x"][i], pl, pc,
                                                 self.r_in, self.pt[l] if (self.pt is not None and l > 0) else None,
                                                 hp["out"][l], self.pw)
        lib.adore_cache_wait_outputs(self.handle)
        self.next += 1

    def host_bytes_per_step(self):
        c, e = self.cfg, self.cfg.elem_bytes
        qkv = 3 * c.batch * c.n_heads * c.head_dim * e * c.n_layers
        x = c.batch * c.hidden * e
        lists = (c.batch * self.r_in * 4 + c.batch * 4) if self.lists is not None else 0
        out = c.n_layers * c.batch * c.n_heads * c.head_dim * e      # the weights stay on the device
        return qkv + x + lists, out

    def close(self):
        if self.handle:
            self.lib.adore_cache_destroy(self.handle)
            self.handle = None


# ------------------------------------------------------------------------------------------------
# CPU baseline (the oracle as it stands, on a bounded sample of the workload)
# ------------------------------------------------------------------------------------------------
def time_oracle(cfg: wl.WorkloadConfig, steps: int, warmup: int, budget_s: float = 25.0):
    """Times the numpy oracle on the first sequences (and, for deep stacks, the first layers) of
    the workload. Returns tokens/s scaled to all layers, the threads used and a description."""
    from oracle.harness import Workload, make_oracle, explicit_as_lists
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        threads = os.cpu_count() or 1
    b = 1 if cfg.batch == 1 else 2
    layers = min(cfg.n_layers, 2)
    sample = cfg.scaled(n_layers=layers)
    w = Workload(sample, b)
    orc = make_oracle(w)
    if sample.prompt:
        orc.append_tokens(w.prompt())
    done, t_total = 0, 0.0
    for s in range(warmup + steps):
        n = orc.n
        lists, counts = w.explicit(s, n)
        ex = explicit_as_lists(lists, counts)
        inputs = []
        for l in range(layers):
            x = w.x_new(n, 0)
            inputs.append((x,) + w.qkv(n, l, x))
        t0 = time.perf_counter()
        for l in range(layers):
            x, q, k, v = inputs[l]
            orc.decode_step(l, q, k, v, x if l == 0 else None, ex if l == 0 else None)
            orc.rebuild(l)
        dt = time.perf_counter() - t0
        if s >= warmup:
            done += 1
            t_total += dt
            if t_total > budget_s:
                break
    per_step = t_total / max(done, 1) * (cfg.n_layers / layers)
    desc = (f"first {b} of {cfg.batch} sequences, {layers} of {cfg.n_layers} layers (time scaled by layers), "
            f"{done} decode steps after the prompt; numpy float64 oracle")
    return b / per_step, threads, desc, per_step * 1e3


def run_reference(args, cfg):
    rank, _, world = dist_env()
    if rank != 0:
        return
    value, threads, desc, ms = time_oracle(cfg, args.steps, args.warmup, budget_s=120.0)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": dict(workload_desc(cfg), step_order=args.order, score_source=args.score_source),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def workload_desc(cfg):
    return {"workload": cfg.name, "batch": cfg.batch, "layers": cfg.n_layers, "heads": cfg.n_heads,
            "head_dim": cfg.head_dim, "hidden": cfg.hidden, "capacity": cfg.capacity, "topk": cfg.topk,
            "rebuild_max": cfg.rebuild_max, "rebuild_mode": cfg.rebuild_mode, "rebuild_p": cfg.rebuild_p,
            "prompt": cfg.prompt, "parallelism": "replicas",
            "l2": "inputs larger than L2 (KV cache per step >> 126 MB)" if kv_bytes(cfg) > 2.5e8
            else "L2 flushed between timed iterations"}


def kv_bytes(cfg):
    return 2 * cfg.n_layers * cfg.batch * cfg.n_heads * cfg.capacity * cfg.head_dim * cfg.elem_bytes


# ------------------------------------------------------------------------------------------------
# roofline arithmetic
# ------------------------------------------------------------------------------------------------
def attention_bytes_per_launch(cfg, occ: float) -> float:
    """Algorithmic bytes of one attention launch: all occupied key rows + the current token's, only
    the kept value rows, q and out, the emitted weights, and the admitted K/V row."""
    e, dh = cfg.elem_bytes, cfg.head_dim
    cand = occ + 1
    per_bh = (cand + min(cfg.topk, cand) + 2) * dh * e + (cfg.capacity + 1) * 4 + 2 * dh * e
    return cfg.batch * cfg.n_heads * per_bh


def rebuild_flops_bytes_per_launch(cfg, rows: float):
    n_out = 2 * cfg.n_heads * cfg.head_dim
    flops = 2.0 * rows * cfg.hidden * n_out
    bytes_ = (n_out * cfg.hidden + rows * cfg.hidden + rows * n_out) * cfg.elem_bytes
    return flops, bytes_


def run_labels(args):
    """Times adore_label_tokens on weights of config 4's shape (32 layers x 32 sequences x 32 heads x 1025 slots, K = 512):
    one JSON line with the time per call and the rate at which the weights are read."""
    import torch
    from paper_2407_02328_b200 import build
    build.build()
    from paper_2407_02328_b200 import adore as lib
    cfg = wl.get_config(4)
    L, B, H, S, K = cfg.n_layers, cfg.batch, cfg.n_heads, cfg.capacity + 1, cfg.topk
    g = torch.Generator(device="cuda")
    g.manual_seed(cfg.seed)
    w = torch.rand((L, B, H, S), generator=g, device="cuda") ** 8          # long-tailed
    keep = torch.rand((L, B, H, S), generator=g, device="cuda") < 0.5      # about K positive entries per row
    w = torch.where(keep, w, torch.zeros_like(w))
    w = (w / w.sum(-1, keepdim=True).clamp_min(1e-30)).contiguous()
    sets = torch.empty((L, B, H, K // 2), dtype=torch.int32, device="cuda")
    count = torch.empty((B, S), dtype=torch.int32, device="cuda")
    label = torch.empty((B, S), dtype=torch.uint8, device="cuda")
    cov = torch.empty((L, B), dtype=torch.float32, device="cuda")
    mass = torch.empty_like(cov)
    st = torch.cuda.current_stream().cuda_stream
    call = lambda: lib.adore_label_tokens(w, L, B, H, S, K, st, sets, count, label, cov, mass)
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    n = args.steps or 20
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(n):
        call()
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / n
    peaks, kind = measured_peaks()
    gbs = 2 * w.numel() * 4 / (ms * 1e-3) / 1e9                             # the weights are read twice (sets, statistics)
    print(json.dumps({"metric": "label construction, calls/s", "value": 1e3 / ms, "unit": "calls/s", "ms_per_call": ms,
                      "config": {"workload": "labels_cfg4_shape", "layers": L, "batch": B, "heads": H, "slots": S, "topk": K,
                                 "l2": "weights 134 MB > L2"},
                      "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                   "frac": gbs / peaks["hbm_gbs"], "peak_source": f"{kind} (copy)", "traffic": None},
                      "gpu_launches": 3 * n, "data": "synthetic"}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=3,
                    help="workload 1..4 (default 3: the largest single-layer config); 5 = one point of the capacity x batch "
                         "sweep, chosen with --capacity and --batch")
    ap.add_argument("--capacity", type=int, default=512, help="sweep point: C in {128,256,512,1024,2048}")
    ap.add_argument("--batch", type=int, default=32, help="sweep point: B in {1,8,32,128,256}")
    ap.add_argument("--sweep", action="store_true", help="run all 25 sweep points, one short JSON line each")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-largest", action="store_true", help="skip the config-4 run that the default (config 3) line carries")
    ap.add_argument("--largest-steps", type=int, default=8, help="timed steps of that config-4 run")
    ap.add_argument("--leg", action="store_true", help=argparse.SUPPRESS)      # this process IS that config-4 run
    ap.add_argument("--min-timed-ms", type=float, default=1000.0,
                    help="the timed steps are replayed (state put back outside the events) until their device time adds up to this")
    ap.add_argument("--max-repeats", type=int, default=200)
    ap.add_argument("--score-source", default="controller", choices=["controller", "attention", "controller-relative"],
                    help="attention: tokens ranked by cumulative attention weight (the H2O baselines' score), no controller; "
                         "controller-relative: position feature = distance to the current token, every token re-scored every step")
    ap.add_argument("--labels", action="store_true", help="time the label-construction entry point instead of the decode step")
    ap.add_argument("--order", default="attend-first", choices=["attend-first", "rebuild-first"],
                    help="rebuild-first: select, rebuild, then one attention with R_max+1 query rows per sequence "
                         "(adore_step_begin / adore_attend_rows); no end-to-end pass in that order")
    ap.add_argument("--rebuild-max", type=int, default=None,
                    help="override the configuration's R_max (tokens rebuilt per sequence and step), e.g. the paper's 32")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return
    if args.labels:
        run_labels(args)
        return
    cfg = sweep_point(args.capacity, args.batch) if args.config == 5 else wl.get_config(args.config)
    if args.rebuild_max is not None:
        cfg = cfg.scaled(name=f"{cfg.name}_r{args.rebuild_max}", rebuild_max=args.rebuild_max)
    if args.steps is None:
        args.steps = default_steps(cfg) if args.impl == "ours" else 3
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    from paper_2407_02328_b200 import build
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    from paper_2407_02328_b200 import adore as lib

    K, W = args.steps, args.warmup
    with_e2e = not args.no_e2e and args.order == "attend-first"
    total = W + K                                       # warm-up and timed steps; every other pass replays the timed ones
    run = DeviceRun(cfg, total, rank, args.order, args.score_source)
    flush = None
    if kv_bytes(cfg) <= 2.5e8:
        flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(W):
        run.step()
    lib.adore_cache_sync_status(run.handle)

    # Every pass below replays the SAME K steps: the small state (slot maps, token table, scores) is snapshotted here and
    # put back before each pass, so that all of them see the same list lengths and occupancy. The K/V rows are copied
    # aside and put back too (on the device): on rows that do not belong to the restored maps the attention kernel
    # measured ~4 % slower.
    snap = np.zeros(lib.adore_cache_export_state(run.handle, None), np.uint8)
    lib.adore_cache_export_state(run.handle, snap)
    next0 = run.next
    kv_shape = (cfg.n_layers, cfg.batch, cfg.n_heads, cfg.capacity, cfg.head_dim)
    kv_live = [lib.device_view(p, kv_shape, run.dt) for p in lib.adore_cache_kv(run.handle, 0)]
    kv_keep = [t.clone() for t in kv_live]

    def rewind():
        lib.adore_cache_import_state(run.handle, snap)
        for live, keep in zip(kv_live, kv_keep):
            live.copy_(keep)
        torch.cuda.synchronize()
        run.next = next0

    def timed_pass():
        """The K steps once, device time in ms on this rank (events on the stream the library launches on)."""
        if flush is None:
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record()
            for _ in range(K):
                run.step()
            lib.adore_cache_join(run.handle)            # the last step's side-stream work counts too
            ev1.record()
            barrier()
            return ev0.elapsed_time(ev1)
        pairs = []                                      # small workloads: flush L2 between steps
        for _ in range(K):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            run.step()
            lib.adore_cache_join(run.handle)
            b.record()
            pairs.append((a, b))
        barrier()
        return sum(a.elapsed_time(b) for a, b in pairs)

    # ---- timed region: the K steps, replayed until the device time adds up to about a second; max over ranks per
    # repeat, median over the repeats ----
    launches0 = lib.adore_cache_launch_count(run.handle)
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        time.sleep(0.3)                                 # let the sampler come up
    barrier()
    t_timed0 = time.time()
    first = max_over_ranks(timed_pass(), world, dev)
    launches = lib.adore_cache_launch_count(run.handle) - launches0
    repeats = int(min(args.max_repeats, max(1, math.ceil(args.min_timed_ms / max(first, 1e-3)))))
    per_repeat = [first]
    for _ in range(repeats - 1):
        rewind()
        barrier()
        per_repeat.append(max_over_ranks(timed_pass(), world, dev))
    t_timed1 = time.time()
    lib.adore_cache_sync_status(run.handle)
    ms_total = float(np.median(per_repeat))
    value = whole_job_tokens_per_s(cfg.batch, K, world, ms_total)

    # ---- end to end through the host-buffer entry point (same repeats, median) ----
    e2e = None
    if with_e2e:
        rewind()
        run.make_host_inputs(run.next, K)
        e2e_runs = []
        for r in range(max(1, min(repeats, args.max_repeats // 2))):
            if r:
                rewind()
            barrier()
            t0 = time.perf_counter()
            for _ in range(K):
                run.step_host()
            torch.cuda.synchronize()
            e2e_runs.append(max_over_ranks((time.perf_counter() - t0) * 1e3, world, dev))
        e2e_ms = float(np.median(e2e_runs))
        h2d, d2h = run.host_bytes_per_step()
        e2e = {"value": whole_job_tokens_per_s(cfg.batch, K, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms / K,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "repeats": len(e2e_runs),
               "excludes": "per-slot weights (emitted on the device for device-side consumers, not copied to the host)"}

    # ---- per-stage pass (events around every launch, stages one after the other) for the roofline figures ----
    st_ms, st_n, rows_sum, stage_steps = [0.0] * 4, [0] * 4, 0, 0
    stage_repeats = max(1, min(repeats, args.max_repeats // 2))
    t_stage0 = time.time()
    for _ in range(stage_repeats):
        rewind()
        rows0 = lib.adore_cache_rebuild_rows(run.handle)
        lib.adore_cache_set_stage_timing(run.handle, 1)
        lib.adore_cache_stage_times(run.handle)
        for _ in range(K):
            if flush is not None:
                flush.zero_()
            run.step()
        ms_i, n_i = lib.adore_cache_stage_times(run.handle)
        lib.adore_cache_set_stage_timing(run.handle, 0)
        rows_sum += lib.adore_cache_rebuild_rows(run.handle) - rows0
        stage_steps += K
        st_ms = [a + b for a, b in zip(st_ms, ms_i)]
        st_n = [a + b for a, b in zip(st_n, n_i)]
    t_stage1 = time.time()
    rows = rows_sum / max(stage_steps, 1)                # rebuilt rows per step
    lib.adore_cache_sync_status(run.handle)

    # ---- group pass: the step's own schedule (selection and controller beside the attention, rebuilds beside the
    # following layers); device time from the start of the step's attention to the later of {last attention / new
    # token's row written, controller chain done} ----
    group_ms = group_main_ms = group_steps = 0
    if args.order == "attend-first":
        for _ in range(stage_repeats):
            rewind()
            lib.adore_cache_set_stage_timing(run.handle, 2)
            lib.adore_cache_group_times(run.handle)
            for _ in range(K):
                if flush is not None:
                    flush.zero_()
                run.step()
            g_ms, g_main, g_n = lib.adore_cache_group_times(run.handle)
            lib.adore_cache_set_stage_timing(run.handle, 0)
            group_ms += g_ms
            group_main_ms += g_main
            group_steps += g_n
        lib.adore_cache_sync_status(run.handle)
    clocks = clocks_stage = None
    if sampler:
        sampler.close()
        clocks = sampler.window(t_timed0, t_timed1, "timed region (all repeats)")
        clocks_stage = sampler.window(t_stage0, t_stage1, "per-stage pass")

    peaks, peak_kind = measured_peaks()
    occ = min(cfg.capacity, cfg.retained_max + rows / cfg.batch)
    att_ms = st_ms[0] / max(st_n[0], 1)
    sel_ms = st_ms[1] / max(stage_steps, 1)
    adm_ms = st_ms[3] / max(stage_steps, 1)
    reb_ms = st_ms[2] / max(st_n[2], 1)
    att_bytes = attention_bytes_per_launch(cfg, occ)
    reb_flops, reb_bytes = rebuild_flops_bytes_per_launch(cfg, rows)
    att_gbs = att_bytes / (att_ms * 1e-3) / 1e9 if att_ms > 0 else 0.0
    stages = {
        "admit_layer0": {"ms_per_step": adm_ms},
        "attention": {"bound": "hbm", "ms_per_launch": att_ms, "launches_per_step": cfg.n_layers,
                      "algorithmic_bytes": att_bytes, "achieved": att_gbs, "unit": "GB/s", "peak": peaks["hbm_gbs"],
                      "frac": att_gbs / peaks["hbm_gbs"], "frac_of_nominal_8TBs": att_gbs / NOMINAL_HBM_GBS},
        "controller_select": {"ms_per_step": sel_ms},
    }
    sel_bytes = 4 * (3 * cfg.ctrl_hidden * (cfg.hidden + cfg.ctrl_hidden)) + cfg.batch * cfg.hidden * cfg.elem_bytes
    group_bytes = att_bytes * cfg.n_layers + sel_bytes
    both_ms = att_ms * cfg.n_layers + sel_ms + adm_ms
    both_gbs = group_bytes / (both_ms * 1e-3) / 1e9 if both_ms > 0 else 0.0
    stages["attention_plus_selection"] = {
        "bound": "hbm", "algorithmic_bytes": group_bytes, "unit": "GB/s", "peak": peaks["hbm_gbs"],
        "stages_added": {"ms_per_step": both_ms, "achieved": both_gbs, "frac": both_gbs / peaks["hbm_gbs"],
                         "note": "per-stage pass: the stages run one after the other and their times are added"}}
    if group_steps:
        ov_ms = group_ms / group_steps
        ov_gbs = group_bytes / (ov_ms * 1e-3) / 1e9
        stages["attention_plus_selection"]["overlapped"] = {
            "ms_per_step": ov_ms, "achieved": ov_gbs, "frac": ov_gbs / peaks["hbm_gbs"],
            "frac_of_nominal_8TBs": ov_gbs / NOMINAL_HBM_GBS,
            "note": "the step's own schedule: device time from the start of the attention to the later of {last "
                    "attention / new token's row written, controller chain done}"
                    + ("; the rebuilds of the earlier layers run inside this window on their own stream" if cfg.n_layers > 1 else "")}
        cr_ms = group_main_ms / group_steps
        cr_gbs = group_bytes / (cr_ms * 1e-3) / 1e9
        stages["attention_plus_selection"]["overlapped_without_controller_tail"] = {
            "ms_per_step": cr_ms, "achieved": cr_gbs, "frac": cr_gbs / peaks["hbm_gbs"],
            "note": "same window closed where the step's main stream is done with the group (last attention / new token's "
                    "row written): the controller of token n is started when the attention of layer 0 is done, beside what "
                    "follows, because its score is first read by the NEXT step's selection"}
        stages["attention_plus_selection"].update(achieved=ov_gbs, frac=ov_gbs / peaks["hbm_gbs"], frac_is="overlapped")
    else:
        stages["attention_plus_selection"].update(achieved=both_gbs, frac=both_gbs / peaks["hbm_gbs"], frac_is="stages_added")
    # every algorithmic byte of a step (attention of all layers, controller + selection, rebuild of all layers) over the
    # free-running step time: what the whole step makes of the HBM (the rebuilds share the bandwidth with the attention)
    step_bytes = group_bytes + (reb_bytes * cfg.n_layers if rows > 0 else 0)
    step_ms = ms_total / K
    step_gbs = step_bytes / (step_ms * 1e-3) / 1e9
    stages["step_hbm"] = {"algorithmic_bytes": step_bytes, "ms_per_step": step_ms, "achieved": step_gbs, "unit": "GB/s",
                          "peak": peaks["hbm_gbs"], "frac": step_gbs / peaks["hbm_gbs"]}
    tensor_bound = cfg.dtype == "bf16" and rows >= 300
    if reb_ms > 0 and rows > 0:
        if tensor_bound:
            tf = reb_flops / (reb_ms * 1e-3) / 1e12
            # which cuBLAS figure the launch is put against follows the clocks seen while it was timed: at (nearly) full
            # clock the burst figure, under the power cap the sustained one
            ck = clocks_stage or {}
            full_clock = bool(ck.get("sm_mhz")) and ck["sm_mhz"] >= 0.95 * (ck.get("sm_max_mhz") or peaks.get("sm_max_mhz", 1965.0))
            which = "burst" if (full_clock or not ck.get("sm_mhz")) else "sustained"
            peak_tf = peaks["bf16_tflops"] if which == "burst" else peaks["bf16_tflops_sustained"]
            stages["rebuild"] = {"bound": "tensor", "ms_per_launch": reb_ms, "rows_per_launch": rows, "flops": reb_flops,
                                 "achieved": tf, "unit": "TFLOP/s", "peak": peak_tf, "frac": tf / peak_tf, "frac_is": which,
                                 "frac_of_burst": tf / peaks["bf16_tflops"], "frac_of_sustained": tf / peaks["bf16_tflops_sustained"],
                                 "sm_mhz_while_timed": ck.get("sm_mhz")}
        else:
            gb = reb_bytes / (reb_ms * 1e-3) / 1e9
            stages["rebuild"] = {"bound": "hbm", "ms_per_launch": reb_ms, "rows_per_launch": rows,
                                 "algorithmic_bytes": reb_bytes, "achieved": gb, "unit": "GB/s", "peak": peaks["hbm_gbs"],
                                 "frac": gb / peaks["hbm_gbs"]}
    dominant = "rebuild" if ("rebuild" in stages and st_ms[2] > st_ms[0]) else "attention"
    d = stages[dominant]
    kernel_name = {"attention": "attention kernel", "rebuild": "rebuild projection"}[dominant]
    traffic, traffic_from = ncu_traffic(kernel_name, cfg, rows)
    roofline = {"kernel": kernel_name, "bound": d["bound"], "achieved": d["achieved"], "peak": d["peak"], "unit": d["unit"],
                "frac": d["frac"],
                "peak_source": f"{peak_kind} ({d.get('frac_is', 'copy') if d['bound'] == 'tensor' else 'copy'})",
                "traffic": traffic, "traffic_source": traffic_from,
                "share_of_step": {"attention": (st_ms[0] + st_ms[3]) / max(sum(st_ms), 1e-9),
                                  "controller_select": st_ms[1] / max(sum(st_ms), 1e-9),
                                  "rebuild": st_ms[2] / max(sum(st_ms), 1e-9)}}

    prompt_load = None
    if cfg.prompt:
        n_prompt = cfg.batch * cfg.prompt
        prompt_load = {"tokens": n_prompt, "layers": cfg.n_layers, "ms": run.prompt_ms,
                       "tokens_per_s": n_prompt / (run.prompt_ms * 1e-3) if run.prompt_ms > 0 else None,
                       "what": "adore_cache_append_tokens (controller scan, bulk selection, projection of the residents) "
                               "+ adore_cache_fill_layer for every further layer; device time, once, before the decode steps"}
    run.close()
    del run, kv_live, kv_keep
    torch.cuda.empty_cache()

    # ---- the HBM target is stated for the largest configuration: its own short run, in a process of its own ----
    largest = None
    if rank == 0 and world == 1 and cfg_index(cfg) == 3 and not args.no_largest and not args.leg:
        largest = run_largest_leg(args)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, threads, desc, _ = time_oracle(cfg, 3, 1)
        cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
                "ms_per_step": ms_total / K, "steps_per_s": K / (ms_total * 1e-3), "repeats": len(per_repeat),
                "ms_per_step_min_max": [min(per_repeat) / K, max(per_repeat) / K],
                "timed_ms_total": float(sum(per_repeat)), "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
                "config": dict(workload_desc(cfg), step_order=args.order, score_source=args.score_source), "clocks": clocks,
                "clocks_stage_pass": clocks_stage, "e2e": e2e, "gpu_launches": int(launches),
                "roofline": roofline, "stages": stages, "prompt_load": prompt_load, "cpu_baseline": cpu,
                "largest_config": largest}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_largest_leg(args):
    """Config 4 (32 layers, B 32, C 1024: the configuration the HBM target is stated for) in a process of its own, a few
    timed steps; returns the part of its line that the metric names."""
    cmd = [sys.executable, os.path.abspath(__file__), "--config", "4", "--leg", "--no-cpu-baseline",
           "--steps", str(args.largest_steps), "--warmup", "3", "--min-timed-ms", "400", "--max-repeats", "12"]
    try:
        res = subprocess.run(cmd, capture_output=True, text=True, timeout=900)
    except subprocess.TimeoutExpired:
        return {"error": "the config-4 run did not finish in 900 s"}
    if res.returncode != 0:
        return {"error": (res.stderr.strip().splitlines() or ["failed"])[-1][:300]}
    d = json.loads(res.stdout.strip().splitlines()[-1])
    st = d["stages"]
    return {"workload": d["config"]["workload"], "steps": d["steps"], "repeats": d["repeats"], "ms_per_step": d["ms_per_step"],
            "tokens_per_s": d["value"], "steps_per_s": d["steps_per_s"], "gpu_launches": d["gpu_launches"], "clocks": d["clocks"],
            "attention": st["attention"], "attention_plus_selection": st["attention_plus_selection"],
            "controller_select": st["controller_select"], "rebuild": st.get("rebuild"), "step_hbm": st.get("step_hbm"),
            "prompt_load": d.get("prompt_load"), "e2e": d.get("e2e")}


if __name__ == "__main__":
    main()
