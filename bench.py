#!/usr/bin/env python
"""Benchmark of the KV-cache hot path on one (or N independent) B200.

Workload (N=1): the single long ReAct session of configuration C2 — 8B-class KV geometry
(32 layers x 8 KV heads x 128, bf16: 2 MiB per 16-token block), 40 GiB HBM pool (20,480 blocks),
host tier of up to 120 GiB — under tier pressure: between two LLM calls of the session, half of its
idle KV is pushed out of HBM (the engine's own victim order), so every call hashes and looks up the
whole context, reloads the evicted half of its prefix from the second tier, admits the new blocks
and, after prefill, is evicted again. One step = one such call = every stage of the path:
apply ops -> hash -> lookup -> classify -> select victims -> offload -> reload -> admit.

Two measurements of the same steps:
  value : second tier resident in HBM and tokens resident on the device (inputs in HBM when the timed
          region starts); the mover runs HBM<->HBM and is measured against the HBM roofline.
  e2e   : the real thing through the same C-ABI calls: tokens come from pinned host buffers, the
          second tier is pinned host memory, every offload / reload crosses the host link inside the
          timed region.
Side measurements in the same line: `e2e_inclusive_tiers` (the e2e steps with clean host copies kept),
`e2e_two_sessions` (two such sessions taking turns on an HBM pool that holds one and a half of them: no artificial
pressure, offload + reload per call against one kvt_exchange per call), `metadata_stress` (C4 shape).
`--impl reference` times the CPU oracle (plain single-threaded C++) on the same steps.
Prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_39819_b200 import workloads as W  # noqa: E402

METRIC = "KV block GB/s (HBM & host link) vs roofline; blocks hashed+looked up/sec"
GiB = 1 << 30


def mover_traffic_ratio():
    """DRAM traffic of the mover kernel per algorithmic byte (read + write), taken from the tracked summary of its
    ncu capture: (dram__bytes_read.sum + dram__bytes_write.sum) / (2 x payload bytes) of a 1024-block launch, the
    row "traffic / algorithmic" of the summary's counter table. Traffic grows in proportion to the blocks moved, so
    the ratio is scaled to the bench's launches. None if the summary is missing."""
    import re
    try:
        text = open(os.path.join(ROOT, "profiles", "mover_8b_hbm_to_hbm.md")).read()
    except OSError:
        return None
    m = re.search(r"^\|\s*traffic / algorithmic\s*\|\s*([0-9.]+)\s*\|", text, flags=re.M)
    return float(m.group(1)) if m else None


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--seed", type=int, default=1)
    ap.add_argument("--hbm-gib", type=float, default=40.0)
    ap.add_argument("--host-gib", type=float, default=120.0)
    ap.add_argument("--cpu-steps", type=int, default=6, help="steps of the bounded CPU-oracle sample")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--skip-cpu", action="store_true")
    ap.add_argument("--skip-stress", action="store_true", help="skip the C4-shaped metadata measurement")
    ap.add_argument("--skip-inclusive", action="store_true", help="skip the extra end-to-end run with inclusive tiers")
    ap.add_argument("--skip-two-tenants", action="store_true", help="skip the extra end-to-end run with two sessions")
    ap.add_argument("--skip-c3", action="store_true", help="skip the C3 arm (32 sessions, GLM-scale blocks, 120 GiB pool)")
    ap.add_argument("--c3-host-gib", type=float, default=48.0, help="pinned host tier of the C3 arm")
    return ap.parse_args()


# ---- workload ---------------------------------------------------------------------------------------------
def split_turns(trace):
    """Splits a C2 trace into (spawn events, [(events before the call, contexts of the call, events after
    it)]). In C2 the only event that follows a call is the removal of that call's scratch message."""
    setup = [ev for ev in trace if ev[0] == "spawn"]
    turns, pre, i = [], [], len(setup)
    while i < len(trace):
        ev = trace[i]
        i += 1
        if ev[0] != "call":
            pre.append(ev)
            continue
        post = []
        if i < len(trace) and trace[i][0] == "remove":
            post.append(trace[i])
            i += 1
        turns.append((pre, ev[1], post))
        pre = []
    return setup, turns


def make_turns(seed, n_needed):
    target, max_turns = 131072, 100
    while True:
        trace = W.trace_c2(seed, target_tokens=target, max_turns=max_turns)
        setup, turns = split_turns(trace)
        if len(turns) >= n_needed + 1:
            return setup, turns, target
        target *= 2
        max_turns = max(max_turns, 2 * n_needed)


def apply_event(eng, ev, tok):
    k = ev[0]
    if k == "spawn": eng.spawn(ev[1])
    elif k == "append": eng.append(ev[1], tok(ev[2]))
    elif k == "replace": eng.replace(ev[1], ev[2], ev[3], tok(ev[4]))
    elif k == "remove": eng.remove(ev[1], ev[2], ev[3])
    elif k == "one_off": eng.one_off(ev[1], ev[2], ev[3])
    elif k == "terminate": eng.terminate(ev[1])
    else: raise ValueError(k)


CPU_PRESSURE_CAP = 512   # blocks evicted per step in the CPU-oracle runs (bounded sample: 1 GiB each way)


def pressure_evict(eng, cap=None):
    """Other tenants push half of the session's resident blocks out of HBM. With `cap`, at most that
    many live blocks are moved (dead ones are dropped either way)."""
    n = eng.get_stats()["occ_hbm"] // 2
    if cap is not None and n:
        _v, s = eng.select_victims(W.TIER_HBM, n)
        n = min(n, int((s == 0).sum()) + cap)
    if n:
        W.evict(eng, n)


def run_step(eng, turn, tok, opt, pressure=True, timers=None, cap=None):
    """One LLM call of the session through the whole path, then the tier pressure between calls."""
    pre, ctxs, post = turn
    t0 = time.perf_counter()
    for ev in pre:
        apply_event(eng, ev, tok)
    t1 = time.perf_counter()
    W.run_call(eng, ctxs, opt)
    t2 = time.perf_counter()
    for ev in post:
        apply_event(eng, ev, tok)
    if pressure:
        pressure_evict(eng, cap)
    t3 = time.perf_counter()
    if timers is not None:
        timers["ops_ms"] += (t1 - t0) * 1e3
        timers["call_ms"] += (t2 - t1) * 1e3
        timers["pressure_ms"] += (t3 - t2) * 1e3


class StageTimer:
    """Wall-clock per API entry point (each of them synchronises its stream before returning, except
    apply_op and classify, whose device time then shows up in the next synchronising call)."""

    NAMES = ("map_blocks", "select_victims", "offload", "reload", "get_block_map", "release", "append", "replace",
             "remove", "one_off", "prefill_done", "get_stats")

    def __init__(self, eng):
        self.ms = {}
        self.calls = {}
        for name in self.NAMES:
            fn = getattr(eng, name)
            setattr(eng, name, self._wrap(name, fn))

    def _wrap(self, name, fn):
        def inner(*a, **k):
            t = time.perf_counter()
            r = fn(*a, **k)
            key = name
            if name == "map_blocks":
                key = "map_lookup(hash+lookup)" if a[1] == 0 else "map_admit"
            self.ms[key] = self.ms.get(key, 0.0) + (time.perf_counter() - t) * 1e3
            self.calls[key] = self.calls.get(key, 0) + 1
            return r
        return inner

    def reset(self):
        self.ms, self.calls = {}, {}


# ---- helpers ------------------------------------------------------------------------------------------------
def mem_available_bytes():
    try:
        for ln in open("/proc/meminfo"):
            if ln.startswith("MemAvailable"):
                avail = int(ln.split()[1]) * 1024
                break
        else:
            return 0
        try:
            lim = open("/sys/fs/cgroup/memory.max").read().strip()
            if lim != "max":
                cur = int(open("/sys/fs/cgroup/memory.current").read())
                avail = min(avail, int(lim) - cur)
        except OSError:
            pass
        return avail
    except OSError:
        return 0


class ClockSampler:
    """SM clock and throttle reasons sampled in the background while an arm runs: NVML read-outs every 5 ms from a
    thread (the timed region of the in-device arm lasts tens of ms), or, if NVML cannot be loaded, nvidia-smi
    polled every 50 ms. stop(t0, t1) keeps the samples taken inside the timed window [t0, t1] (host wall clock),
    or all samples of the arm if the window saw fewer than two. Read-only: no setting of the GPU is touched."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NVML_REASONS = ((0x8, "hw_slowdown"), (0x40, "hw_thermal_slowdown"), (0x20, "sw_thermal_slowdown"), (0x4, "sw_power_cap"))

    def __init__(self, gpu_index, torch=None):
        self.rows, self.p, self.thread, self.source = [], None, None, "none"
        try:
            import threading
            import pynvml
            pynvml.nvmlInit()
            h = None
            if torch is not None:
                try:
                    uuid = str(torch.cuda.get_device_properties(torch.cuda.current_device()).uuid)
                    h = pynvml.nvmlDeviceGetHandleByUUID(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
                except Exception:
                    h = None
            if h is None:
                h = pynvml.nvmlDeviceGetHandleByIndex(gpu_index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            self.running = True

            def loop():
                while self.running:
                    try:
                        mhz = float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM))
                        bits = int(pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h))
                        self.rows.append((time.time(), mhz, self.max_mhz, [nm for b, nm in self.NVML_REASONS if bits & b]))
                    except Exception:
                        pass
                    time.sleep(0.005)
            self.thread = threading.Thread(target=loop, daemon=True)
            self.thread.start()
            self.source = "nvml, 5 ms"
            return
        except Exception:
            self.thread = None
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                       "-i", str(gpu_index), "-lms", "50"], stdout=self.f, stderr=subprocess.DEVNULL)
            self.source = "nvidia-smi, 50 ms"
        except OSError:
            self.p = None

    def _smi_rows(self):
        import datetime
        time.sleep(0.06)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        rows = []
        for ln in self.f:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(parts[1]), float(parts[2]),
                             [nm for nm, v in zip(names, parts[5:9]) if v.lower().startswith("active")]))
            except ValueError:
                continue
        self.f.close()
        os.unlink(self.f.name)
        return rows

    def stop(self, t0=None, t1=None):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "window": "none", "source": self.source}
        if self.thread is not None:
            self.running = False
            self.thread.join(timeout=1)
            rows, slack = list(self.rows), 0.0
        elif self.p is not None:
            rows, slack = self._smi_rows(), 0.05
        else:
            return out
        inside = [r for r in rows if t0 is not None and t0 - slack <= r[0] <= t1 + slack]
        use, out["window"] = (inside, "timed region") if len(inside) >= 2 else (rows, "whole arm (timed region shorter than the sampling period)")
        if use:
            out.update(sm_mhz=float(np.median([r[1] for r in use])), sm_max_mhz=float(max(r[2] for r in use)),
                       reasons=sorted({x for r in use for x in r[3]}), samples=len(use))
        return out


def host_info():
    model = "unknown"
    try:
        for ln in open("/proc/cpuinfo"):
            if ln.lower().startswith("model name"):
                model = ln.split(":", 1)[1].strip()
                break
    except OSError:
        pass
    mem = 0
    try:
        for ln in open("/proc/meminfo"):
            if ln.startswith("MemTotal"):
                mem = int(ln.split()[1]) // (1 << 20)
    except OSError:
        pass
    return {"model": model, "cores": os.cpu_count(), "mem_total_gib": mem}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return json.load(open(p)).get("hbm_gbs", 6650.0), "measured"
    return 6650.0, "fallback"


def hbm_copy_this_run(torch):
    """Plain torch copy of 2 GiB (read + write bytes, best of 10): the same measurement as the pool's recorded
    copy peak, taken in this run for comparison."""
    a = torch.empty(2 * GiB, dtype=torch.uint8, device="cuda")
    b = torch.empty(2 * GiB, dtype=torch.uint8, device="cuda")
    best = 1e9
    for i in range(12):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); b.copy_(a); e1.record(); torch.cuda.synchronize()
        if i >= 2:
            best = min(best, e0.elapsed_time(e1))
    del a, b
    torch.cuda.empty_cache()
    return 2 * 2 * GiB / best / 1e6


def host_link_peaks(torch):
    """1 GiB pinned cudaMemcpyAsync in each direction, best of 10 (the host-link roofline)."""
    h = torch.empty(GiB, dtype=torch.uint8, pin_memory=True)
    d = torch.empty(GiB, dtype=torch.uint8, device="cuda")
    out = {}
    for name, fn in (("h2d", lambda: d.copy_(h, non_blocking=True)), ("d2h", lambda: h.copy_(d, non_blocking=True))):
        best = 1e9
        for i in range(12):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record(); torch.cuda.synchronize()
            if i >= 2:
                best = min(best, a.elapsed_time(b))
        out[name] = GiB / best / 1e6
    del h, d
    return out


# ---- GPU arms -------------------------------------------------------------------------------------------------
def gpu_arm(args, torch, B, setup, turns, n_ff, e2e, n_host_blocks, n_hbm_blocks, rank=0, world=1, barrier=None,
            policy_flags=0):
    """Fast-forwards n_ff turns untimed, runs W warm-up steps, then times exactly K steps."""
    W_, K = args.warmup, args.steps
    geo = W.GEO_8B
    max_tok = 1 << 21
    eng = B.Engine(n_hbm_blocks=n_hbm_blocks, n_host_blocks=n_host_blocks, max_contexts=4, max_tokens=max_tok,
                   max_messages=1 << 13, max_batch_blocks=max_tok // 16, host_pool_on_device=not e2e, zero_pools=False,
                   policy_flags=policy_flags, **geo.kwargs())
    eng.set_profiling(True)
    # token sources: device tensors (value arm) or pinned host tensors (e2e arm)
    cache = {}

    def tok(arr):
        k = id(arr)
        if k not in cache:
            t = torch.from_numpy(arr.view(np.int32))
            cache[k] = t.cuda() if not e2e else t.pin_memory()
        return cache[k]

    used = turns[: n_ff + W_ + K]
    for pre, _c, _post in used:
        for ev in pre:
            if ev[0] in ("append", "replace"):
                tok(ev[2] if ev[0] == "append" else ev[4])
    torch.cuda.synchronize()
    opt = W.ReplayOptions(payload=None, record_states=False)
    for ev in setup:
        apply_event(eng, ev, tok)
    # fast-forward; the blocks admitted here get a key-derived payload so movement can be verified later
    base = (torch.arange(eng.block_bytes // 4, dtype=torch.int64, device="cuda") * 0x9E3779B1) & 0xFFFFFFFF
    pool = eng.hbm_pool.view(eng.n_chunks, eng.n_hbm_blocks, eng.chunk_bytes)
    written = {}
    for t in range(n_ff):
        pre, ctxs, post = used[t]
        for ev in pre:
            apply_event(eng, ev, tok)
        info = eng.map_blocks(ctxs, 0)
        adm = eng.map_blocks(ctxs, 1)
        keys, tier, slot = eng.get_block_map(ctxs[0])
        for b in range(int(info[0]["hit_len"]), int(adm[0]["n_held"])):
            if tier[b] == 0 and len(written) < 512 and b % 7 == 0:
                key = int(keys[b])
                w = ((base + (key & 0xFFFFFFFF)) & 0xFFFFFFFF) ^ (key >> 32)
                pool[:, int(slot[b]), :] = w.to(torch.int32).view(torch.uint8).view(eng.n_chunks, eng.chunk_bytes)
                written[key] = True
        for c in ctxs:
            eng.prefill_done(c)
        for ev in post:
            apply_event(eng, ev, tok)
    pressure_evict(eng)
    for t in range(n_ff, n_ff + W_):
        run_step(eng, used[t], tok, opt)
    timer = StageTimer(eng)
    timers = {"ops_ms": 0.0, "call_ms": 0.0, "pressure_ms": 0.0}
    torch.cuda.synchronize()
    if barrier:
        barrier()
    s0 = eng.get_stats()
    timer.reset()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    wall0 = time.time()
    ev0.record()
    torch.cuda.nvtx.range_push("kvt_timed")      # lets a profiler restrict its launch list to the timed steps
    for t in range(n_ff + W_, n_ff + W_ + K):
        run_step(eng, used[t], tok, opt, timers=timers)
    torch.cuda.nvtx.range_pop()
    ev1.record()
    torch.cuda.synchronize()
    wall1 = time.time()
    if barrier:
        barrier()
    ms = ev0.elapsed_time(ev1)
    s1 = eng.get_stats()
    d = {k: s1[k] - s0[k] for k in s1}
    # verification: every block written during the fast-forward still holds its key-derived payload,
    # wherever the offload / reload cycles have left it
    n_ok = n_seen = 0
    for tier in (0, 1):
        keys = eng.get_entries(tier)["key"]
        for s in np.nonzero(keys)[0]:
            key = int(keys[s])
            if key in written and n_seen < 64:
                n_seen += 1
                w = ((base + (key & 0xFFFFFFFF)) & 0xFFFFFFFF) ^ (key >> 32)
                want = w.to(torch.int32).view(torch.uint8).cpu().numpy()
                n_ok += int(np.array_equal(eng.read_block(tier, int(s)), want))
    tok_bytes = sum(4 * len(ev[2] if ev[0] == "append" else ev[4]) for pre, _c, _p in used[n_ff + W_:] for ev in pre
                    if ev[0] in ("append", "replace"))
    res = dict(ms=ms, stats=d, stage_ms=dict(timer.ms), stage_calls=dict(timer.calls), timers=timers,
               verified=(n_ok, n_seen), tok_bytes=tok_bytes, block_bytes=eng.block_bytes, wall=(wall0, wall1))
    eng.close()
    del eng, pool, cache, base, timer
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    return res


def shift_ctx(turns, setup, by):
    """The same session under other context ids (so that two sessions can share an engine)."""
    def ev_(ev):
        return (ev[0], ev[1] + by) + tuple(ev[2:])
    return [ev_(ev) for ev in setup], [([ev_(ev) for ev in pre], [c + by for c in ctxs], [ev_(ev) for ev in post])
                                       for pre, ctxs, post in turns]


def two_tenant_arm(args, torch, B, n_ff, use_exchange, n_hbm_blocks=12288, n_host_blocks=12288):
    """End-to-end side measurement without artificial pressure: two C2 sessions (seeds s, s + 1) take turns on an
    HBM pool that holds one and a half of them (24 GiB) over a pinned host tier. Every call finds part of its prefix
    on the host tier and has to push part of the other session out: with `use_exchange` the replay driver issues
    the reload and the offload as one kvt_exchange (both directions of the link at once), otherwise as kvt_offload
    followed by kvt_reload. Returns payload GB/s over the timed calls."""
    W_, K = args.warmup, args.steps
    sa, ta, _ = make_turns(args.seed, W_ + K + 4)
    sb, tb, _ = make_turns(args.seed + 1, W_ + K + 4)
    sb, tb = shift_ctx(tb, sb, 1)
    n = min(len(ta), len(tb))
    ff = n - (W_ + K)
    max_tok = 1 << 22
    eng = B.Engine(n_hbm_blocks=n_hbm_blocks, n_host_blocks=n_host_blocks, max_contexts=4, max_tokens=max_tok,
                   max_messages=1 << 14, max_batch_blocks=max_tok // 16, zero_pools=False, **W.GEO_8B.kwargs())
    cache = {}

    def tok(arr):
        k = id(arr)
        if k not in cache:
            cache[k] = torch.from_numpy(arr.view(np.int32)).pin_memory()
        return cache[k]

    opt = W.ReplayOptions(payload=None, record_states=False, use_exchange=use_exchange)
    for ev in sa + sb:
        apply_event(eng, ev, tok)

    def call(turn):
        pre, ctxs, post = turn
        for ev in pre:
            apply_event(eng, ev, tok)
        W.run_call(eng, ctxs, opt)
        for ev in post:
            apply_event(eng, ev, tok)

    for t in range(ff + W_):
        call(ta[t]); call(tb[t])
    torch.cuda.synchronize()
    s0 = eng.get_stats()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for t in range(ff + W_, ff + W_ + K):
        call(ta[t]); call(tb[t])
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1)
    s1 = eng.get_stats()
    d = {k: s1[k] - s0[k] for k in s1}
    out = {"value": kv_bytes(d, eng.block_bytes) / (ms / 1e3) / 1e9, "ms_per_call": ms / (2 * K),
           "offloaded_per_call": d["offloaded"] / (2 * K), "reloaded_per_call": d["reloaded"] / (2 * K),
           "dropped_per_call": d["dropped"] / (2 * K)}
    eng.close()
    del eng, cache
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    return out


def c3_arm(args, torch, B, link):
    """C3 at full size, as a timed run: 32 concurrent agent sessions with subagents (32 K - 258 K tokens each,
    ~216 K blocks of demand), GLM-scale KV (92 x 8 x 128 bf16, 5.75 MiB per block), HBM pool 120 GiB = 21,370
    blocks, pinned host tier. No pressure is added: the sessions do not fit, so every round evicts in the engine's
    victim order, offloads what is live, drops what is dead and reloads prefixes on the sessions' next calls. Tokens
    come from pageable host arrays through the C ABI; payload bytes are whatever the pools hold (the movement is
    real, the content is not produced). The whole trace is timed with the wall clock (every call synchronises)."""
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    if hasattr(torch._C, "_host_emptyCache"):
        torch._C._host_emptyCache()
    geo = W.GEO_GLM
    free_b, _ = torch.cuda.mem_get_info()
    n_hbm = min(21370, int((free_b - 8 * GiB) // geo.block_bytes))
    n_host = min(int(args.c3_host_gib * GiB), int(mem_available_bytes() * 0.4)) // geo.block_bytes
    if n_hbm < 4000 or n_host < 1000:
        return {"skipped": f"needs memory: {n_hbm} HBM blocks, {n_host} host blocks possible"}
    trace, n_ctx = W.trace_c3(args.seed)
    eng = B.Engine(n_hbm_blocks=n_hbm, n_host_blocks=n_host, max_contexts=n_ctx, max_tokens=1 << 24, max_messages=1 << 16,
                   zero_pools=False, **geo.kwargs())
    eng.set_profiling(True)
    opt = W.ReplayOptions(payload=None, record_states=False)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    n_calls = 0
    for _i, kind, _rec in W.replay(eng, trace, opt):
        n_calls += kind == "call"
    torch.cuda.synchronize()
    sec = time.perf_counter() - t0
    st = eng.get_stats()
    moved = (st["offloaded"] - st["offloaded_clean"] + st["reloaded"]) * eng.block_bytes
    mover_s = st["mover_ns"] / 1e9
    out = {
        "workload": f"C3: 32 sessions + subagents, seed {args.seed}, {n_calls} batched calls, GLM-scale blocks of "
                    f"{eng.block_bytes} B, HBM pool {n_hbm} blocks ({n_hbm * eng.block_bytes / GiB:.0f} GiB), pinned host "
                    f"tier {n_host} blocks ({n_host * eng.block_bytes / GiB:.0f} GiB); natural pressure only",
        "value": moved / sec / 1e9, "unit": "GB/s (payload offloaded + reloaded over the host link / wall time of the whole trace)",
        "seconds": sec, "blocks_hashed": st["blocks_hashed"], "blocks_hashed_looked_up_per_s": st["blocks_hashed"] / sec,
        "inserted": st["inserted"], "offloaded": st["offloaded"], "reloaded": st["reloaded"], "dropped": st["dropped"],
        "hit_ratio": (st["hits_hbm"] + st["hits_host"]) / max(st["blocks_hashed"], 1),
        "host_link": {"achieved": st["mover_bytes"] / mover_s / 1e9 if mover_s else 0.0, "unit": "GB/s while a move is running",
                      "frac": (st["mover_bytes"] / mover_s / 1e9) / (0.5 * (link["h2d"] + link["d2h"])) if mover_s else 0.0},
        "lookup_kernels_blocks_per_s": st["lookup_blocks"] / (st["lookup_ns"] / 1e9) if st["lookup_ns"] else None,
        "gpu_launches": st["kernel_launches"],
    }
    eng.close()
    del eng
    gc.collect()
    torch.cuda.empty_cache()
    if hasattr(torch._C, "_host_emptyCache"):
        torch._C._host_emptyCache()
    return out


def cpu_stage_arm():
    """The oracle, as it stands, on the C4 inputs stage by stage and on a C5-sized block gather, on this machine's
    host cores: one thread (the oracle's own engine calls), plus an all-cores figure for the two embarrassingly
    parallel stages (block digests, block copies) with plain std::thread."""
    from oracle import kvt_oracle as O
    O.build()
    n_res, cb, n_calls = 1 << 20, 16128, 64
    inp = W.inputs_c4(1, n_resident=n_res, chain_blocks=cb, n_calls=n_calls)
    eng = O.OracleEngine(n_hbm_blocks=n_res, n_host_blocks=0, max_contexts=n_calls + 1, metadata_only=True, **W.GEO_TOY.kwargs())
    keys = np.concatenate([O.hash_tokens(c) for c in inp.chain_tokens])
    eng.debug_load_resident(keys, inp.state, inp.stamp, inp.depth, inp.slot, 0)
    for i, t in enumerate(inp.calls):
        eng.spawn(i)
        eng.append(i, t)

    def timed(fn):
        t0 = time.perf_counter()
        r = fn()
        return time.perf_counter() - t0, r
    t_look, info = timed(lambda: eng.map_blocks(list(range(n_calls)), 0))
    t_cls, _ = timed(lambda: eng.get_states(0))
    t_sel, (v, _s) = timed(lambda: eng.select_victims(0, n_res // 10))
    n_blocks = int(info["n_blocks"].sum())
    cores = os.cpu_count() or 1
    tok = np.concatenate(inp.calls)
    t_hash1, _ = timed(lambda: O.hash_tokens(tok))
    t_dig1, _ = timed(lambda: O.par_digests(tok, 0, 1))
    t_digN, _ = timed(lambda: O.par_digests(tok, 0, cores))
    # C5-shaped gather: 256 permuted 2 MiB blocks (0.5 GiB, far beyond the caches) out of a 320-block pool into a contiguous tier
    bb, n_pool, n = W.GEO_8B.block_bytes, 320, 256
    rng = np.random.default_rng(5)
    src = np.ones(n_pool * bb, dtype=np.uint8)
    dst = np.ones(n * bb, dtype=np.uint8)
    ids = rng.permutation(n_pool)[:n]
    O.par_copy_blocks(dst, src, bb, ids[:64], np.arange(64), 1)          # touch the code path once
    t_cp1, _ = timed(lambda: O.par_copy_blocks(dst, src, bb, ids, np.arange(n), 1))
    t_cpN, _ = timed(lambda: O.par_copy_blocks(dst, src, bb, ids, np.arange(n), cores))
    return {
        "metadata_c4": {
            "workload": f"the C4 inputs of metadata_stress: {n_res} resident blocks, {n_calls} calls x {cb} blocks, select 10%",
            "cores": 1,
            "hash_lookup_blocks_per_s": n_blocks / t_look, "hash_lookup_s": t_look,
            "classify_s": t_cls, "classify_mappings_per_s": n_blocks / t_cls,
            "select_s": t_sel, "select_resident_blocks_per_s": n_res / t_sel, "victims": int(len(v)),
            "hash_only_blocks_per_s": len(tok) // 16 / t_hash1,
            "digests_blocks_per_s_1_thread": len(tok) // 16 / t_dig1,
            "digests_blocks_per_s_all_cores": len(tok) // 16 / t_digN, "all_cores": cores,
        },
        "mover_c5": {
            "workload": f"{n} permuted blocks of {bb} B gathered from a {n_pool}-block pool into a contiguous tier (memcpy)",
            "GBs_1_thread": n * bb / t_cp1 / 1e9, "GBs_all_cores": n * bb / t_cpN / 1e9, "all_cores": cores,
        },
    }


def metadata_stress(torch, B, hbm_peak, reps=5):
    """C4-shaped side measurement of the metadata stages at scale (the C2 calls above are launch-latency
    sized): 1 Mi resident blocks, one LOOKUP batch of 64 calls x 16,128 blocks, classification of the
    resulting 1.03 M mappings, selection of 10% of the pool. Kernel times come from the library's own
    CUDA events, call times from events around the C-ABI call. Algorithmic bytes per unit: hash 72 B per
    block (64 B tokens + 8 B key), fused lookup 64 B per block (two 32-byte table sectors), classify 16 B
    per mapping (8 B key + one 8-byte count update), select 8 B per resident block + 4 B per victim."""
    n_res, n_calls, cb = 1 << 20, 64, 16128
    inp = W.inputs_c4(1, n_resident=n_res, chain_blocks=cb, n_calls=n_calls)
    eng = B.Engine(n_hbm_blocks=n_res, n_host_blocks=0, max_contexts=n_calls + 1, metadata_only=True,
                   max_tokens=(n_calls + 2) * cb * 16 * 2, max_messages=1024, max_batch_blocks=n_calls * cb,
                   **W.GEO_TOY.kwargs())
    keys = np.concatenate([B.hash_tokens(torch.from_numpy(c.view(np.int32)).cuda()).cpu().numpy().view(np.uint64)
                           for c in inp.chain_tokens])
    eng.debug_load_resident(keys, inp.state, inp.stamp, inp.depth, inp.slot, 0)
    ids = list(range(n_calls))
    call_tok = [torch.from_numpy(t.view(np.int32)).cuda() for t in inp.calls]
    eng.set_profiling(True)

    def timed(fn):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); r = fn(); b.record(); torch.cuda.synchronize()
        return a.elapsed_time(b), r

    look_ms, cls_ms, sel_ms, cls_edit_ms, cls_full_ms, cls_done_ms, cls_k, cls_edit_k, cls_edit_warm_ms, cls_edit_warm_k = [], [], [], [], [], [], [], [], [], []
    s0 = None
    flush = torch.empty(1 << 29, dtype=torch.uint8, device="cuda")   # 512 MiB > L2: every timed call starts cold
    vbuf = eng.victim_buffers(n_res // 10)   # pinned output arrays: the victim list is written there by the last kernel
    for rep in range(reps + 1):
        if rep == 1:
            s0 = eng.get_stats()          # the first repetition is the warm-up
        for i in ids:                     # fresh contexts every repetition: every block is digested, none is resumed
            eng.spawn(i)
            eng.append(i, call_tok[i])
        flush.fill_(rep)
        ms, info = timed(lambda: eng.map_blocks(ids, 0))
        look_ms.append(ms)
        flush.fill_(rep + 1)
        c0 = eng.get_stats()
        cls_ms.append(timed(lambda: eng.classify())[0])      # event-driven: the 64 contexts of the batch are new mappings
        cls_k.append((eng.get_stats()["classify_ns"] - c0["classify_ns"]) / 1e6)
        eng.set_classify_mode(1)                             # the full recomputation over all contexts, for comparison
        flush.fill_(rep + 1)
        cls_full_ms.append(timed(lambda: eng.classify())[0])
        eng.set_classify_mode(0)
        for c in ids:
            eng.prefill_done(c)
        flush.fill_(rep + 1)
        cls_done_ms.append(timed(lambda: eng.classify())[0])  # every context's messages went from Active to Suspended
        eng.pin(0, 0, 1)                                     # one context's message changes state: 16,128 of its blocks
        flush.fill_(rep + 1)
        c0 = eng.get_stats()
        cls_edit_ms.append(timed(lambda: eng.classify())[0])
        cls_edit_k.append((eng.get_stats()["classify_ns"] - c0["classify_ns"]) / 1e6)
        eng.unpin(0, 0, 1)                                   # and back, this time with whatever the caches hold
        c0 = eng.get_stats()
        cls_edit_warm_ms.append(timed(lambda: eng.classify())[0])
        cls_edit_warm_k.append((eng.get_stats()["classify_ns"] - c0["classify_ns"]) / 1e6)
        flush.fill_(rep + 2)
        torch.cuda.synchronize()
        ms, (v, _st) = timed(lambda: eng.select_victims(0, n_res // 10, out=vbuf))
        sel_ms.append(ms)
        for i in ids:
            eng.terminate(i)
        eng.classify()                    # takes the ended contexts' mappings away (not timed)
    s1 = eng.get_stats()
    d = {k: s1[k] - s0[k] for k in s1}
    n_blocks = int(info["n_blocks"].sum())
    hit = float(info["hit_len"].sum()) / n_blocks
    look_k = d["lookup_ns"] / 1e6 / reps
    sel_k = d["select_ns"] / 1e6 / reps
    med = lambda x: float(np.median(x[1:]))
    out = {
        "workload": f"C4: {n_res} resident blocks (dead 30 / idle 40 / active 30 %), LOOKUP batch of {n_calls} calls x {cb} "
                    f"blocks ({hit:.0%} prefix hits), classify, select 10%; median of {reps} after 1 warm-up; L2 flushed "
                    f"(512 MiB fill) before every timed call",
        "hash_lookup": {"blocks_per_call": n_blocks, "call_ms": med(look_ms), "kernels_ms": look_k,
                        "blocks_per_s": n_blocks / (med(look_ms) / 1e3), "blocks_per_s_kernels": n_blocks / (look_k / 1e3),
                        "algorithmic_bytes_per_block": 136, "achieved_GBs": n_blocks * 136 / (look_k / 1e3) / 1e9,
                        "frac_hbm": n_blocks * 136 / (look_k / 1e3) / 1e9 / hbm_peak},
        "classify": {"mappings": n_blocks, "entries": n_res, "call_ms": med(cls_ms),
                     "what": "event-driven update after the LOOKUP batch: 64 new contexts x 16,128 mappings",
                     "kernels_ms": med(cls_k),
                     "achieved_GBs": 16 * n_blocks / (med(cls_k) / 1e3) / 1e9,
                     "frac_hbm": 16 * n_blocks / (med(cls_k) / 1e3) / 1e9 / hbm_peak,
                     "after_one_context_changed_state_ms": med(cls_edit_ms),
                     "after_one_context_changed_state_kernels_ms": med(cls_edit_k),
                     "after_one_context_changed_state_warm_l2_ms": med(cls_edit_warm_ms),
                     "after_one_context_changed_state_warm_l2_kernels_ms": med(cls_edit_warm_k),
                     "after_all_contexts_suspended_ms": med(cls_done_ms),
                     "full_recomputation_ms": med(cls_full_ms)},
        "select": {"resident": n_res, "victims": len(v), "call_ms": med(sel_ms), "kernels_ms": sel_k,
                   "resident_blocks_per_s": n_res / (med(sel_ms) / 1e3),
                   "achieved_GBs": (8 * n_res + 4 * len(v)) / (sel_k / 1e3) / 1e9,
                   "frac_hbm": (8 * n_res + 4 * len(v)) / (sel_k / 1e3) / 1e9 / hbm_peak},
    }
    eng.close()
    del eng, flush
    torch.cuda.empty_cache()
    return out


def cpu_arm(args, setup, turns, n_ff, n_steps, n_warm, n_hbm_blocks, n_host_blocks):
    """The CPU oracle, as it stands, on the same steps: payload copies are plain memcpy on one core."""
    from oracle import kvt_oracle
    kvt_oracle.build()
    eng = kvt_oracle.OracleEngine(n_hbm_blocks=n_hbm_blocks, n_host_blocks=n_host_blocks, max_contexts=4,
                                  **W.GEO_8B.kwargs())
    opt = W.ReplayOptions(payload=None, record_states=False)
    ident = lambda a: a
    for ev in setup:
        apply_event(eng, ev, ident)
    for t in range(n_ff):
        pre, ctxs, post = turns[t]
        for ev in pre:
            apply_event(eng, ev, ident)
        eng.map_blocks(ctxs, 0)
        eng.map_blocks(ctxs, 1)
        for c in ctxs:
            eng.prefill_done(c)
        for ev in post:
            apply_event(eng, ev, ident)
    pressure_evict(eng, CPU_PRESSURE_CAP)
    for t in range(n_ff, n_ff + n_warm):
        run_step(eng, turns[t], ident, opt, cap=CPU_PRESSURE_CAP)
    timer = StageTimer(eng)
    s0 = eng.get_stats()
    timer.reset()
    t0 = time.perf_counter()
    for t in range(n_ff + n_warm, n_ff + n_warm + n_steps):
        run_step(eng, turns[t], ident, opt, cap=CPU_PRESSURE_CAP)
    sec = time.perf_counter() - t0
    s1 = eng.get_stats()
    d = {k: s1[k] - s0[k] for k in s1}
    return dict(sec=sec, stats=d, block_bytes=eng.block_bytes, stage_ms=dict(timer.ms))


def reduce_over_ranks(local, dist=None, device="cpu"):
    """Whole-job figures from per-rank ones: 'ms' is the maximum over ranks (the job is as slow as its
    slowest rank), every other entry is summed (units processed by all ranks). Ranks are independent
    sessions; this is the only communication of a multi-GPU run and it happens outside the timed region."""
    if dist is None:
        return dict(local)
    import torch
    keys = sorted(local)
    t = torch.tensor([float(local[k]) for k in keys], dtype=torch.float64, device=device)
    mx = t.clone()
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    dist.all_reduce(mx, op=dist.ReduceOp.MAX)
    return {k: (mx[i].item() if k == "ms" else t[i].item()) for i, k in enumerate(keys)}


def kv_bytes(d, block_bytes):
    return (d["offloaded"] + d["reloaded"]) * block_bytes


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    W_, K = args.warmup, args.steps
    n_hbm_blocks = int(args.hbm_gib * GiB) // W.GEO_8B.block_bytes
    setup, turns, target = make_turns(args.seed + rank, W_ + K + 4)
    n_ff = len(turns) - (W_ + K)
    workload = (f"C2 single long ReAct session under tier pressure: seed {args.seed}, {len(turns)} turns to "
                f"{target} tokens, fast-forward {n_ff} turns then {W_}+{K} timed calls; 8B-class KV 32x8x128 bf16 "
                f"(2 MiB/block); HBM pool {n_hbm_blocks} blocks ({args.hbm_gib:g} GiB)")

    if args.impl == "reference":
        if rank != 0:
            return
        n_host_blocks = min(int(args.host_gib * GiB), int(mem_available_bytes() * 0.5)) // W.GEO_8B.block_bytes
        r = cpu_arm(args, setup, turns, n_ff, K, W_, n_hbm_blocks, n_host_blocks)
        gbs = kv_bytes(r["stats"], r["block_bytes"]) / r["sec"] / 1e9
        line = {
            "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus, "steps": K,
            "warmup": W_, "ms_per_step": r["sec"] * 1e3 / K, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "u8", "data": "synthetic",
            "config": {"workload": workload, "host_tier_blocks": n_host_blocks},
            "blocks_hashed_looked_up_per_s": r["stats"]["blocks_hashed"] / r["sec"],
            "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle", "host": host_info(),
                             "stage_wall_ms_per_step": {k: round(x / K, 3) for k, x in r["stage_ms"].items()},
                             "sample": f"the same {K} calls with the tier pressure capped at {CPU_PRESSURE_CAP} blocks "
                                       f"(1 GiB each way) per step; whole path incl. payload memcpy; one thread"},
            "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        }
        print(json.dumps(line))
        return

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    from paper_2609_39819_b200 import build as kbuild
    kbuild.build_lib()       # every rank asks; a file lock lets one of them compile and the others wait for the result
    barrier = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        barrier = lambda: (dist.barrier(), torch.cuda.synchronize())
        barrier()
    from paper_2609_39819_b200 import binding as B
    B.load_library()
    hbm_peak, peak_kind = measured_peaks()
    link = host_link_peaks(torch)
    hbm_now = hbm_copy_this_run(torch)

    # ---- value arm: everything resident in HBM ------------------------------------------------------------
    sampler = ClockSampler(local_rank, torch)
    free_b, _total = torch.cuda.mem_get_info()
    want2 = int(args.host_gib * GiB) // W.GEO_8B.block_bytes
    fit2 = int((free_b - n_hbm_blocks * W.GEO_8B.block_bytes - 6 * GiB) // W.GEO_8B.block_bytes)
    tier2_dev_blocks = max(min(want2, fit2), 9000)
    v = gpu_arm(args, torch, B, setup, turns, n_ff, False, tier2_dev_blocks, n_hbm_blocks, rank, world, barrier)
    clocks = sampler.stop(*v["wall"])

    # ---- e2e arm: pinned host tier, tokens from pinned host buffers ---------------------------------------
    e = None
    host_blocks = 0
    if not args.skip_e2e:
        # pinned host tier: the configured size, but never more than this rank's share of half the free host RAM
        budget = min(int(args.host_gib * GiB), int(mem_available_bytes() * 0.5) // max(world, 1))
        host_blocks = budget // W.GEO_8B.block_bytes
        if world > 1:                # every rank must take the same decision below
            import torch.distributed as dist
            hb = torch.tensor([host_blocks], dtype=torch.int64, device="cuda")
            dist.all_reduce(hb, op=dist.ReduceOp.MIN)
            host_blocks = int(hb.item())
        if host_blocks >= 5000:      # the session keeps up to ~4.5 K blocks in the host tier
            sampler = ClockSampler(local_rank, torch)
            e = gpu_arm(args, torch, B, setup, turns, n_ff, True, host_blocks, n_hbm_blocks, rank, world, barrier)
            clocks_e2e = sampler.stop(*e["wall"])

    vbytes = kv_bytes(v["stats"], v["block_bytes"])
    dist = None
    if world > 1:
        import torch.distributed as dist
    tot = reduce_over_ranks({"ms": v["ms"], "bytes": vbytes, "hashed": v["stats"]["blocks_hashed"],
                             "launches": v["stats"]["kernel_launches"]}, dist, "cuda")
    ms, tot_bytes, tot_hashed, launches = tot["ms"], tot["bytes"], tot["hashed"], tot["launches"]
    if e:
        te = reduce_over_ranks({"ms": e["ms"], "bytes": kv_bytes(e["stats"], e["block_bytes"])}, dist, "cuda")
        e_ms, e_bytes = te["ms"], te["bytes"]
    if rank != 0:
        return

    st = v["stats"]
    mover_s = st["mover_ns"] / 1e9
    achieved = 2 * st["mover_bytes"] / mover_s / 1e9 if mover_s else 0.0
    per_launch_bytes = 2 * st["mover_bytes"] / max(st["mover_launches"], 1)
    traffic_ratio = mover_traffic_ratio()
    roofline = {
        "bound": "hbm", "kernel": "k_move_tiles<8>", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s",
        "frac": achieved / hbm_peak, "peak_kind": f"{peak_kind} copy bandwidth (MEASURED_PEAKS.json hbm_gbs)",
        "frac_of_nominal_8TBs": achieved / 8000.0, "torch_copy_gbs_this_run": hbm_now,
        "launches": st["mover_launches"], "avg_launch_ms": mover_s * 1e3 / max(st["mover_launches"], 1),
        "algorithmic_bytes_per_launch": per_launch_bytes,
        "traffic": None if traffic_ratio is None else traffic_ratio * per_launch_bytes,
        "traffic_source": "profiles/mover_8b_hbm_to_hbm.md (ncu capture of a 1024-block launch, scaled by blocks moved)",
    }
    line = {
        "metric": METRIC, "value": tot_bytes / (ms / 1e3) / 1e9, "unit": "GB/s", "n_gpus": args.gpus, "steps": K,
        "warmup": W_, "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u8", "data": "synthetic",
        "config": {"workload": workload, "second_tier_blocks_value_arm": tier2_dev_blocks,
                   "host_tier_blocks_e2e_arm": host_blocks,
                   "l2": "inputs larger than L2: every step streams GiBs of KV blocks; no flush needed",
                   "per_rank": "independent session per GPU, no collective on the data path" if world > 1 else "1 GPU"},
        "blocks_hashed_looked_up_per_s": tot_hashed / (ms / 1e3),
        "kv_blocks_moved_per_step": (st["offloaded"] + st["reloaded"]) / K,
        "blocks_hashed_per_step": st["blocks_hashed"] / K,
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": roofline,
        "stage_wall_ms_per_step": {k: round(x / K, 4) for k, x in v["stage_ms"].items()},
        "verified_blocks": {"value_arm": v["verified"], "e2e_arm": e["verified"] if e else None},
        "host_cpu": host_info(),
    }
    if e:
        es = e["stats"]
        e_mover_s = es["mover_ns"] / 1e9
        line["clocks_e2e"] = clocks_e2e
        line["e2e"] = {
            "value": e_bytes / (e_ms / 1e3) / 1e9, "unit": "GB/s", "ms_per_step": e_ms / K,
            "h2d_bytes_per_step": (es["bytes_h2d"] + e["tok_bytes"]) / K,
            # payload gathered to the host tier + what the calls return: two block maps per call
            # (13 B per block), victim lists (5 B per victim), one 128-byte status block per synchronising call
            "d2h_bytes_per_step": (es["bytes_d2h"] + 26 * es["blocks_hashed"] + 5 * (es["offloaded"] + es["dropped"])
                                   + 128 * sum(e["stage_calls"].values())) / K,
        }
        line["host_link"] = {
            "achieved": es["mover_bytes"] / e_mover_s / 1e9 if e_mover_s else 0.0, "unit": "GB/s",
            "peak_h2d": link["h2d"], "peak_d2h": link["d2h"],
            "frac": (es["mover_bytes"] / e_mover_s / 1e9) / (0.5 * (link["h2d"] + link["d2h"])) if e_mover_s else 0.0,
            "peak_kind": "measured: 1 GiB pinned cudaMemcpyAsync per direction, best of 10, this run",
            "stage_wall_ms_per_step": {k: round(x / K, 4) for k, x in e["stage_ms"].items()},
        }
    if e and not args.skip_inclusive and world == 1:
        # the same end-to-end steps with inclusive tiers: reloaded blocks keep a clean host copy, so the next
        # offload of them moves no bytes (a 24 GiB host tier is enough for the session and its copies)
        i = gpu_arm(args, torch, B, setup, turns, n_ff, True, min(host_blocks, 12288), n_hbm_blocks, policy_flags=2)
        ist = i["stats"]
        line["e2e_inclusive_tiers"] = {
            "value": kv_bytes(ist, i["block_bytes"]) / (i["ms"] / 1e3) / 1e9, "unit": "GB/s (blocks offloaded + reloaded, "
            "whether or not bytes had to move)", "ms_per_step": i["ms"] / K,
            "offloaded_per_step": ist["offloaded"] / K, "offloaded_without_copy_per_step": ist["offloaded_clean"] / K,
            "reloaded_per_step": ist["reloaded"] / K, "bytes_over_link_per_step": (ist["bytes_d2h"] + ist["bytes_h2d"]) / K,
            "verified_blocks": i["verified"],
        }
    if hasattr(torch._C, "_host_emptyCache"):
        torch._C._host_emptyCache()      # give the pinned pools of the arms above back to the OS
    if e and not args.skip_two_tenants and world == 1 and mem_available_bytes() > 32 * GiB:
        seq = two_tenant_arm(args, torch, B, n_ff, False)
        dup = two_tenant_arm(args, torch, B, n_ff, True)
        line["e2e_two_sessions"] = {
            "workload": "two C2 sessions (seeds s, s+1) taking turns on a 24 GiB HBM pool (1.5 sessions) over a 24 GiB "
                        "pinned host tier; no artificial pressure: every call reloads part of its own prefix and "
                        "pushes part of the other session out",
            "unit": "GB/s (blocks offloaded + reloaded)", "offload_then_reload": seq, "one_exchange_per_call": dup,
        }
    if e and not args.skip_c3 and world == 1:
        line["c3"] = c3_arm(args, torch, B, link)
    if not args.skip_stress and world == 1:
        line["metadata_stress"] = metadata_stress(torch, B, hbm_peak)
    if not args.skip_cpu and world == 1:
        n_host_blocks = min(int(args.host_gib * GiB), int(mem_available_bytes() * 0.5)) // W.GEO_8B.block_bytes
        c = cpu_arm(args, setup, turns, n_ff, min(args.cpu_steps, K), 1, n_hbm_blocks, n_host_blocks)
        line["cpu_baseline"] = {
            "value": kv_bytes(c["stats"], c["block_bytes"]) / c["sec"] / 1e9, "unit": "GB/s", "cores": 1,
            "kind": "oracle",
            "sample": f"first {min(args.cpu_steps, K)} of the {K} timed calls (after 1 warm-up) with the tier pressure "
                      f"capped at {CPU_PRESSURE_CAP} blocks (1 GiB each way) per step; whole path incl. payload "
                      f"memcpy; {c['sec']:.1f} s on one thread",
            "blocks_hashed_looked_up_per_s": c["stats"]["blocks_hashed"] / c["sec"],
            "stage_wall_ms_per_step": {k: round(x / min(args.cpu_steps, K), 3) for k, x in c["stage_ms"].items()},
            "host": host_info(),
        }
        line["cpu_baseline"].update(cpu_stage_arm())
    print(json.dumps(line))


if __name__ == "__main__":
    main()
