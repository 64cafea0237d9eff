"""Seeded synthetic inputs and the replay driver shared by the tests and the benchmark.

This module holds none of the method's arithmetic (no hashing, no table, no classification, no
ordering, no copies): it only draws random agent traces and id lists and sequences API calls on an
engine object. It works with any engine exposing the method names of the CUDA binding
(`paper_2609_39819_b200.binding.Engine`); the tests also drive the CPU oracle's front end through it.
It imports neither of them.

The traces stand in for the paper's Codex-on-TerminalBench and production agent traces (Section
2.2, Table 1; Section 8.1), which are not available: token ids are uniform random, message sizes,
edit probabilities and pool geometries follow the five benchmark configurations (C1..C5).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

VOCAB = 151552
TIER_HBM, TIER_HOST, TIER_REMOTE, TIER_NONE = 0, 1, 2, 0xFF
MAP_LOOKUP, MAP_ADMIT = 0, 1
GiB = 1 << 30
GPU_ONLY_STATS = ("table_rebuilds", "tombstones", "kernel_launches", "mover_launches", "mover_ns", "mover_bytes",
                  "lookup_ns", "lookup_blocks", "select_ns", "select_slots", "blocks_rehashed", "classify_ns", "classify_items")
STATE_COPY, STATE_HAS_COPY = 0xFE, 0x80


# ------------------------------------------------------------------------------------------------
# KV geometries
# ------------------------------------------------------------------------------------------------
@dataclass(frozen=True)
class Geometry:
    name: str
    n_layers: int
    n_kv_heads: int
    head_dim: int
    elem_bytes: int = 2

    @property
    def chunk_bytes(self):  # one (layer, K|V) slice of a 16-token block
        return 16 * self.n_kv_heads * self.head_dim * self.elem_bytes

    @property
    def n_chunks(self):
        return 2 * self.n_layers

    @property
    def block_bytes(self):
        return self.chunk_bytes * self.n_chunks

    def kwargs(self):
        return dict(n_layers=self.n_layers, n_kv_heads=self.n_kv_heads, head_dim=self.head_dim,
                    elem_bytes=self.elem_bytes)


GEO_TOY = Geometry("toy-2x2x64", 2, 2, 64)          # 16 KiB / block
GEO_128K = Geometry("mid-4x4x128", 4, 4, 128)       # 128 KiB / block
GEO_512K = Geometry("mid-8x8x128", 8, 8, 128)       # 512 KiB / block
GEO_8B = Geometry("8b-32x8x128", 32, 8, 128)        # 2 MiB / block (128 KiB / token)
GEO_GLM = Geometry("glm-92x8x128", 92, 8, 128)      # 5.75 MiB / block (368 KiB / token)


# ------------------------------------------------------------------------------------------------
# Traces: lists of events
#   ("spawn", ctx) ("fork", parent, child, end) ("append", ctx, tokens) ("replace", ctx, s, e, tokens)
#   ("remove", ctx, s, e) ("one_off", ctx, s, e_or_None) ("terminate", ctx) ("call", [ctx, ...])
#   ("pin", ctx, s, e) ("unpin", ctx, s, e)
# A "call" is one LLM call per listed context, carried through the whole cache path by `replay`.
# ------------------------------------------------------------------------------------------------
def _tokens(rng, n):
    return rng.integers(0, VOCAB, size=int(n), dtype=np.uint32)


def _loguniform(rng, a, b):
    return int(math.floor(a * math.exp(rng.random() * math.log(b / a))))


def trace_c1(seed: int):
    """C1: one root context, 3 calls, 2-6 appended messages of 50-400 tokens per call; per appended
    message replace (p=0.1), remove (p=0.05) or fork a subagent (p=0.05). A subagent appends 1-2
    messages (one_off with p=0.5), runs one call, idles through the parent's next call, then appends
    once more, runs a second call and terminates. Every third seed pins the root's first message
    right after appending it (a system prompt); every sixth unpins it again before the last call."""
    rng = np.random.default_rng([1, seed])
    ev = [("spawn", 0)]
    n_msgs = 0
    next_ctx = 1
    pending = []
    for _call in range(3):
        if _call == 2 and seed % 6 == 0:
            ev.append(("unpin", 0, 0, 1))
        for _ in range(int(rng.integers(2, 7))):
            ev.append(("append", 0, _tokens(rng, rng.integers(50, 401))))
            n_msgs += 1
            if n_msgs == 1 and _call == 0 and seed % 3 == 0:
                ev.append(("pin", 0, 0, 1))
            u = rng.random()
            if u < 0.10 and n_msgs:
                j = int(rng.integers(0, n_msgs))
                ev.append(("replace", 0, j, j + 1, _tokens(rng, rng.integers(50, 401))))
            elif u < 0.15 and n_msgs > 1:
                j = int(rng.integers(0, n_msgs))
                ev.append(("remove", 0, j, j + 1))
                n_msgs -= 1
            elif u < 0.20 and next_ctx < 60:
                child = next_ctx
                next_ctx += 1
                ev.append(("fork", 0, child, n_msgs))
                if rng.random() < 0.5:
                    ev.append(("one_off", child, 0, None))
                for _k in range(int(rng.integers(1, 3))):
                    ev.append(("append", child, _tokens(rng, rng.integers(50, 401))))
                ev.append(("call", [child]))
                pending.append(child)
        ev.append(("call", [0]))
        for child in pending:
            ev.append(("append", child, _tokens(rng, rng.integers(50, 401))))
            ev.append(("call", [child]))
            ev.append(("terminate", child))
        pending = []
    return ev


def trace_c2(seed: int, target_tokens: int = 131072, max_turns: int = 100, scale: float = 1.0):
    """C2: one long ReAct session. Each turn appends an assistant message (100-2K tokens) and a
    tool result (200-8K tokens), both log-uniform, then calls; replace p=0.08 / remove p=0.04 of a
    non-first message per turn; one scratch message per call that is marked one_off and removed
    after the call. `scale` shrinks message sizes and the target for quick tests."""
    rng = np.random.default_rng([2, seed])
    ev = [("spawn", 0), ("append", 0, _tokens(rng, max(16, int(600 * scale))))]  # system prompt
    lens = [len(ev[-1][2])]
    for _turn in range(max_turns):
        for lo, hi in ((100, 2048), (200, 8192)):
            n = max(1, int(_loguniform(rng, lo, hi) * scale))
            ev.append(("append", 0, _tokens(rng, n)))
            lens.append(n)
        u = rng.random()
        if u < 0.08 and len(lens) > 1:
            j = int(rng.integers(1, len(lens)))
            n = max(1, int(_loguniform(rng, 100, 2048) * scale))
            ev.append(("replace", 0, j, j + 1, _tokens(rng, n)))
            lens[j] = n
        elif u < 0.12 and len(lens) > 2:
            j = int(rng.integers(1, len(lens)))
            ev.append(("remove", 0, j, j + 1))
            lens.pop(j)
        n = max(1, int(rng.integers(50, 401) * scale))
        ev.append(("append", 0, _tokens(rng, n)))
        ev.append(("one_off", 0, len(lens), len(lens) + 1))
        ev.append(("call", [0]))
        ev.append(("remove", 0, len(lens), len(lens) + 1))
        if sum(lens) >= target_tokens * scale:
            break
    return ev


def trace_c3(seed: int, n_sessions: int = 32, min_len: int = 32768, max_len: int = 264192, scale: float = 1.0):
    """C3: concurrent sessions grown turn by turn (round-robin, one batch call per round), each
    forking 0-4 subagents that share its prefix, run 1-5 calls, terminate and return a summary the
    parent later replaces or removes with p=0.3."""
    rng = np.random.default_rng([3, seed])
    ev = []
    targets = [int(_loguniform(rng, min_len, max_len) * scale) for _ in range(n_sessions)]
    lens = [[] for _ in range(n_sessions)]
    n_forks = [int(rng.integers(0, 5)) for _ in range(n_sessions)]
    summaries = [[] for _ in range(n_sessions)]  # message indices of subagent summaries
    next_ctx = n_sessions
    for s in range(n_sessions):
        ev.append(("spawn", s))
        n = max(16, int(600 * scale))
        ev.append(("append", s, _tokens(rng, n)))
        lens[s].append(n)
        if s % 4 == 0:
            ev.append(("pin", s, 0, 1))   # every fourth session pins its system prompt
    live = set(range(n_sessions))
    while live:
        batch = []
        for s in sorted(live):
            for lo, hi in ((100, 2048), (200, 8192)):
                n = max(1, int(_loguniform(rng, lo, hi) * scale))
                ev.append(("append", s, _tokens(rng, n)))
                lens[s].append(n)
            if summaries[s] and rng.random() < 0.3:
                j = summaries[s].pop(0)
                if rng.random() < 0.5:
                    n = max(1, int(_loguniform(rng, 100, 1024) * scale))
                    ev.append(("replace", s, j, j + 1, _tokens(rng, n)))
                    lens[s][j] = n
                else:
                    ev.append(("remove", s, j, j + 1))
                    lens[s].pop(j)
                    summaries[s] = [k - 1 if k > j else k for k in summaries[s]]
            batch.append(s)
        ev.append(("call", batch))
        for s in list(batch):
            if n_forks[s] and rng.random() < 0.15:
                n_forks[s] -= 1
                child = next_ctx
                next_ctx += 1
                ev.append(("fork", s, child, len(lens[s])))
                for _k in range(int(rng.integers(1, 6))):
                    n = max(1, int(_loguniform(rng, 200, 4096) * scale))
                    ev.append(("append", child, _tokens(rng, n)))
                    ev.append(("call", [child]))
                ev.append(("terminate", child))
                n = max(1, int(_loguniform(rng, 100, 1024) * scale))
                ev.append(("append", s, _tokens(rng, n)))
                summaries[s].append(len(lens[s]))
                lens[s].append(n)
            if sum(lens[s]) >= targets[s]:
                ev.append(("terminate", s))
                live.discard(s)
    return ev, next_ctx


def trace_c3_timed(seed: int, n_sessions: int = 32, min_len: int = 32768, max_len: int = 264192, scale: float = 1.0,
                   long_wait_p: float = 0.0):
    """C3 with a notion of time (Section 6.2: newly suspended KV waits while tools, sub-agents or other physical
    stages run). Same sessions, turns, forks and edits as trace_c3, but every call is a batch of one and the order
    of the calls comes from an event clock: after a call a session is busy for the call itself (0.3-1.5 s) plus a
    tool wait, log-uniform 1-6 s, or 30-120 s with probability long_wait_p; a parent waits for its subagent, whose
    calls take their own turns on the clock. Returns (events, number of context ids used)."""
    import heapq
    rng = np.random.default_rng([33, seed])
    ev = []
    targets = [int(_loguniform(rng, min_len, max_len) * scale) for _ in range(n_sessions)]
    lens = [[] for _ in range(n_sessions)]
    n_forks = [int(rng.integers(0, 5)) for _ in range(n_sessions)]
    summaries = [[] for _ in range(n_sessions)]
    next_ctx = n_sessions
    ready = []          # (time, tie-break, kind, session, payload)
    tick = 0

    def wait():
        t = 0.3 + 1.2 * rng.random()
        t += _loguniform(rng, 30, 120) if rng.random() < long_wait_p else _loguniform(rng, 1, 6)
        return t

    for s in range(n_sessions):
        ev.append(("spawn", s))
        n = max(16, int(600 * scale))
        ev.append(("append", s, _tokens(rng, n)))
        lens[s].append(n)
        if s % 4 == 0:
            ev.append(("pin", s, 0, 1))
        heapq.heappush(ready, (rng.random(), tick, "turn", s, None))
        tick += 1
    while ready:
        now, _t, kind, s, pay = heapq.heappop(ready)
        if kind == "turn":
            for lo, hi in ((100, 2048), (200, 8192)):
                n = max(1, int(_loguniform(rng, lo, hi) * scale))
                ev.append(("append", s, _tokens(rng, n)))
                lens[s].append(n)
            if summaries[s] and rng.random() < 0.3:
                j = summaries[s].pop(0)
                if rng.random() < 0.5:
                    n = max(1, int(_loguniform(rng, 100, 1024) * scale))
                    ev.append(("replace", s, j, j + 1, _tokens(rng, n)))
                    lens[s][j] = n
                else:
                    ev.append(("remove", s, j, j + 1))
                    lens[s].pop(j)
                    summaries[s] = [k - 1 if k > j else k for k in summaries[s]]
            ev.append(("call", [s]))
            if sum(lens[s]) >= targets[s]:
                ev.append(("terminate", s))
                continue
            if n_forks[s] and rng.random() < 0.15:      # the parent now waits for a subagent
                n_forks[s] -= 1
                child = next_ctx
                next_ctx += 1
                ev.append(("fork", s, child, len(lens[s])))
                heapq.heappush(ready, (now + wait(), tick, "sub", s, (child, int(rng.integers(1, 6)))))
            else:
                heapq.heappush(ready, (now + wait(), tick, "turn", s, None))
            tick += 1
        else:                                            # one call of a subagent
            child, left = pay
            n = max(1, int(_loguniform(rng, 200, 4096) * scale))
            ev.append(("append", child, _tokens(rng, n)))
            ev.append(("call", [child]))
            if left > 1:
                heapq.heappush(ready, (now + wait(), tick, "sub", s, (child, left - 1)))
            else:
                ev.append(("terminate", child))
                n = max(1, int(_loguniform(rng, 100, 1024) * scale))
                ev.append(("append", s, _tokens(rng, n)))
                summaries[s].append(len(lens[s]))
                lens[s].append(n)
                heapq.heappush(ready, (now + wait(), tick, "turn", s, None))
            tick += 1
    return ev, next_ctx


# ------------------------------------------------------------------------------------------------
# C4: metadata-only lookup / eviction stress
# ------------------------------------------------------------------------------------------------
@dataclass
class C4Inputs:
    chain_tokens: list           # resident chains: token arrays
    chain_slot0: list            # first slot of each chain
    state: np.ndarray            # per resident block
    stamp: np.ndarray
    depth: np.ndarray
    slot: np.ndarray
    calls: list                  # incoming call token arrays
    n_resident: int = 0


def inputs_c4(seed: int = 1, n_resident: int = 1 << 20, chain_blocks: int = 16128, n_calls: int = 64,
              stamp_bits: int = 24):
    """Resident chains (state mix dead 30% / idle 40% / active 30%, uniform stamps) plus incoming
    calls that share a random 0-90% prefix with a resident chain."""
    rng = np.random.default_rng([4, seed])
    chains, slot0 = [], []
    left, s0 = n_resident, 0
    while left > 0:
        nb = min(chain_blocks, left)
        chains.append(_tokens(rng, nb * 16))
        slot0.append(s0)
        s0 += nb
        left -= nb
    u = rng.random(n_resident)
    state = np.where(u < 0.3, 0, np.where(u < 0.7, 1, 2)).astype(np.uint8)
    stamp = rng.integers(0, 1 << stamp_bits, size=n_resident, dtype=np.uint32)
    depth = np.concatenate([np.arange(len(c) // 16, dtype=np.uint32) for c in chains])
    slot = np.arange(n_resident, dtype=np.uint32)
    calls = []
    for i in range(n_calls):
        src = chains[i % len(chains)]
        nb_src = len(src) // 16
        shared = min(int(rng.random() * 0.9 * chain_blocks), nb_src)
        calls.append(np.concatenate([src[: shared * 16], _tokens(rng, (chain_blocks - shared) * 16)]))
    return C4Inputs(chains, slot0, state, stamp, depth, slot, calls, n_resident)


# ------------------------------------------------------------------------------------------------
# C5: id lists for the movement sweep
# ------------------------------------------------------------------------------------------------
def ids_c5(seed: int, n: int, pool_slots: int, permuted: bool):
    """n distinct slot ids of a pool: 0..n-1, or a seeded random selection in random order."""
    if not permuted:
        return np.arange(n, dtype=np.uint32)
    rng = np.random.default_rng([5, seed, n, pool_slots])
    return rng.permutation(pool_slots)[:n].astype(np.uint32)


# ------------------------------------------------------------------------------------------------
# Payloads: a pure function of the block key, so any slot can be verified at any time
# ------------------------------------------------------------------------------------------------
def payload_normal_bf16(key: int, block_bytes: int) -> np.ndarray:
    """Seeded standard-normal values rounded to bf16 (round to nearest even), as bytes."""
    rng = np.random.default_rng(int(key))
    x = rng.standard_normal(block_bytes // 2, dtype=np.float32).view(np.uint32)
    r = ((x >> 16) & 1) + 0x7FFF
    return ((x + r) >> 16).astype(np.uint16).view(np.uint8)


def payload_pattern(key: int, block_bytes: int) -> np.ndarray:
    """Cheap 32-bit counter pattern keyed by the block key."""
    lo, hi = int(key) & 0xFFFFFFFF, int(key) >> 32
    i = np.arange(block_bytes // 4, dtype=np.uint64)
    w = ((lo + i * 0x9E3779B1) & 0xFFFFFFFF) ^ hi
    return w.astype(np.uint32).view(np.uint8)


# ------------------------------------------------------------------------------------------------
# Replay driver
# ------------------------------------------------------------------------------------------------
@dataclass
class ReplayOptions:
    payload: object = None        # callable(key, block_bytes) -> uint8 array, or None (metadata only)
    writer: object = None         # callable(engine, slot, key): writes a new HBM block's payload in place (large blocks)
    record_states: bool = True    # record per-tier states / entries after every call (slow on big pools)
    verify_payload_every: int = 0 # every k-th call, read back every occupied slot and compare with payload(key)
    use_exchange: bool = False    # a call's reloads and the offloads that make room for them go out as one exchange
    counters: dict = field(default_factory=dict)


def evict(eng, n, n_pinned_incoming=0, reload_slots=None):
    """Frees n HBM slots in the engine's victim order: dead blocks are dropped, live ones go to the
    host tier, for which room is made first by releasing the host tier's own first victims. Pinned
    blocks are only asked for when Pinned blocks are coming in, and only for as many (Algorithm 1).
    With `reload_slots` (host slots the caller wants back in HBM) the offload and that reload are issued
    together."""
    rec = {}
    victims, vstates = eng.select_victims(TIER_HBM, n)
    if len(victims) < n and n_pinned_incoming > 0:
        want = len(victims) + min(n - len(victims), n_pinned_incoming)
        victims, vstates = eng.select_victims(TIER_HBM, want, include_pinned=True)
    rec["victims"] = victims.copy()
    rec["vstates"] = vstates.copy()
    # victims that need a free host slot: live ones without a clean host copy
    n_live = int((((vstates & 0x7F) > 0) & ((vstates & STATE_HAS_COPY) == 0)).sum())
    free_host = eng.n_host_blocks - eng.get_stats()["occ_host"]
    if n_live > free_host:
        hv, hs = eng.select_victims(TIER_HOST, n_live - free_host)
        rec["host_victims"] = hv.copy()
        rec["host_vstates"] = hs.copy()
        if len(hv) and getattr(eng, "n_remote_blocks", 0):
            # a third tier exists: the host tier's victims move down instead of being lost (clean copies of HBM
            # blocks are simply released), after the remote tier has made room by releasing its own first victims
            copies = hs == STATE_COPY
            if copies.any():
                eng.release(TIER_HOST, hv[copies])
            down, dstates = hv[~copies], hs[~copies]
            n_down = int(((dstates & 0x7F) > 0).sum())
            free_remote = eng.n_remote_blocks - eng.get_stats()["occ_remote"]
            if n_down > free_remote:
                rv, rs = eng.select_victims(TIER_REMOTE, n_down - free_remote)
                rec["remote_victims"] = rv.copy()
                if len(rv):
                    eng.release(TIER_REMOTE, rv)
            if len(down):
                rec["demote"] = eng.move(TIER_HOST, TIER_REMOTE, down)
        elif len(hv):
            eng.release(TIER_HOST, hv)
    if reload_slots is not None and len(reload_slots):
        # both directions in one call; what found no free HBM slot at the start follows once the offload has made room
        rc, n_out, n_drop, n_in = eng.exchange(victims, reload_slots)
        rec["exchange"] = (rc, n_out, n_drop, n_in)
        if n_in < len(reload_slots):
            rec["reload"] = eng.reload(reload_slots[n_in:])
    elif len(victims):
        rec["offload"] = eng.offload(victims)
    return rec


def run_call(eng, ctxs, opt: ReplayOptions):
    """One LLM call per listed context through the cache path: lookup, make room following
    Algorithm 1's release order (victims come from the engine), reload host hits, admit, write the
    new blocks' payload ("prefill"), prefill-done. Returns everything the engine reported."""
    rec = {}
    info = eng.map_blocks(ctxs, MAP_LOOKUP)
    rec["lookup"] = info.copy()
    st = eng.get_stats()
    free_hbm = eng.n_hbm_blocks - st["occ_hbm"]
    need = int(info["n_hit_host"].sum()) + int(info["n_hit_remote"].sum()) + int(info["n_admissible"].sum()) - free_hbm
    host_slots, remote_slots = [], []
    for c, inf in zip(ctxs, info):
        if inf["n_hit_host"] or inf["n_hit_remote"]:
            _keys, tier, slot = eng.get_block_map(c)
            h = int(inf["hit_len"])
            host_slots.append(slot[:h][tier[:h] == TIER_HOST])
            remote_slots.append(slot[:h][tier[:h] == TIER_REMOTE])
    hs = rs = None
    if host_slots:
        hs = np.concatenate(host_slots)
        hs = hs[np.sort(np.unique(hs, return_index=True)[1])]  # a shared host block is reloaded once
        rs = np.concatenate(remote_slots)
        rs = rs[np.sort(np.unique(rs, return_index=True)[1])]
        hs, rs = (hs if len(hs) else None), (rs if len(rs) else None)
    if need > 0 and opt.use_exchange and hs is not None:
        rec.update(evict(eng, need, int(info["n_pinned"].sum()), reload_slots=hs))
    else:
        if need > 0:
            rec.update(evict(eng, need, int(info["n_pinned"].sum())))
        if hs is not None:
            rec["reload"] = eng.reload(hs)
    if rs is not None:
        rec["promote"] = eng.move(TIER_REMOTE, TIER_HBM, rs)   # remote hits come straight up into HBM
    adm = eng.map_blocks(ctxs, MAP_ADMIT)
    rec["admit"] = adm.copy()
    maps = []
    for c, inf in zip(ctxs, adm):
        keys, tier, slot = eng.get_block_map(c)
        maps.append((keys.copy(), tier.copy(), slot.copy()))
        if opt.payload is not None or opt.writer is not None:
            for b in range(int(inf["hit_len"]), int(inf["n_held"])):
                if tier[b] == TIER_HBM:
                    if opt.writer is not None:
                        opt.writer(eng, int(slot[b]), int(keys[b]))
                    else:
                        eng.write_block(TIER_HBM, int(slot[b]), opt.payload(int(keys[b]), eng.block_bytes))
    rec["maps"] = maps
    for c in ctxs:
        eng.prefill_done(c)
    opt.counters["calls"] = opt.counters.get("calls", 0) + 1
    if opt.record_states:
        rec["states"] = [eng.get_states(t).copy() for t in engine_tiers(eng)]
        rec["entries"] = [eng.get_entries(t) for t in engine_tiers(eng)]
    rec["stats"] = {k: v for k, v in eng.get_stats().items() if k not in GPU_ONLY_STATS}
    if opt.payload is not None and opt.verify_payload_every and opt.counters["calls"] % opt.verify_payload_every == 0:
        rec["payload_ok"] = verify_payload(eng, opt.payload)
    return rec


def engine_tiers(eng):
    return (TIER_HBM, TIER_HOST, TIER_REMOTE) if getattr(eng, "n_remote_blocks", 0) else (TIER_HBM, TIER_HOST)


def verify_payload(eng, payload) -> bool:
    """Every occupied slot of every tier holds payload(key) of the block it is registered for."""
    for tier in engine_tiers(eng):
        keys = eng.get_entries(tier)["key"]
        for s in np.nonzero(keys)[0]:
            if not np.array_equal(eng.read_block(tier, int(s)), payload(int(keys[s]), eng.block_bytes)):
                return False
    return True


def replay(eng, trace, opt: ReplayOptions | None = None):
    """Generator: applies the trace to `eng`, yielding (event index, event kind, record)."""
    opt = opt or ReplayOptions()
    for i, ev in enumerate(trace):
        kind = ev[0]
        if kind == "spawn":
            eng.spawn(ev[1]); rec = None
        elif kind == "fork":
            eng.fork(ev[1], ev[2], ev[3]); rec = None
        elif kind == "append":
            eng.append(ev[1], ev[2]); rec = None
        elif kind == "replace":
            eng.replace(ev[1], ev[2], ev[3], ev[4]); rec = None
        elif kind == "remove":
            eng.remove(ev[1], ev[2], ev[3]); rec = None
        elif kind == "one_off":
            eng.one_off(ev[1], ev[2], ev[3]); rec = None
        elif kind == "terminate":
            eng.terminate(ev[1]); rec = None
        elif kind == "pin":
            eng.pin(ev[1], ev[2], ev[3]); rec = None
        elif kind == "unpin":
            eng.unpin(ev[1], ev[2], ev[3]); rec = None
        elif kind == "call":
            rec = run_call(eng, ev[1], opt)
        else:
            raise ValueError(kind)
        yield i, kind, rec


def records_equal(a, b, path="rec"):
    """Deep comparison of two replay records; returns None or the path of the first difference."""
    if isinstance(a, dict):
        if not isinstance(b, dict) or a.keys() != b.keys():
            return f"{path}: keys {sorted(a) if isinstance(a, dict) else a} vs {sorted(b) if isinstance(b, dict) else b}"
        for k in a:
            r = records_equal(a[k], b[k], f"{path}.{k}")
            if r:
                return r
        return None
    if isinstance(a, (list, tuple)):
        if not isinstance(b, (list, tuple)) or len(a) != len(b):
            return f"{path}: length"
        for i, (x, y) in enumerate(zip(a, b)):
            r = records_equal(x, y, f"{path}[{i}]")
            if r:
                return r
        return None
    if isinstance(a, np.ndarray) or isinstance(b, np.ndarray):
        a, b = np.asarray(a), np.asarray(b)
        if a.shape != b.shape or a.dtype != b.dtype or not np.array_equal(a, b):
            if a.shape == b.shape and a.dtype == b.dtype and a.dtype.names is None:
                bad = np.nonzero(a != b)[0][:5]
                return f"{path}: arrays differ at {bad.tolist()} ({a[bad].tolist()} vs {b[bad].tolist()})"
            return f"{path}: arrays differ ({a!r} vs {b!r})"
        return None
    return None if a == b else f"{path}: {a!r} vs {b!r}"
