"""Policy replay metrics on the synthetic traces: KV hit ratio, zombie-page share and wrong-direction
eviction ratio (definitions of Sections 2.4 and 8.1), for the paper's policy and its two ablations
("w/o RO": oldest-first inside the Suspended tier; "w/o LT": no lifecycle tracking, one tier).

Harness-side analysis only: it sequences engine calls through `workloads.replay` and post-processes what
the engine reported; it works with any engine exposing the binding's method names.

    python -m paper_2609_39819_b200.policy_metrics [--sessions 16] [--scale 0.125] [--hbm 1024] [--host 1024]
"""
from __future__ import annotations

import argparse

import numpy as np

from . import workloads as W

POLICIES = {                      # name -> (suspended_order, policy_flags)
    "lifecycle + MRU (paper)": (0, 0),
    "w/o RO (lifecycle + LRU)": (1, 0),
    "w/o LT (MRU only)": (0, 1),
    "no lifecycle + LRU": (1, 1),
    "lifecycle + MRU, unreachable blocks dead": (0, 4),
}


def replay_metrics(eng, trace):
    """Replays `trace` on `eng`; returns a dict of metrics.

    hit ratio        = reusable-prefix blocks found resident / blocks of all calls (cache-hit input tokens over
                       input tokens, at block granularity);
    zombie share     = after every call, resident blocks (both tiers) whose true state is dead / resident blocks
                       (mean and peak over calls);
    wrong direction  = among live blocks evicted from HBM in a call, the share whose next use (next call whose
                       token sequence contains the block) comes before the next use of the blocks that displaced
                       them in that call (median next use of the blocks admitted or reloaded by that call)."""
    opt = W.ReplayOptions(payload=None, record_states=True)
    calls = []
    for _i, kind, rec in W.replay(eng, trace, opt):
        if kind == "call":
            calls.append(rec)
    # next use of every key: call indices at which it appears in some context's token sequence
    uses = {}
    for t, rec in enumerate(calls):
        for keys, _tier, _slot in rec["maps"]:
            for k in keys.tolist():
                uses.setdefault(k, []).append(t)

    def next_use(key, t):
        lst = uses.get(key)
        if not lst:
            return np.inf
        j = np.searchsorted(lst, t, side="right")
        return lst[j] if j < len(lst) else np.inf

    hit = tot = 0
    zshare = []
    wrong = judged = 0
    prev_keys = [None, None]
    for t, rec in enumerate(calls):
        hit += int(rec["lookup"]["hit_len"].sum())
        tot += int(rec["lookup"]["n_blocks"].sum())
        occ = dead = 0
        for st in rec["states"]:                                # every tier the engine has
            occ += int((st != 0xFF).sum())
            dead += int((st == 0).sum())
        zshare.append(dead / occ if occ else 0.0)
        if "victims" in rec and prev_keys[0] is not None and len(rec["victims"]):
            n_done = rec["offload"][1] if "offload" in rec else 0
            victims = rec["victims"][:n_done]
            vkeys = prev_keys[0][victims]                       # keys the victim slots held before this call
            # incoming blocks of this call: admitted (new) or reloaded prefix blocks, now in HBM
            incoming = []
            for (keys, tier, _slot), inf in zip(rec["maps"], rec["admit"]):
                incoming += keys[int(inf["hit_len"]): int(inf["n_held"])].tolist()
            if incoming:
                t_in = float(np.median([next_use(k, t) for k in incoming]))
                for k in vkeys.tolist():
                    nu = next_use(k, t)
                    if np.isinf(nu) and np.isinf(t_in):
                        continue
                    judged += 1
                    wrong += nu < t_in
        prev_keys = [rec["entries"][0]["key"].copy(), rec["entries"][1]["key"].copy()]
    st = eng.get_stats()
    return {"calls": len(calls), "hit_ratio": hit / max(tot, 1), "zombie_share_mean": float(np.mean(zshare)),
            "zombie_share_peak": float(np.max(zshare)), "wrong_direction_ratio": wrong / judged if judged else 0.0,
            "evictions_judged": judged, "offloaded": st["offloaded"], "reloaded": st["reloaded"], "dropped": st["dropped"]}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--sessions", type=int, default=16)
    ap.add_argument("--scale", type=float, default=0.125)
    ap.add_argument("--hbm", type=int, default=1024)
    ap.add_argument("--host", type=int, default=1024)
    ap.add_argument("--seed", type=int, default=1)
    ap.add_argument("--timed", action="store_true", help="order the calls by an event clock with tool waits (trace_c3_timed)")
    ap.add_argument("--long-wait-p", type=float, default=0.0, help="with --timed: share of tool waits of 30-120 s")
    ap.add_argument("--remote", type=int, default=0, help="adds a row for the paper's policy with a third tier of this many blocks")
    a = ap.parse_args()
    from . import binding as B
    if a.timed:
        trace, n_ctx = W.trace_c3_timed(a.seed, n_sessions=a.sessions, scale=a.scale, long_wait_p=a.long_wait_p)
    else:
        trace, n_ctx = W.trace_c3(a.seed, n_sessions=a.sessions, scale=a.scale)
    print(f"C3-shaped trace{' with an event clock' if a.timed else ''}: {a.sessions} sessions, scale {a.scale}, HBM {a.hbm} blocks, host tier {a.host} blocks, "
          f"metadata-only engines on the GPU")
    print("| policy | hit ratio | zombie share mean / peak | wrong-direction evictions | judged | offloaded | dropped |")
    print("|---|---:|---:|---:|---:|---:|---:|")
    rows = [(name, order, flags, 0) for name, (order, flags) in POLICIES.items()]
    if a.remote:
        rows.append((f"lifecycle + MRU, third tier of {a.remote} blocks", 0, 0, a.remote))
    for name, order, flags, n_remote in rows:
        eng = B.Engine(n_hbm_blocks=a.hbm, n_host_blocks=a.host, n_remote_blocks=n_remote, max_contexts=n_ctx,
                       metadata_only=True, suspended_order=order, policy_flags=flags, max_tokens=1 << 22,
                       max_messages=1 << 15, **W.GEO_GLM.kwargs())
        m = replay_metrics(eng, trace)
        print(f"| {name} | {m['hit_ratio']:.3f} | {m['zombie_share_mean']:.3f} / {m['zombie_share_peak']:.3f} | "
              f"{m['wrong_direction_ratio']:.3f} | {m['evictions_judged']} | {m['offloaded']} | {m['dropped']} |")
        eng.close()


if __name__ == "__main__":
    main()
