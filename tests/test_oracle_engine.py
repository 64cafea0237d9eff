"""Pins of the CPU oracle's engine semantics: the paper's state-machine sentences, the shared-KV
example, Algorithm 1's order, brute force on tiny pools, round trips and global invariants."""
import numpy as np
import pytest

import scenarios as S
from paper_2609_39819_b200 import workloads as W


@pytest.fixture
def make(oracle):
    return lambda **kw: oracle.OracleEngine(**kw)


@pytest.mark.parametrize("scenario", S.ALL, ids=lambda f: f.__name__)
def test_scenario(make, scenario):
    scenario(make)


def test_pinned_competes_only_with_pinned(make):
    S.pinned_competes_only_with_pinned(make, W.run_call, lambda: W.ReplayOptions(payload=None, record_states=False))


def test_mixed_pool_lru_switch(make):
    S.mixed_pool_example(make, order=1)


def test_error_codes(make, oracle):
    ops = {k[3:]: getattr(oracle, k) for k in dir(oracle) if k.startswith("OP_")}
    S.error_codes(make, ops)


def check_invariants(eng):
    """Global invariants that hold after every call whatever the trace."""
    st = eng.get_stats()
    keys_all = []
    for tier, n in ((0, eng.n_hbm_blocks), (1, eng.n_host_blocks)):
        ent = eng.get_entries(tier)
        occ = int((ent["key"] != 0).sum())
        assert occ == st["occ_hbm" if tier == 0 else "occ_host"] <= n      # occupancy never exceeds capacity
        keys_all.append(ent["key"][ent["key"] != 0])
        states = eng.get_states(tier)
        assert np.all((states == 0xFF) == (ent["key"] == 0))
        assert np.all(ent["inflight"][ent["key"] == 0] == 0)
    keys_all = np.concatenate(keys_all)
    assert len(np.unique(keys_all)) == len(keys_all)                        # each key in exactly one (tier, slot)
    assert st["hits_hbm"] + st["hits_host"] + st["misses"] == st["blocks_hashed"]
    assert st["inserted"] - st["dropped"] == st["occ_hbm"] + st["occ_host"]


@pytest.mark.parametrize("seed", [0, 1, 2, 3, 4, 5, 7, 39, 63, 86, 102, 120])
def test_c1_replay_invariants_and_bruteforce_states(make, seed):
    eng = make(n_hbm_blocks=128, n_host_blocks=512, max_contexts=64, **W.GEO_TOY.kwargs())
    opt = W.ReplayOptions(payload=W.payload_normal_bf16, verify_payload_every=1)
    for _i, kind, rec in W.replay(eng, W.trace_c1(seed), opt):
        if kind != "call":
            continue
        assert rec["payload_ok"]
        check_invariants(eng)
        # classification equals the literal double loop over blocks x mappings
        for tier in (0, 1):
            assert np.array_equal(eng.get_states(tier), eng.classify_bruteforce(tier))
        # no victim is in flight; victims come in Algorithm 1's order
        if "vstates" in rec:
            assert np.all(np.diff(rec["vstates"].astype(int)) >= 0)
        assert int(eng.get_entries(0)["inflight"].sum() + eng.get_entries(1)["inflight"].sum()) == 0


def test_c1_pool_is_under_pressure():
    """The tiny configuration must actually exercise eviction, offload and reload."""
    from oracle import kvt_oracle
    tot = {"offloaded": 0, "reloaded": 0, "dropped": 0, "adopted": 0}
    for seed in (7, 39, 63, 86, 120):
        eng = kvt_oracle.OracleEngine(n_hbm_blocks=128, n_host_blocks=512, max_contexts=64, **W.GEO_TOY.kwargs())
        for _ in W.replay(eng, W.trace_c1(seed), W.ReplayOptions(payload=None, record_states=False)):
            pass
        st = eng.get_stats()
        for k in tot:
            tot[k] += st[k]
    assert tot["offloaded"] > 0 and tot["reloaded"] > 0 and tot["dropped"] > 0, tot


def test_scaled_c2_and_c3_traces_replay(make):
    eng = make(n_hbm_blocks=96, n_host_blocks=64, max_contexts=64, **W.GEO_TOY.kwargs())
    n_calls = 0
    for _i, kind, rec in W.replay(eng, W.trace_c2(1, scale=1 / 32), W.ReplayOptions(payload=W.payload_pattern, verify_payload_every=5)):
        n_calls += kind == "call"
    check_invariants(eng)
    assert n_calls > 20 and W.verify_payload(eng, W.payload_pattern)
    st = eng.get_stats()
    assert st["dropped"] > 0      # a single session only ever evicts its own dead suffixes
    trace, n_ctx = W.trace_c3(1, n_sessions=6, scale=1 / 64)
    eng = make(n_hbm_blocks=256, n_host_blocks=256, max_contexts=n_ctx, **W.GEO_TOY.kwargs())
    for _i, kind, rec in W.replay(eng, trace, W.ReplayOptions(payload=None, record_states=False)):
        pass
    check_invariants(eng)
    # sessions 0 and 4 pinned their system prompt: they outlive their termination until it is unpinned
    assert eng.get_stats()["n_contexts"] == 2 and int((eng.get_states(0) == 3).sum() + (eng.get_states(1) == 3).sum()) > 0
    eng.unpin(0, 0, 1)
    eng.unpin(4, 0, 1)
    assert eng.get_stats()["n_contexts"] == 0
    assert int((eng.get_states(0) == 3).sum() + (eng.get_states(1) == 3).sum()) == 0


@pytest.mark.parametrize("flags", [0, 2])
def test_replay_with_exchange_moves_the_same_blocks(make, flags):
    """The driver's exchange mode (reloads and the offloads that make room for them in one call) is, by definition,
    offload followed by reload: the same blocks end up in the same slots with the same metadata as with the two
    separate calls, and every payload byte survives."""
    trace, n_ctx = W.trace_c3(1, n_sessions=8, scale=1 / 32)
    out = []
    for use in (False, True):
        eng = make(n_hbm_blocks=256, n_host_blocks=320, max_contexts=n_ctx, policy_flags=flags, **W.GEO_TOY.kwargs())
        opt = W.ReplayOptions(payload=W.payload_pattern, record_states=False, verify_payload_every=9, use_exchange=use)
        n_x = 0
        for _i, kind, rec in W.replay(eng, trace, opt):
            if kind == "call":
                n_x += "exchange" in rec
                assert rec.get("payload_ok", True)
        check_invariants(eng) if not flags else None
        assert W.verify_payload(eng, W.payload_pattern)
        st = eng.get_stats()
        ent = [eng.get_entries(t) for t in (0, 1)]
        out.append((n_x, st, ent))
    assert out[0][0] == 0 and out[1][0] > 0
    assert out[0][1] == out[1][1]
    for t in (0, 1):
        for k in out[0][2][t]:
            assert np.array_equal(out[0][2][t][k], out[1][2][t][k]), (t, k)


@pytest.mark.parametrize("flags", [0, 2])
def test_replay_with_a_remote_tier_keeps_more_blocks_reusable(make, flags):
    """C3-shaped trace with a small host tier: without a third tier the host tier's victims are lost, with one
    they move down and come back when their session calls again: more prefix hits, fewer dropped live blocks,
    every payload byte intact on all three tiers."""
    trace, n_ctx = W.trace_c3(1, n_sessions=8, scale=1 / 32)
    res = {}
    for n_remote in (0, 512):
        eng = make(n_hbm_blocks=256, n_host_blocks=96, n_remote_blocks=n_remote, max_contexts=n_ctx, policy_flags=flags,
                   **W.GEO_TOY.kwargs())
        opt = W.ReplayOptions(payload=W.payload_pattern, record_states=False, verify_payload_every=9)
        for _i, kind, rec in W.replay(eng, trace, opt):
            if kind == "call":
                assert rec.get("payload_ok", True)
        assert W.verify_payload(eng, W.payload_pattern)
        res[n_remote] = eng.get_stats()
    a, b = res[0], res[512]
    assert b["demoted"] > 0 and b["promoted"] > 0 and b["hits_remote"] > 0
    assert b["hits_hbm"] + b["hits_host"] + b["hits_remote"] > a["hits_hbm"] + a["hits_host"]
    assert b["dropped"] < a["dropped"]


def test_timed_trace_shows_the_recency_direction(make):
    """C3 with an event clock and tool waits of 1-6 s (Section 6.2's premise: what was suspended last comes back
    last): evicting the most recently suspended blocks first keeps more reusable KV than LRU does; with a tail of
    very long waits the order turns around (the stragglers are what LRU evicts)."""
    from paper_2609_39819_b200 import policy_metrics as PM
    res = {}
    for lw in (0.0, 0.1):
        trace, n_ctx = W.trace_c3_timed(1, n_sessions=16, scale=1 / 32, long_wait_p=lw)
        for order in (0, 1):
            eng = make(n_hbm_blocks=400, n_host_blocks=400, max_contexts=n_ctx, suspended_order=order, metadata_only=True,
                       **W.GEO_TOY.kwargs())
            res[lw, order] = PM.replay_metrics(eng, trace)
            check_invariants(eng)
    assert res[0.0, 0]["hit_ratio"] > res[0.0, 1]["hit_ratio"] + 0.05 and res[0.0, 0]["dropped"] < res[0.0, 1]["dropped"]
    assert res[0.1, 1]["hit_ratio"] > res[0.1, 0]["hit_ratio"]


def test_incremental_appends_hash_like_one_shot(make, oracle):
    """Hashing a context after piecewise appends equals hashing the concatenation in one shot."""
    rng = np.random.default_rng(21)
    eng = make(n_hbm_blocks=64, n_host_blocks=8, max_contexts=4, **S.TOY)
    eng.spawn(0)
    parts = []
    for n in (5, 27, 16, 1, 100, 63):
        parts.append(S.toks(rng, n))
        eng.append(0, parts[-1])
        S.call(eng, 0)
        assert np.array_equal(eng.get_block_map(0)[0], oracle.hash_tokens(np.concatenate(parts)))


def test_kv_size_sanity():
    """Section 1 quotes 93 GB of KV for a 258K-token request; the GLM-scale geometry used here gives
    a figure of the same size (within 5%)."""
    bytes_per_token = W.GEO_GLM.block_bytes // 16
    assert bytes_per_token == 376832
    assert abs(258_000 * bytes_per_token / 1e9 - 93) / 93 < 0.05


def test_policy_metrics_on_a_small_trace(make):
    """Hit ratio, zombie share and wrong-direction ratio are well defined and the ablations behave as
    Section 8.3 describes: without lifecycle tracking zombies pile up and are copied instead of dropped."""
    from paper_2609_39819_b200 import policy_metrics as PM
    trace, n_ctx = W.trace_c3(1, n_sessions=8, scale=1 / 32)
    res = {}
    for name, (order, flags) in PM.POLICIES.items():
        eng = make(n_hbm_blocks=256, n_host_blocks=256, max_contexts=n_ctx, metadata_only=True, suspended_order=order,
                   policy_flags=flags, **W.GEO_TOY.kwargs())
        res[name] = PM.replay_metrics(eng, trace)
        m = res[name]
        assert 0 < m["hit_ratio"] < 1 and 0 <= m["wrong_direction_ratio"] <= 1 and m["zombie_share_peak"] <= 1
    paper, no_lt = res["lifecycle + MRU (paper)"], res["w/o LT (MRU only)"]
    assert no_lt["zombie_share_mean"] > paper["zombie_share_mean"]
    assert no_lt["offloaded"] > paper["offloaded"]
