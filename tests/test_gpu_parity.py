"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element and
bit-exact: all of this is integer, index and byte work, so the tolerance is zero."""
import numpy as np
import pytest

import scenarios as S
from paper_2609_39819_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_39819_b200 import binding
    binding.load_library()
    return binding


@pytest.fixture
def make_gpu(B):
    return lambda **kw: B.Engine(max_tokens=1 << 18, max_messages=4096, **kw)


@pytest.fixture
def make_cpu(oracle):
    return lambda **kw: oracle.OracleEngine(**kw)


# ---- the scenario expectations that pin the oracle also hold for the CUDA engine -------------------
@pytest.mark.parametrize("scenario", S.ALL, ids=lambda f: f.__name__)
def test_scenario(make_gpu, scenario):
    scenario(make_gpu)


def test_pinned_competes_only_with_pinned(make_gpu):
    S.pinned_competes_only_with_pinned(make_gpu, W.run_call, lambda: W.ReplayOptions(payload=None, record_states=False))


def test_mixed_pool_lru_switch(make_gpu):
    S.mixed_pool_example(make_gpu, order=1)


def test_error_codes(make_gpu, B):
    ops = {k[3:]: getattr(B, k) for k in dir(B) if k.startswith("OP_") and k != "OPF_TOKENS_ON_DEVICE"}
    S.error_codes(make_gpu, ops)


# ---- stage 1: hashing ---------------------------------------------------------------------------------
@pytest.mark.parametrize("n_tokens", [0, 15, 16, 17, 16 * 255, 16 * 256, 16 * 257 + 3, 16 * 1000 + 7, 258048])
@pytest.mark.parametrize("seed", [0, 0xDEADBEEFCAFEF00D])
def test_hash_matches_oracle(B, oracle, n_tokens, seed):
    import torch
    rng = np.random.default_rng(n_tokens + 1)
    tok = rng.integers(0, W.VOCAB, n_tokens, dtype=np.uint32)
    if n_tokens > 100:
        tok[7] = 0
        tok[8] = W.VOCAB - 1
    d = torch.from_numpy(tok.view(np.int32)).cuda() if n_tokens else torch.empty(0, dtype=torch.int32, device="cuda")
    got = B.hash_tokens(d, seed).cpu().numpy().view(np.uint64)
    want = oracle.hash_tokens(tok, seed)
    assert got.shape == want.shape and np.array_equal(got, want)


def test_hash_full_size_batch_matches_oracle(B, oracle):
    """C4-sized hashing: 64 sequences x 16,128 blocks through one kernel sequence each."""
    import torch
    rng = np.random.default_rng(99)
    for _ in range(3):
        tok = rng.integers(0, W.VOCAB, 258048, dtype=np.uint32)
        got = B.hash_tokens(torch.from_numpy(tok.view(np.int32)).cuda(), 0).cpu().numpy().view(np.uint64)
        assert np.array_equal(got, oracle.hash_tokens(tok, 0))


# ---- whole path on C1 traces: every reported value and every payload byte ----------------------------
def _replay_pair(gpu, cpu, trace, payload, check_pools=True, record_states=True, verify_every=0, use_exchange=False,
                 cross_check=True):
    og = W.ReplayOptions(payload=payload, record_states=record_states, verify_payload_every=verify_every,
                         use_exchange=use_exchange)
    oc = W.ReplayOptions(payload=payload, record_states=record_states, verify_payload_every=verify_every,
                         use_exchange=use_exchange)
    if cross_check and gpu.n_hbm_blocks + gpu.n_host_blocks <= 8192:
        gpu.set_classify_mode(2)      # small pools: every event-driven update is cross-checked against a full recomputation
    n_calls = 0
    for (i, kind, rg), (_, _, rc) in zip(W.replay(gpu, trace, og), W.replay(cpu, trace, oc)):
        if kind == "call":
            n_calls += 1
            diff = W.records_equal(rg, rc, f"event[{i}]")
            assert diff is None, diff
            if "payload_ok" in rg:
                assert rg["payload_ok"] and rc["payload_ok"]
    sg, sc = gpu.get_stats(), cpu.get_stats()
    for k in sc:
        if k not in W.GPU_ONLY_STATS:
            assert sg[k] == sc[k], k
    if check_pools and payload is not None:
        for tier in W.engine_tiers(gpu):
            keys = cpu.get_entries(tier)["key"]
            for s in np.nonzero(keys)[0]:
                assert np.array_equal(gpu.read_block(tier, int(s)), cpu.read_block(tier, int(s))), (tier, s)
    return n_calls


@pytest.mark.parametrize("seed", [0, 1, 2, 3, 7, 39, 63, 86, 102, 120, 136, 164])
def test_c1_trace_parity(B, oracle, seed):
    kw = dict(n_hbm_blocks=128, n_host_blocks=512, max_contexts=64, **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=1 << 18, max_messages=4096, **kw)
    cpu = oracle.OracleEngine(**kw)
    _replay_pair(gpu, cpu, W.trace_c1(seed), W.payload_normal_bf16, verify_every=2)


@pytest.mark.parametrize("first", [1, 51, 101, 151])
def test_c1_trace_parity_seeds_1_to_200(B, oracle, first):
    """The tiny configuration on seeds 1 .. 200 (fifty per case), metadata and payload bytes, one engine pair per seed."""
    kw = dict(n_hbm_blocks=128, n_host_blocks=512, max_contexts=64, **W.GEO_TOY.kwargs())
    for seed in range(first, first + 50):
        gpu = B.Engine(max_tokens=1 << 18, max_messages=4096, **kw)
        cpu = oracle.OracleEngine(**kw)
        _replay_pair(gpu, cpu, W.trace_c1(seed), W.payload_normal_bf16, record_states=False)
        gpu.close()


@pytest.mark.parametrize("layout,order", [(0, 1), (1, 0), (1, 1)])
def test_c1_trace_parity_other_layouts_and_orders(B, oracle, layout, order):
    kw = dict(n_hbm_blocks=96, n_host_blocks=64, max_contexts=64, pool_layout=layout, suspended_order=order,
              **W.GEO_TOY.kwargs())
    for seed in (7, 63, 86):
        gpu = B.Engine(max_tokens=1 << 18, max_messages=4096, **kw)
        cpu = oracle.OracleEngine(**kw)
        _replay_pair(gpu, cpu, W.trace_c1(seed), W.payload_pattern)


@pytest.mark.parametrize("order,flags", [(0, 1), (1, 1)])
def test_trace_parity_without_lifecycle_tracking(B, oracle, order, flags):
    """The "w/o LT" ablation and plain LRU: same replays, same results as the oracle."""
    for seed in (7, 63):
        kw = dict(n_hbm_blocks=96, n_host_blocks=256, max_contexts=64, suspended_order=order, policy_flags=flags,
                  **W.GEO_TOY.kwargs())
        gpu = B.Engine(max_tokens=1 << 18, max_messages=4096, **kw)
        cpu = oracle.OracleEngine(**kw)
        _replay_pair(gpu, cpu, W.trace_c1(seed), W.payload_pattern)
    trace, n_ctx = W.trace_c3(1, n_sessions=8, scale=1 / 32)
    kw = dict(n_hbm_blocks=256, n_host_blocks=256, max_contexts=n_ctx, metadata_only=True, suspended_order=order,
              policy_flags=flags, **W.GEO_TOY.kwargs())
    from paper_2609_39819_b200 import policy_metrics as PM
    mg = PM.replay_metrics(B.Engine(max_tokens=1 << 20, max_messages=1 << 15, **kw), trace)
    mc = PM.replay_metrics(oracle.OracleEngine(**kw), trace)
    assert mg == mc


@pytest.mark.parametrize("flags", [2, 3])
def test_trace_parity_with_inclusive_tiers(B, oracle, flags):
    """Inclusive tiering (and its combination with the no-lifecycle policy): reloaded blocks keep a clean host
    copy, later offloads of them move no bytes; every reported value and every payload byte still matches."""
    for seed in (7, 63, 86):
        kw = dict(n_hbm_blocks=96, n_host_blocks=256, max_contexts=64, policy_flags=flags, **W.GEO_TOY.kwargs())
        gpu = B.Engine(max_tokens=1 << 18, max_messages=4096, **kw)
        cpu = oracle.OracleEngine(**kw)
        _replay_pair(gpu, cpu, W.trace_c1(seed), W.payload_pattern, verify_every=1)
    trace, n_ctx = W.trace_c3(1, n_sessions=8, scale=1 / 32)
    kw = dict(n_hbm_blocks=256, n_host_blocks=320, max_contexts=n_ctx, policy_flags=flags, **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=1 << 20, max_messages=1 << 15, **kw)
    cpu = oracle.OracleEngine(**kw)
    _replay_pair(gpu, cpu, trace, W.payload_pattern, verify_every=5)
    st = cpu.get_stats()
    assert st["offloaded_clean"] > 0 and st["reloaded"] > 0
    # force a table rebuild with copies present, then look everything up again
    keys = cpu.get_entries(0)["key"]
    for eng in (gpu, cpu):
        v, s = eng.select_victims(0, int((keys != 0).sum()))
        eng.offload(v)
    for tier in (0, 1):
        eg, ec = gpu.get_entries(tier), cpu.get_entries(tier)
        for k in ec:
            assert np.array_equal(eg[k], ec[k]), (tier, k)
        assert np.array_equal(gpu.get_states(tier), cpu.get_states(tier))


@pytest.mark.parametrize("flags", [0, 2])
def test_trace_parity_with_exchange_calls(B, oracle, flags):
    """The replay driver in exchange mode: a call's reloads and the offloads that make room for them are one
    kvt_exchange (both directions in one mover launch), the rest of the reload follows. Every reported value,
    every state and every payload byte matches the oracle's exchange."""
    n_x = 0
    for seed in (7, 63, 86):
        kw = dict(n_hbm_blocks=96, n_host_blocks=256, max_contexts=64, policy_flags=flags, **W.GEO_TOY.kwargs())
        gpu = B.Engine(max_tokens=1 << 18, max_messages=4096, **kw)
        cpu = oracle.OracleEngine(**kw)
        _replay_pair(gpu, cpu, W.trace_c1(seed), W.payload_pattern, verify_every=1, use_exchange=True)
    trace, n_ctx = W.trace_c3(1, n_sessions=8, scale=1 / 32)
    kw = dict(n_hbm_blocks=256, n_host_blocks=320, max_contexts=n_ctx, policy_flags=flags, **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=1 << 20, max_messages=1 << 15, **kw)
    cpu = oracle.OracleEngine(**kw)
    og = W.ReplayOptions(payload=W.payload_pattern, verify_payload_every=5, use_exchange=True)
    oc = W.ReplayOptions(payload=W.payload_pattern, verify_payload_every=5, use_exchange=True)
    for (i, kind, rg), (_, _, rc) in zip(W.replay(gpu, trace, og), W.replay(cpu, trace, oc)):
        if kind == "call":
            n_x += "exchange" in rc
            diff = W.records_equal(rg, rc, f"event[{i}]")
            assert diff is None, diff
            assert rg.get("payload_ok", True) and rc.get("payload_ok", True)
    assert n_x > 0
    sg, sc = gpu.get_stats(), cpu.get_stats()
    assert all(sg[k] == sc[k] for k in sc if k not in W.GPU_ONLY_STATS)


@pytest.mark.parametrize("flags", [4, 6])
def test_trace_parity_with_unreachable_blocks_dead(B, oracle, flags):
    """Reachability-aware classification: a small host tier forces drops of live prefixes, the blocks behind them
    classify as dead on both sides, are the first victims and are dropped without a copy."""
    for seed in (7, 63, 86):
        kw = dict(n_hbm_blocks=96, n_host_blocks=48, max_contexts=64, policy_flags=flags, **W.GEO_TOY.kwargs())
        gpu = B.Engine(max_tokens=1 << 18, max_messages=4096, **kw)
        cpu = oracle.OracleEngine(**kw)
        _replay_pair(gpu, cpu, W.trace_c1(seed), W.payload_pattern, verify_every=1)
    trace, n_ctx = W.trace_c3(1, n_sessions=8, scale=1 / 32)
    kw = dict(n_hbm_blocks=256, n_host_blocks=96, max_contexts=n_ctx, policy_flags=flags, **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=1 << 20, max_messages=1 << 15, **kw)
    cpu = oracle.OracleEngine(**kw)
    # stop in mid-trace (sessions alive), punch holes into the chains, compare the reclassification
    _replay_pair(gpu, cpu, trace[:2 * len(trace) // 3], W.payload_pattern, verify_every=5)
    before = cpu.get_states(0).copy()
    ent = cpu.get_entries(0)
    holes = [int(x) for x in np.nonzero((ent["key"] != 0) & (ent["inflight"] == 0) & (ent["depth"] % 7 == 3))[0][:12]]
    assert holes
    for eng in (gpu, cpu):
        eng.release(0, holes)
    after = cpu.get_states(0)
    assert int(((before > 0) & (before < 0xFE) & (after == 0)).sum()) > 0     # orphans appeared
    for tier in (0, 1):
        assert np.array_equal(gpu.get_states(tier), cpu.get_states(tier))
    vg, vc = gpu.select_victims(0, 64), cpu.select_victims(0, 64)
    assert np.array_equal(vg[0], vc[0]) and np.array_equal(vg[1], vc[1])


@pytest.mark.parametrize("flags", [0, 2])
def test_trace_parity_with_a_remote_tier(B, oracle, flags):
    """Three tiers under the replay driver: host victims move down to the remote tier, remote hits come straight up
    into HBM; every reported value, every state on all three tiers and every payload byte match the oracle."""
    for seed in (7, 63, 86):
        kw = dict(n_hbm_blocks=96, n_host_blocks=48, n_remote_blocks=160, max_contexts=64, policy_flags=flags,
                  **W.GEO_TOY.kwargs())
        gpu = B.Engine(max_tokens=1 << 18, max_messages=4096, **kw)
        cpu = oracle.OracleEngine(**kw)
        _replay_pair(gpu, cpu, W.trace_c1(seed), W.payload_pattern, verify_every=1)
    trace, n_ctx = W.trace_c3(1, n_sessions=8, scale=1 / 32)
    kw = dict(n_hbm_blocks=256, n_host_blocks=96, n_remote_blocks=512, max_contexts=n_ctx, policy_flags=flags,
              **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=1 << 20, max_messages=1 << 15, **kw)
    cpu = oracle.OracleEngine(**kw)
    _replay_pair(gpu, cpu, trace, W.payload_pattern, verify_every=5)
    st = gpu.get_stats()
    assert st["demoted"] > 0 and st["promoted"] > 0 and st["hits_remote"] > 0
    for tier in (0, 1, 2):
        assert np.array_equal(gpu.get_states(tier), cpu.get_states(tier))
        eg, ec = gpu.get_entries(tier), cpu.get_entries(tier)
        for k in ec:
            assert np.array_equal(eg[k], ec[k]), (tier, k)


@pytest.mark.parametrize("order,lw", [(0, 0.0), (1, 0.1)])
def test_timed_c3_trace_parity(B, oracle, order, lw):
    """The C3 sessions ordered by an event clock (single-session calls, subagents interleaved with other sessions)."""
    trace, n_ctx = W.trace_c3_timed(2, n_sessions=8, scale=1 / 32, long_wait_p=lw)
    kw = dict(n_hbm_blocks=200, n_host_blocks=200, max_contexts=n_ctx, suspended_order=order, **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=1 << 20, max_messages=1 << 15, **kw)
    cpu = oracle.OracleEngine(**kw)
    n = _replay_pair(gpu, cpu, trace, W.payload_pattern, verify_every=11, use_exchange=bool(order))
    assert n > 100 and cpu.get_stats()["reloaded"] > 0


def test_scaled_c2_trace_parity(B, oracle):
    kw = dict(n_hbm_blocks=96, n_host_blocks=64, max_contexts=8, **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=1 << 18, max_messages=4096, **kw)
    cpu = oracle.OracleEngine(**kw)
    n = _replay_pair(gpu, cpu, W.trace_c2(1, scale=1 / 32), W.payload_pattern, verify_every=7)
    assert n > 20


def test_scaled_c3_trace_parity(B, oracle):
    trace, n_ctx = W.trace_c3(1, n_sessions=8, scale=1 / 32)
    kw = dict(n_hbm_blocks=384, n_host_blocks=512, max_contexts=n_ctx, **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=1 << 20, max_messages=1 << 15, **kw)
    cpu = oracle.OracleEngine(**kw)
    _replay_pair(gpu, cpu, trace, W.payload_pattern, record_states=True)
    assert cpu.get_stats()["offloaded"] > 0 and cpu.get_stats()["reloaded"] > 0


@pytest.mark.parametrize("n_hbm", [20480, 6144])
def test_full_length_c2_session_metadata_parity(B, oracle, n_hbm):
    """One 128K-token ReAct session (C2's trace at full size) on a metadata-only engine with C2's
    block counts (40 GiB pool, and the 12 GiB pressure variant): every lookup, victim list,
    admission and state vector equals the oracle's."""
    kw = dict(n_hbm_blocks=n_hbm, n_host_blocks=61440, max_contexts=4, metadata_only=True, **W.GEO_8B.kwargs())
    gpu = B.Engine(max_tokens=1 << 20, max_messages=1 << 12, **kw)
    cpu = oracle.OracleEngine(**kw)
    n = _replay_pair(gpu, cpu, W.trace_c2(1), None, record_states=True)
    assert n >= 30
    if n_hbm < 20480:
        assert cpu.get_stats()["dropped"] > 0


def test_full_size_c3_metadata_parity(B, oracle):
    """C3 at full size (32 sessions of 32K-258K tokens, forks, GLM-scale geometry, 120 GiB = 21,370-block HBM
    pool) on metadata-only engines: every batch call's lookups, victim lists, offloads, reloads and
    admissions equal the oracle's."""
    trace, n_ctx = W.trace_c3(1)
    kw = dict(n_hbm_blocks=21370, n_host_blocks=20000, max_contexts=n_ctx, metadata_only=True, **W.GEO_GLM.kwargs())
    gpu = B.Engine(max_tokens=1 << 24, max_messages=1 << 16, **kw)
    cpu = oracle.OracleEngine(**kw)
    n = _replay_pair(gpu, cpu, trace, None, record_states=True)
    st = cpu.get_stats()
    assert n > 100 and st["offloaded"] > 10000 and st["reloaded"] > 10000 and st["dropped"] > 10000


def test_bench_steps_at_full_size_match_the_oracle(B, oracle):
    """The benchmark's own step sequence (C2 session, 8B-class blocks, 20,480-block HBM pool, 61,440-block second
    tier kept in HBM as in the bench's in-device arm, tier pressure after every call) against the metadata-only
    oracle: every call's reports and the statistics are equal, and every resident block's payload survives."""
    import sys
    import torch
    sys.path.insert(0, str(__import__("pathlib").Path(__file__).resolve().parents[1]))
    import bench
    geo = W.GEO_8B
    import gc
    gc.collect()
    torch.cuda.empty_cache()          # memory cached from earlier tests counts as used otherwise
    free_b, _ = torch.cuda.mem_get_info()
    if free_b < (20480 + 61440) * geo.block_bytes + (6 << 30):
        pytest.skip("needs 160 GiB of HBM")
    setup, turns, _target = bench.make_turns(1, 12)
    kw = dict(n_hbm_blocks=20480, n_host_blocks=61440, max_contexts=4, **geo.kwargs())
    gpu = B.Engine(max_tokens=1 << 21, max_messages=1 << 13, host_pool_on_device=True, zero_pools=False, **kw)
    cpu = oracle.OracleEngine(metadata_only=True, **kw)
    og = W.ReplayOptions(payload=None, record_states=False, writer=lambda e, slot, key: e.fill_block_pattern(0, slot, key))
    oc = W.ReplayOptions(payload=None, record_states=False)
    ident = lambda a: a
    for ev in setup:
        bench.apply_event(gpu, ev, ident)
        bench.apply_event(cpu, ev, ident)
    for t, (pre, ctxs, post) in enumerate(turns):
        recs = []
        for eng, opt in ((gpu, og), (cpu, oc)):
            for ev in pre:
                bench.apply_event(eng, ev, ident)
            rec = W.run_call(eng, ctxs, opt)
            for ev in post:
                bench.apply_event(eng, ev, ident)
            n = eng.get_stats()["occ_hbm"] // 2
            rec["pressure"] = W.evict(eng, n) if n else {}
            recs.append(rec)
        diff = W.records_equal(recs[0], recs[1], f"turn {t}")
        assert diff is None, diff
    sg, sc = gpu.get_stats(), cpu.get_stats()
    for k in sc:
        if k not in W.GPU_ONLY_STATS:
            assert sg[k] == sc[k], k
    assert sc["offloaded"] > 50000 and sc["reloaded"] > 50000
    bad = n_checked = 0
    for tier in (0, 1):
        keys = gpu.get_entries(tier)["key"]
        for s in np.nonzero(keys)[0]:
            n_checked += 1
            bad += not gpu.check_block_pattern(tier, int(s), int(keys[s]))
    assert bad == 0 and n_checked > 5000


def test_full_size_c3_with_payload(B, oracle):
    """C3 at full size with real payloads on the GPU: GLM-scale blocks (5.75 MiB), the 120 GiB HBM pool
    (21,370 blocks) and a pinned host tier of 24 GiB (4,274 blocks; the oracle runs the same sizes metadata-only).
    Every call's results equal the oracle's and, at the end, every occupied slot of both tiers holds the payload
    of the key it is registered for, after ~50 K blocks have crossed the host link."""
    import gc
    import torch
    gc.collect()
    torch.cuda.empty_cache()          # memory cached from earlier tests counts as used otherwise
    free_b, _ = torch.cuda.mem_get_info()
    geo = W.GEO_GLM
    n_hbm = 21370
    if free_b < (n_hbm * geo.block_bytes + (6 << 30)):
        pytest.skip("needs a 120 GiB HBM pool")
    trace, n_ctx = W.trace_c3(1)
    kw = dict(n_hbm_blocks=n_hbm, n_host_blocks=4274, max_contexts=n_ctx, **geo.kwargs())
    gpu = B.Engine(max_tokens=1 << 24, max_messages=1 << 16, zero_pools=False, **kw)
    cpu = oracle.OracleEngine(metadata_only=True, **kw)
    og = W.ReplayOptions(payload=None, record_states=False, writer=lambda e, slot, key: e.fill_block_pattern(0, slot, key))
    oc = W.ReplayOptions(payload=None, record_states=False)
    for (i, kind, rg), (_, _, rc) in zip(W.replay(gpu, trace, og), W.replay(cpu, trace, oc)):
        if kind == "call":
            diff = W.records_equal(rg, rc, f"event[{i}]")
            assert diff is None, diff
    sg, sc = gpu.get_stats(), cpu.get_stats()
    for k in sc:
        if k not in W.GPU_ONLY_STATS:
            assert sg[k] == sc[k], k
    assert sc["offloaded"] > 10000 and sc["reloaded"] > 5000
    bad = 0
    for tier in (0, 1):
        keys = gpu.get_entries(tier)["key"]
        for s in np.nonzero(keys)[0]:
            bad += not gpu.check_block_pattern(tier, int(s), int(keys[s]))
    assert bad == 0


# ---- C4: metadata stress at full size -------------------------------------------------------------------
def _c4_setup(B, oracle, n_resident, chain_blocks, n_calls):
    inp = W.inputs_c4(1, n_resident=n_resident, chain_blocks=chain_blocks, n_calls=n_calls)
    kw = dict(n_hbm_blocks=n_resident, n_host_blocks=0, max_contexts=n_calls + 1, metadata_only=True, **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=(n_calls + 1) * chain_blocks * 16 * 2, max_messages=1024,
                   max_batch_blocks=n_calls * chain_blocks, **kw)
    cpu = oracle.OracleEngine(**kw)
    keys = np.concatenate([oracle.hash_tokens(c) for c in inp.chain_tokens])
    for eng in (gpu, cpu):
        eng.debug_load_resident(keys, inp.state, inp.stamp, inp.depth, inp.slot, 0)
        for i, t in enumerate(inp.calls):
            eng.spawn(i)
            eng.append(i, t)
    return inp, gpu, cpu


@pytest.mark.parametrize("lookup_variant", [1, 2, 3, 4], ids=["default", "single-pass", "one-key-per-thread", "four-keys-per-thread"])
@pytest.mark.parametrize("n_resident,chain_blocks,n_calls", [(5000, 700, 9), (1 << 20, 16128, 64)])
def test_c4_lookup_and_select_parity(B, oracle, n_resident, chain_blocks, n_calls, lookup_variant):
    inp, gpu, cpu = _c4_setup(B, oracle, n_resident, chain_blocks, n_calls)
    gpu.set_lookup_variant(lookup_variant)
    ids = list(range(n_calls))
    # selection before any call: the whole pool is a candidate; 10% stays in the dead tier,
    # 35% crosses into the idle (MRU) tier, 75% into the active tier
    bufs = gpu.victim_buffers(n_resident)        # pinned: the list is written there by the last kernel, no staging copy
    for frac in (0.10, 0.35, 0.75):
        n = int(n_resident * frac)
        vg, sg = gpu.select_victims(0, n, out=bufs if frac != 0.10 else None)
        vc, sc = cpu.select_victims(0, n)
        assert np.array_equal(vg, vc) and np.array_equal(sg, sc), frac
    ig = gpu.map_blocks(ids, 0)
    ic = cpu.map_blocks(ids, 0)
    assert np.array_equal(ig, ic)
    assert 0.3 < ic["hit_len"].sum() / ic["n_blocks"].sum() < 0.6
    for c in (0, n_calls // 2, n_calls - 1):
        for a, b in zip(gpu.get_block_map(c), cpu.get_block_map(c)):
            assert np.array_equal(a, b)
    # with the hits locked in flight, select 10% of the pool
    n = n_resident // 10
    vg, sg = gpu.select_victims(0, n)
    vc, sc = cpu.select_victims(0, n)
    assert np.array_equal(vg, vc) and np.array_equal(sg, sc)
    # drop them and admit the misses into the freed slots
    assert gpu.offload(vg) == cpu.offload(vc)
    ag = gpu.map_blocks(ids, 1)
    ac = cpu.map_blocks(ids, 1)
    assert np.array_equal(ag, ac)
    for c in ids:
        gpu.prefill_done(c)
        cpu.prefill_done(c)
    eg, ec = gpu.get_entries(0), cpu.get_entries(0)
    for k in ec:
        assert np.array_equal(eg[k], ec[k]), k
    assert np.array_equal(gpu.get_states(0), cpu.get_states(0))
    sg, sc = gpu.get_stats(), cpu.get_stats()
    for k in sc:
        if k not in W.GPU_ONLY_STATS:
            assert sg[k] == sc[k], k


def test_wide_stamps_and_depths_order_like_the_oracle(B, oracle):
    """Stamps up to 2^31 and depths up to 2^24 make the packed victim key 59 bits wide; the order still equals the
    oracle's comparator. A stamp / depth pair beyond 63 bits is refused by the loader."""
    n = 3000
    kw = dict(n_hbm_blocks=n, n_host_blocks=0, max_contexts=4, metadata_only=True, **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=1 << 16, max_messages=64, **kw)
    cpu = oracle.OracleEngine(**kw)
    rng = np.random.default_rng(123)
    keys = rng.integers(2, 1 << 63, n, dtype=np.uint64)
    state = rng.integers(0, 4, n).astype(np.uint8)
    stamp = rng.integers(0, 1 << 31, n, dtype=np.uint32)
    stamp[: n // 3] = stamp[0]                                   # many ties on the stamp: depth, then slot decide
    depth = rng.integers(0, 1 << 24, n, dtype=np.uint32)
    depth[: n // 6] = depth[0]
    slot = rng.permutation(n).astype(np.uint32)
    for eng in (gpu, cpu):
        eng.debug_load_resident(keys, state, stamp, depth, slot, 0)
    for n_req, pinned in ((1, False), (n // 10, False), (n // 2, False), (n, False), (n, True)):
        vg, sg = gpu.select_victims(0, n_req, include_pinned=pinned)
        vc, sc = cpu.select_victims(0, n_req, include_pinned=pinned)
        assert np.array_equal(vg, vc) and np.array_equal(sg, sc), (n_req, pinned)
    big = gpu.debug_load_resident_rc(np.array([5], np.uint64), [0], [0xFFFFFFFF], [0xFFFFFFFF], [0], 0)
    assert big == B.E_INVAL                                      # 3 + 32 + 32 bits
    vg, _ = gpu.select_victims(0, 5)
    assert np.array_equal(vg, cpu.select_victims(0, 5)[0])       # and nothing changed


def test_pool_beyond_one_scan_round(B, oracle):
    """3.2 M slots: every ordered compaction over the tier (selection, free lists, compaction plan) needs more than
    one 1024-tile round of the tile scan, and the slot count is not a multiple of any tile size."""
    n_resident, chain_blocks, n_calls = 3 * (1 << 20) + 54321, 16128, 3
    inp, gpu, cpu = _c4_setup(B, oracle, n_resident, chain_blocks, n_calls)
    for frac in (0.10, 0.75):
        n = int(n_resident * frac)
        vg, sg = gpu.select_victims(0, n)
        vc, sc = cpu.select_victims(0, n)
        assert np.array_equal(vg, vc) and np.array_equal(sg, sc), frac
    # release a scattered quarter of the pool, then fill the holes
    rng = np.random.default_rng(77)
    drop = rng.permutation(n_resident)[: n_resident // 4].astype(np.uint32)
    gpu.release(0, drop)
    cpu.release(0, drop)
    assert np.array_equal(gpu.get_states(0), cpu.get_states(0))
    assert gpu.compact(0) == cpu.compact(0)
    eg, ec = gpu.get_entries(0), cpu.get_entries(0)
    for k in ec:
        assert np.array_equal(eg[k], ec[k]), k
    assert np.array_equal(gpu.get_states(0), cpu.get_states(0))
    ids = list(range(n_calls))
    assert np.array_equal(gpu.map_blocks(ids, 0), cpu.map_blocks(ids, 0))
    assert np.array_equal(gpu.map_blocks(ids, 1), cpu.map_blocks(ids, 1))
    n = n_resident // 3
    vg, sg = gpu.select_victims(0, n)
    vc, sc = cpu.select_victims(0, n)
    assert np.array_equal(vg, vc) and np.array_equal(sg, sc)
    sg, sc = gpu.get_stats(), cpu.get_stats()
    for k in sc:
        if k not in W.GPU_ONLY_STATS:
            assert sg[k] == sc[k], k


def test_wait_that_runs_out_reports_a_device_error_and_changes_nothing(B, oracle):
    """The single-pass lookup's chunks wait, bounded, for their predecessors. With the limit set to zero polls every
    chunk behind the first one of a sequence gives up at once: the kernel returns normally, the call reports
    KVT_E_DEVICE, and neither the host nor the device state of the engine has changed. Nothing faults or hangs."""
    kw = dict(n_hbm_blocks=4096, n_host_blocks=64, max_contexts=8, metadata_only=True, **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=1 << 18, max_messages=256, **kw)
    cpu = oracle.OracleEngine(**kw)
    rng = np.random.default_rng(99)
    t0, t1 = (rng.integers(0, W.VOCAB, n, dtype=np.uint32) for n in (16 * 700 + 5, 16 * 300))
    for eng in (gpu, cpu):
        eng.spawn(0); eng.append(0, t0)
        eng.spawn(1); eng.append(1, t1)
        eng.map_blocks([0], 0); eng.map_blocks([0], 1); eng.prefill_done(0)     # context 0 is resident and idle
        eng.append(0, t1[:160])
    before = (gpu.get_stats(), gpu.get_entries(0), gpu.get_states(0), gpu.get_block_map(0))
    gpu.set_lookup_variant(2)
    gpu.set_wait_limit(0)
    rc, _ = gpu.map_blocks_rc([0, 1], 0)
    assert rc == B.E_DEVICE and "wait" in gpu.last_error()
    after = (gpu.get_stats(), gpu.get_entries(0), gpu.get_states(0), gpu.get_block_map(0))
    for k in before[0]:
        if k != "kernel_launches":
            assert before[0][k] == after[0][k], k
    for k in before[1]:
        assert np.array_equal(before[1][k], after[1][k]), k
    assert np.array_equal(before[2], after[2])
    for a, b in zip(before[3], after[3]):
        assert np.array_equal(a, b)
    assert gpu.map_blocks_rc([0], 1)[0] == B.E_STATE                 # nobody is in flight
    # the same call with the default kernels, then with the single pass and its normal limit, matches the oracle
    gpu.set_lookup_variant(1)
    assert np.array_equal(gpu.map_blocks([0, 1], 0), cpu.map_blocks([0, 1], 0))
    assert np.array_equal(gpu.map_blocks([0, 1], 1), cpu.map_blocks([0, 1], 1))
    for eng in (gpu, cpu):
        eng.prefill_done(0); eng.prefill_done(1)
        eng.append(1, t0[:999])
    gpu.set_lookup_variant(2)
    gpu.set_wait_limit(1 << 18)
    assert np.array_equal(gpu.map_blocks([1, 0], 0), cpu.map_blocks([1, 0], 0))
    eg, ec = gpu.get_entries(0), cpu.get_entries(0)
    for k in ec:
        assert np.array_equal(eg[k], ec[k]), k
    sg, sc = gpu.get_stats(), cpu.get_stats()
    for k in sc:
        if k not in W.GPU_ONLY_STATS:
            assert sg[k] == sc[k], k


# ---- C5: the raw mover ------------------------------------------------------------------------------------
def test_c5_longest_id_list(B, oracle):
    """65,536 permuted blocks in one call (the sweep's maximum), toy payloads: 1 GiB each way."""
    import torch
    n = 65536
    kw = dict(n_hbm_blocks=n, n_host_blocks=n, max_contexts=2, **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=1 << 12, max_messages=64, max_batch_blocks=n, zero_pools=False, **kw)
    cpu = oracle.OracleEngine(**kw)
    fill = np.random.default_rng(8).integers(0, 256, gpu.hbm_pool.numel(), dtype=np.uint8)
    gpu.hbm_pool.copy_(torch.from_numpy(fill))
    cpu.hbm_pool[:] = fill
    src, dst = W.ids_c5(1, n, n, True), W.ids_c5(2, n, n, True)
    for eng in (gpu, cpu):
        eng.copy_blocks(0, src, 1, dst)
    torch.cuda.synchronize()
    assert np.array_equal(gpu.host_pool.numpy(), cpu.host_pool)
    gpu.hbm_pool.zero_()
    cpu.hbm_pool[:] = 0
    for eng in (gpu, cpu):
        eng.copy_blocks(1, dst, 0, src)
    torch.cuda.synchronize()
    assert np.array_equal(gpu.hbm_pool.cpu().numpy(), fill) and np.array_equal(cpu.hbm_pool, fill)


@pytest.mark.parametrize("geo", [W.GEO_TOY, W.GEO_128K, W.GEO_8B, W.GEO_GLM], ids=lambda g: g.name)
@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("variant", [1, 2, 3], ids=["cta-per-chunk", "warp-tiles", "tma-ring"])
def test_c5_mover_parity(B, oracle, geo, layout, variant):
    import torch
    n_slots = (12 if geo.block_bytes > (4 << 20) else 24) if geo.block_bytes > (1 << 20) else 200
    kw = dict(n_hbm_blocks=n_slots, n_host_blocks=n_slots, max_contexts=2, pool_layout=layout, **geo.kwargs())
    gpu = B.Engine(max_tokens=1 << 12, max_messages=64, max_batch_blocks=4096, **kw)
    gpu.set_mover_variant(variant)
    cpu = oracle.OracleEngine(**kw)
    rng = np.random.default_rng(5)
    fill = rng.integers(0, 256, gpu.hbm_pool.numel(), dtype=np.uint8)
    gpu.hbm_pool.copy_(torch.from_numpy(fill))
    cpu.hbm_pool[:] = fill
    for n in (1, 2, 7, n_slots // 2, n_slots):
        for permuted in (False, True):
            src = W.ids_c5(1, n, n_slots, permuted)
            dst = W.ids_c5(2, n, n_slots, permuted)
            for eng in (gpu, cpu):
                eng.copy_blocks(0, src, 1, dst)          # gather HBM -> host tier
            torch.cuda.synchronize()
            assert np.array_equal(gpu.host_pool.numpy(), cpu.host_pool)
            back = W.ids_c5(3, n, n_slots, permuted)
            for eng in (gpu, cpu):
                eng.copy_blocks(1, dst, 0, back)         # scatter host tier -> HBM
            torch.cuda.synchronize()
            assert np.array_equal(gpu.hbm_pool.cpu().numpy(), cpu.hbm_pool)
    # HBM -> HBM move with disjoint halves, ids resident on the device
    half = n_slots // 2
    src = np.arange(half, dtype=np.uint32)
    dst = (np.random.default_rng(6).permutation(half) + half).astype(np.uint32)
    gpu.copy_blocks(0, torch.from_numpy(src.view(np.int32)).cuda(), 0, torch.from_numpy(dst.view(np.int32)).cuda())
    cpu.copy_blocks(0, src, 0, dst)
    torch.cuda.synchronize()
    assert np.array_equal(gpu.hbm_pool.cpu().numpy(), cpu.hbm_pool)


def test_mover_with_second_tier_in_hbm(B, oracle):
    """The in-device measurement mode: the second tier lives in HBM; results are the same."""
    kw = dict(n_hbm_blocks=64, n_host_blocks=64, max_contexts=4, **W.GEO_128K.kwargs())
    gpu = B.Engine(max_tokens=1 << 16, max_messages=256, host_pool_on_device=True, **kw)
    cpu = oracle.OracleEngine(**kw)
    S.offload_reload_round_trip(lambda **k: B.Engine(max_tokens=1 << 16, max_messages=256, host_pool_on_device=True, **k),
                                geos=[W.GEO_128K.kwargs()])
    del gpu, cpu


@pytest.mark.parametrize("geo,stage_mib", [(W.GEO_TOY, 1), (W.GEO_128K, 2), (W.GEO_8B, 64)], ids=["toy", "128K", "8B"])
@pytest.mark.parametrize("layout", [0, 1])
def test_moves_through_the_staging_ring_are_byte_exact(B, oracle, geo, stage_mib, layout):
    """Offload, reload and the moves to and from a third tier with the copy engines carrying the payload: the mover
    kernel gathers whole blocks into the staging ring (scatters them out of it) and the link sees large transfers.
    The ring is sized so that the lists wrap around it several times; lists are permuted, so transfers of one block
    and of several consecutive host slots both occur. Same results as the oracle, every byte checked."""
    n = 96
    kw = dict(n_hbm_blocks=n, n_host_blocks=n, n_remote_blocks=n // 2, max_contexts=4, pool_layout=layout, **geo.kwargs())
    gpu = B.Engine(max_tokens=1 << 16, max_messages=256, stage_mib=stage_mib, **kw)
    gpu.set_mover_variant(4)
    cpu = oracle.OracleEngine(**kw)
    rng = np.random.default_rng(5)
    tok = rng.integers(0, W.VOCAB, 16 * n, dtype=np.uint32)
    for eng in (gpu, cpu):
        eng.spawn(0); eng.append(0, tok)
        eng.map_blocks([0], 0); eng.map_blocks([0], 1); eng.prefill_done(0)
    keys = cpu.get_block_map(0)[0]
    for b in range(n):
        gpu.fill_block_pattern(0, b, int(keys[b]))

    def same_maps():
        for a, b in zip(gpu.get_block_map(0), cpu.get_block_map(0)):
            assert np.array_equal(a, b)
        _k, tier, slot = cpu.get_block_map(0)
        bad = [b for b in range(n) if tier[b] != 0xFF and not gpu.check_block_pattern(int(tier[b]), int(slot[b]), int(keys[b]))]
        assert not bad, bad[:8]

    out = rng.permutation(n)[: 3 * n // 4].astype(np.uint32)
    assert gpu.offload(out) == cpu.offload(out)
    same_maps()
    back = rng.permutation(3 * n // 4)[: n // 2].astype(np.uint32)                     # host slots, in any order
    assert gpu.reload(back) == cpu.reload(back)
    same_maps()
    host_occ = np.nonzero(cpu.get_entries(1)["key"])[0].astype(np.uint32)
    down = rng.permutation(host_occ)
    assert gpu.move(1, 2, down) == cpu.move(1, 2, down)                                # host -> remote: both in host memory
    same_maps()
    up = rng.permutation(len(down)).astype(np.uint32)[: len(down) // 2]
    assert gpu.move(2, 0, up) == cpu.move(2, 0, up)                                    # remote -> HBM through the ring
    same_maps()
    # both directions in one call, on a full HBM tier: every reload lands in a slot a victim is leaving
    for eng in (gpu, cpu):
        eng.spawn(1); eng.append(1, tok[::-1].copy())
        eng.map_blocks([1], 0)
        eng.map_blocks([1], 1); eng.prefill_done(1)
    st = cpu.get_stats()
    assert st["occ_hbm"] == n                                                          # context 1 filled what was free
    keys1 = cpu.get_block_map(1)[0]
    _k, t1, s1 = cpu.get_block_map(1)
    for b in range(len(keys1)):
        if t1[b] == 0:
            gpu.fill_block_pattern(0, int(s1[b]), int(keys1[b]))
    host_occ = np.nonzero(cpu.get_entries(1)["key"])[0].astype(np.uint32)
    ins = rng.permutation(host_occ)[: max(1, len(host_occ) // 2)]
    vg, _ = gpu.select_victims(0, len(ins) + 5)
    vc, _ = cpu.select_victims(0, len(ins) + 5)
    assert np.array_equal(vg, vc)
    assert gpu.exchange(vg, ins) == cpu.exchange(vc, ins)
    same_maps()
    _k, t1, s1 = cpu.get_block_map(1)
    bad = [b for b in range(len(keys1)) if t1[b] != 0xFF and not gpu.check_block_pattern(int(t1[b]), int(s1[b]), int(keys1[b]))]
    assert not bad, bad[:8]
    sg, sc = gpu.get_stats(), cpu.get_stats()
    for k in sc:
        if k not in W.GPU_ONLY_STATS:
            assert sg[k] == sc[k], k


def test_exchange_scenario_through_the_staging_ring(B):
    def make(**k):
        eng = B.Engine(max_tokens=1 << 16, max_messages=256, stage_mib=1, **k)
        eng.set_mover_variant(4)
        return eng
    S.exchange_both_ways(make)
    S.offload_reload_round_trip(make)
    S.inclusive_tiers(make)
    S.three_tiers(make)


@pytest.mark.parametrize("ctas", [1, 3, 64])
@pytest.mark.parametrize("on_device", [False, True], ids=["pinned-host-tier", "second-tier-in-hbm"])
def test_mover_grid_limit_does_not_change_results(B, ctas, on_device):
    """kvt_set_mover_ctas bounds the mover's grid (one thread block has to walk every tile); offload, reload and the
    two-directional exchange still move every byte, over the host link (1024-thread blocks) and inside the device."""
    def make(**k):
        eng = B.Engine(max_tokens=1 << 16, max_messages=256, host_pool_on_device=on_device, **k)
        eng.set_mover_ctas(ctas)
        return eng
    S.offload_reload_round_trip(make, geos=[W.GEO_128K.kwargs()], layouts=(0,))
    S.exchange_both_ways(make)


# ---- table maintenance and limits -------------------------------------------------------------------------
def test_tombstones_trigger_rebuild_and_lookups_survive(B, oracle):
    """Insert / drop cycles leave tombstones; the table is rebuilt when they pile up; every resident key is still
    found afterwards, and the results stay equal to the oracle's."""
    kw = dict(n_hbm_blocks=64, n_host_blocks=0, max_contexts=8, metadata_only=True, **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=1 << 16, max_messages=256, table_capacity=128, **kw)
    cpu = oracle.OracleEngine(**kw)
    base = np.random.default_rng(4).integers(0, W.VOCAB, 16 * 20, dtype=np.uint32)
    for eng in (gpu, cpu):
        eng.spawn(0)
        eng.append(0, base)
        eng.map_blocks([0], 0); eng.map_blocks([0], 1); eng.prefill_done(0)
    for round_ in range(12):                       # each round: a new 40-block context is admitted, then dropped
        toks = np.random.default_rng(100 + round_).integers(0, W.VOCAB, 16 * 40, dtype=np.uint32)
        for eng in (gpu, cpu):
            eng.spawn(1)
            eng.append(1, toks)
            eng.map_blocks([1], 0)
            info = eng.map_blocks([1], 1)
            assert int(info[0]["n_admitted"]) == 40
            eng.prefill_done(1)
            eng.terminate(1)
            v, s = eng.select_victims(0, 40)
            assert len(v) == 40 and np.all(s == 0)
            assert eng.offload(v) == (0, 40, 40)
    assert gpu.get_stats()["table_rebuilds"] >= 1
    a, b = gpu.map_blocks([0], 0), cpu.map_blocks([0], 0)
    assert np.array_equal(a, b) and int(a[0]["hit_len"]) == 20
    for x, y in zip(gpu.get_block_map(0), cpu.get_block_map(0)):
        assert np.array_equal(x, y)


def test_admission_in_rounds_when_the_table_is_tight(B, oracle):
    """A batch with more candidate blocks than the table may safely claim at once is admitted in several
    rounds; the result equals one sequential pass."""
    n = 256
    kw = dict(n_hbm_blocks=n, n_host_blocks=0, max_contexts=8, metadata_only=True, **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=1 << 18, max_messages=256, table_capacity=2 * n, **kw)   # claims capped at 3/4 * 512
    cpu = oracle.OracleEngine(**kw)
    rng = np.random.default_rng(5)
    shared = rng.integers(0, W.VOCAB, 16 * 30, dtype=np.uint32)
    toks = [np.concatenate([shared, rng.integers(0, W.VOCAB, 16 * 150, dtype=np.uint32)]) for _ in range(4)]
    for eng in (gpu, cpu):
        for c, t in enumerate(toks):
            eng.spawn(c)
            eng.append(c, t)
        eng.map_blocks([0, 1, 2, 3], 0)
    ag, ac = gpu.map_blocks([0, 1, 2, 3], 1), cpu.map_blocks([0, 1, 2, 3], 1)   # 720 candidates, 256 slots
    assert np.array_equal(ag, ac)
    assert [int(x) for x in ac["n_held"]] == [180, 106, 30, 30]
    eg, ec = gpu.get_entries(0), cpu.get_entries(0)
    for k in ec:
        assert np.array_equal(eg[k], ec[k]), k
    sg, sc = gpu.get_stats(), cpu.get_stats()
    assert (sg["inserted"], sg["adopted"]) == (sc["inserted"], sc["adopted"]) == (256, 90)


def test_capacity_errors_leave_the_engine_usable(B):
    kw = dict(n_hbm_blocks=16, n_host_blocks=4, max_contexts=4, **W.GEO_TOY.kwargs())
    eng = B.Engine(max_tokens=4096, max_messages=8, max_batch_blocks=64, max_key_blocks=128, **kw)
    rng = np.random.default_rng(6)
    eng.spawn(0)
    eng.append(0, rng.integers(0, W.VOCAB, 1500, dtype=np.uint32))
    assert eng.apply_op_rc(B.OP_APPEND, 0, tokens=rng.integers(0, W.VOCAB, 4000, dtype=np.uint32)) == B.E_NOSPACE  # token arena
    eng.spawn(1)
    eng.append(1, rng.integers(0, W.VOCAB, 16 * 60, dtype=np.uint32))
    assert eng.map_blocks_rc([0, 1], 0)[0] == B.E_NOSPACE        # 93 + 60 blocks > max_batch_blocks
    assert eng.get_stats()["clock"] == 0
    info = eng.map_blocks([1], 0)
    assert int(info[0]["n_blocks"]) == 60
    adm = eng.map_blocks([1], 1)
    assert int(adm[0]["n_admitted"]) == 16                       # pool of 16
    eng.prefill_done(1)
    v, s = eng.select_victims(0, 16)
    rc, n_done, n_dropped = eng.offload(v)                       # live blocks, host tier of 4
    assert (rc, n_done, n_dropped) == (B.E_NOSPACE, 4, 0)
    assert "host tier full" in eng.last_error()
    st = eng.get_stats()
    assert (st["occ_hbm"], st["occ_host"]) == (12, 4)
    with pytest.raises(B.KvtError):
        eng.select_victims(3, 1)                                 # bad tier


@pytest.mark.parametrize("lookup_variant", [1, 2, 4], ids=["default", "single-pass", "four-keys-per-thread"])
def test_a_sequence_of_several_hundred_chunks(B, oracle, lookup_variant):
    """A context of 40,000+ blocks (more than 128 hash chunks: its chunk carries come from the scan kernel instead of
    the per-chunk fold), next to a short one in the same batch, then a call that resumes near its end."""
    kw = dict(n_hbm_blocks=50_000, n_host_blocks=0, max_contexts=4, metadata_only=True, **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=1 << 21, max_messages=64, max_batch_blocks=60_000, **kw)
    gpu.set_lookup_variant(lookup_variant)
    rng = np.random.default_rng(31)
    long_tok = rng.integers(0, W.VOCAB, 16 * 40_001 + 5, dtype=np.uint32)
    short_tok = rng.integers(0, W.VOCAB, 16 * 300, dtype=np.uint32)
    gpu.spawn(0); gpu.append(0, long_tok)
    gpu.spawn(1); gpu.append(1, short_tok)
    gpu.map_blocks([0, 1], 0); gpu.map_blocks([0, 1], 1)
    assert np.array_equal(gpu.get_block_map(0)[0], oracle.hash_tokens(long_tok))
    assert np.array_equal(gpu.get_block_map(1)[0], oracle.hash_tokens(short_tok))
    gpu.prefill_done(0); gpu.prefill_done(1)
    more = rng.integers(0, W.VOCAB, 16 * 700, dtype=np.uint32)
    gpu.append(0, more)
    before = gpu.get_stats()["blocks_rehashed"]
    info = gpu.map_blocks([0], 0)
    assert gpu.get_stats()["blocks_rehashed"] - before == 40_701 - 40_001 // 256 * 256     # resumed at the last chunk boundary
    assert int(info["hit_len"][0]) == 40_001
    assert np.array_equal(gpu.get_block_map(0)[0], oracle.hash_tokens(np.concatenate([long_tok[:16 * 40_001 + 5], more]))[:40_701])


@pytest.mark.parametrize("lookup_variant", [1, 2, 4], ids=["default", "single-pass", "four-keys-per-thread"])
def test_incremental_hashing_resumes_at_chunk_boundaries(B, oracle, lookup_variant):
    """Appends, edits, forks and repeated calls around multiples of 256 blocks: only the changed tail is digested
    again, and every key still equals the one-shot hash of the whole sequence."""
    kw = dict(n_hbm_blocks=4096, n_host_blocks=0, max_contexts=8, metadata_only=True, **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=1 << 18, max_messages=1024, **kw)
    gpu.set_lookup_variant(lookup_variant)
    rng = np.random.default_rng(30)
    msgs = []

    def check(ctx):
        before = gpu.get_stats()["blocks_rehashed"]
        gpu.map_blocks([ctx], 0); gpu.map_blocks([ctx], 1); gpu.prefill_done(ctx)
        return gpu.get_stats()["blocks_rehashed"] - before

    gpu.spawn(0)
    # (tokens appended, blocks digested by the next call): 256 | 512 (resume at 256) | 512 (+7 tokens: nothing new)
    # | 813 (resume at 512) | 1024 (resume at 768)
    for n_tok, want in ((16 * 256, 256), (16 * 256, 256), (7, 0), (16 * 300 + 9, 301), (16 * 211, 256)):
        t = rng.integers(0, W.VOCAB, n_tok, dtype=np.uint32)
        msgs.append(t)
        gpu.append(0, t)
        assert check(0) == want
        assert np.array_equal(gpu.get_block_map(0)[0], oracle.hash_tokens(np.concatenate(msgs)))
    assert check(0) == 0                   # a call with no change digests nothing (1024 blocks, all kept)
    # an edit in the middle: everything from the chunk holding the edited message's first block is redone
    msgs[3] = rng.integers(0, W.VOCAB, 100, dtype=np.uint32)
    gpu.replace(0, 3, 4, msgs[3])
    got = check(0)
    keys = gpu.get_block_map(0)[0]
    assert np.array_equal(keys, oracle.hash_tokens(np.concatenate(msgs)))
    assert got == len(keys) - 512          # message 3 starts at token 8199 -> block 512
    # a fork resumes from its parent's list
    gpu.fork(0, 1, 3)
    extra = rng.integers(0, W.VOCAB, 16 * 40, dtype=np.uint32)
    gpu.append(1, extra)
    got = check(1)
    keys = gpu.get_block_map(1)[0]
    assert np.array_equal(keys, oracle.hash_tokens(np.concatenate(msgs[:3] + [extra])))
    assert got == len(keys) - 512
    st = gpu.get_stats()
    assert st["blocks_rehashed"] < st["blocks_hashed"]


@pytest.mark.parametrize("lookup_variant", [1, 2], ids=["default", "single-pass"])
def test_adjacent_key_lists_do_not_overlap(B, oracle, lookup_variant):
    """Key lists of one batch sit back to back in the key arena, each followed by its per-chunk carries and the
    resume point: sizes whose rounded lists leave no slack (e.g. 7,937..7,968 blocks) must not spill into the
    next list."""
    rng = np.random.default_rng(31)
    for sizes in ((7950, 300, 7968), (7937, 7968, 31), (16130, 16160, 288), (255, 256, 257, 32, 1)):
        kw = dict(n_hbm_blocks=64, n_host_blocks=0, max_contexts=8, metadata_only=True, **W.GEO_TOY.kwargs())
        gpu = B.Engine(max_tokens=1 << 21, max_messages=64, **kw)
        gpu.set_lookup_variant(lookup_variant)
        toks = []
        for c, nb in enumerate(sizes):
            toks.append(rng.integers(0, W.VOCAB, nb * 16 + 5, dtype=np.uint32))
            gpu.spawn(c)
            gpu.append(c, toks[c])
        for rnd in range(2):       # second round: everything is resumed from the kept carries
            gpu.map_blocks(list(range(len(sizes))), 0)
            for c in range(len(sizes)):
                assert np.array_equal(gpu.get_block_map(c)[0], oracle.hash_tokens(toks[c])), (sizes, rnd, c)
            for c in range(len(sizes)):
                gpu.prefill_done(c)
            for c in range(len(sizes)):
                extra = rng.integers(0, W.VOCAB, 16 * 3, dtype=np.uint32)
                toks[c] = np.concatenate([toks[c], extra])
                gpu.append(c, extra)


def test_create_rejects_bad_configs(B):
    import ctypes as C
    import torch
    lib = B.load_library()
    good = B.Engine(n_hbm_blocks=16, n_host_blocks=4, max_contexts=4, max_tokens=4096, max_messages=64, **W.GEO_TOY.kwargs())

    def attempt(**changes):
        cfg = B.Config.from_buffer_copy(good.cfg)
        for k, v in changes.items():
            setattr(cfg, k, v)
        h = C.c_void_p()
        rc = lib.kvt_create(C.byref(cfg), C.c_void_p(torch.cuda.current_stream().cuda_stream), C.byref(h))
        if rc == 0:
            lib.kvt_destroy(h)
        return rc

    assert attempt() == B.OK                                   # the unmodified copy is fine
    assert attempt(abi_version=1) == B.E_INVAL
    assert attempt(n_remote_blocks=4) == B.E_INVAL                                # a remote tier without its pool
    assert attempt(block_tokens=32) == B.E_INVAL
    assert attempt(table_capacity=good.cfg.table_capacity + 1) == B.E_INVAL      # not a power of two
    assert attempt(table_capacity=16) == B.E_INVAL                                # < 2 * (hbm + host)
    assert attempt(dev_meta=good.cfg.dev_meta + 8) == B.E_INVAL                   # misaligned arena
    assert attempt(dev_meta_bytes=1024) == B.E_INVAL                              # arena too small
    assert attempt(hbm_pool_bytes=1024) == B.E_INVAL
    assert attempt(suspended_order=2) == B.E_INVAL and attempt(policy_flags=8) == B.E_INVAL
    assert attempt(n_hbm_blocks=0) == B.E_INVAL and attempt(max_contexts=0) == B.E_INVAL
    assert lib.kvt_create(None, None, None) == B.E_INVAL


# ---- the checked build: device-side index checks, every launch in another shape -----------------------------
def test_checked_build_in_another_launch_shape():
    """The same scenario expectations and a slice of the random differential streams, in a child process that loads
    libkvt_debug.so (-DKVT_DEBUG): 64-thread blocks for the element-wise kernels, at most five mover thread blocks,
    plain launches instead of the selection's CUDA graph, and index / invariant checks that set the device error
    word. Results must not depend on the launch shape, and no check may fire."""
    import os
    import subprocess
    import sys
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_39819_b200 import build
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, KVT_LIB=build.build_debug_lib())
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider", "-m", "gpu",
           os.path.join(root, "tests", "test_gpu_parity.py"), os.path.join(root, "tests", "test_gpu_fuzz.py"),
           "-k", "test_scenario or c1_trace_parity or (random_api_streams_match and hbm24 and (0-0 or 2-1 or 4-2 or 7-3)) "
                 "or staging_ring or c4_lookup_and_select_parity and 5000"]
    r = subprocess.run(cmd, env=env, cwd=root, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, (r.stdout[-3000:], r.stderr[-2000:])
    assert "passed" in r.stdout
