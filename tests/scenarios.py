"""Scenario checks that take an engine factory, so the same expectations (which come from the
paper's sentences, from hand-worked examples and from brute force) pin the CPU oracle in the
"not gpu" tests and are re-run against the CUDA engine in the "gpu" tests."""
import os

import numpy as np

HBM, HOST = 0, 1
LOOKUP, ADMIT = 0, 1
DEAD, IDLE, ACTIVE, PINNED, FREE = 0, 1, 2, 3, 0xFF
E_INVAL, E_NOCTX, E_RANGE, E_STATE, E_NOSPACE, E_BUFSZ = -1, -2, -3, -4, -5, -6

TOY = dict(n_layers=2, n_kv_heads=2, head_dim=64)
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def toks(rng, n):
    return rng.integers(0, 151552, int(n), dtype=np.uint32)


def call(eng, ctx, done=True):
    """lookup + admit (+ prefill-done) of one context with free space assumed."""
    a = eng.map_blocks([ctx], LOOKUP)[0]
    b = eng.map_blocks([ctx], ADMIT)[0]
    if done:
        eng.prefill_done(ctx)
    return a, b


def states(eng, tier=HBM):
    return [int(x) for x in eng.get_states(tier)]


# ---- Section 5.2 runtime transitions, one context ------------------------------------------------
def state_machine_single_context(make):
    eng = make(n_hbm_blocks=16, n_host_blocks=4, max_contexts=4, **TOY)
    rng = np.random.default_rng(1)
    eng.spawn(0)
    eng.append(0, toks(rng, 64))                         # 4 blocks
    a, b = call(eng, 0, done=False)
    assert (a["n_blocks"], a["hit_len"], a["n_admissible"]) == (4, 0, 4)
    assert (b["n_admitted"], b["n_held"]) == (4, 4)
    assert states(eng)[:5] == [ACTIVE] * 4 + [FREE]      # participating in a request: Active
    assert list(eng.select_victims(HBM, 16)[0]) == []    # in-flight KV is never a victim
    eng.prefill_done(0)
    assert states(eng)[:4] == [IDLE] * 4                 # prefill complete: Suspended
    a = eng.map_blocks([0], LOOKUP)[0]
    assert (a["hit_len"], a["n_hit_hbm"], a["n_admissible"]) == (4, 4, 0)
    assert states(eng)[:4] == [ACTIVE] * 4               # next request reactivates
    eng.map_blocks([0], ADMIT)
    eng.prefill_done(0)
    eng.terminate(0)
    assert states(eng)[:4] == [DEAD] * 4                 # context terminates: Expired
    assert eng.get_stats()["n_contexts"] == 0


# ---- remove / replace: suffix invalidation from the edited message's first block -----------------
def suffix_invalidation(make):
    eng = make(n_hbm_blocks=32, n_host_blocks=4, max_contexts=4, **TOY)
    rng = np.random.default_rng(2)
    eng.spawn(0)
    msgs = [toks(rng, n) for n in (40, 24, 50, 30)]      # bounds [0,40) [40,64) [64,114) [114,144): 9 blocks
    for m in msgs:
        eng.append(0, m)
    call(eng, 0)
    keys0 = eng.get_block_map(0)[0].copy()
    assert states(eng)[:9] == [IDLE] * 9
    eng.replace(0, 2, 3, toks(rng, 10))                  # message 2 starts at token 64 -> block 4
    assert states(eng)[:9] == [IDLE] * 4 + [DEAD] * 5    # takes effect at the op, later messages included
    a, b = call(eng, 0, done=False)
    keys1 = eng.get_block_map(0)[0]
    assert a["hit_len"] == 4 and np.array_equal(keys1[:4], keys0[:4])
    assert not np.intersect1d(keys1[4:], keys0[4:]).size  # every key from that block on is new
    eng.prefill_done(0)
    # removing message 1 (starts at token 40, inside block 2): block 2 straddles and dies too
    eng.remove(0, 1, 2)
    st = states(eng)
    keys, tier, slot = eng.get_block_map(0)
    assert [st[s] for s in slot[:2]] == [IDLE, IDLE]
    assert all(st[s] == DEAD for s in slot[2:] if s != 0xFFFFFFFF)
    # an edit of the last message only kills its own blocks
    eng2 = make(n_hbm_blocks=32, n_host_blocks=4, max_contexts=4, **TOY)
    eng2.spawn(0)
    for m in msgs:
        eng2.append(0, m)
    call(eng2, 0)
    eng2.remove(0, 3, 4)                                 # starts at token 114 -> block 7
    assert states(eng2)[:9] == [IDLE] * 7 + [DEAD] * 2


# ---- fork: shared prefix, independent states; the paper's shared-KV example (Section 6.1) --------
def fork_and_shared_kv(make):
    eng = make(n_hbm_blocks=32, n_host_blocks=4, max_contexts=4, **TOY)
    rng = np.random.default_rng(3)
    eng.spawn(0)
    for n in (32, 32, 32):
        eng.append(0, toks(rng, n))                      # 6 blocks, message j = blocks 2j, 2j+1
    call(eng, 0)
    eng.fork(0, 1, 2)                                    # child shares messages 0,1 = blocks 0..3
    assert states(eng)[:6] == [ACTIVE] * 4 + [IDLE] * 2  # child's inherited messages are Active
    eng.append(1, toks(rng, 32))
    a, b = call(eng, 1)
    assert a["hit_len"] == 4 and b["n_admitted"] == 2    # identical prefixes hash identically
    assert states(eng)[:8] == [IDLE] * 8
    # parent removes message 1: its KV (blocks 2..5 for the parent) expires for the parent only;
    # the child still holds a Suspended reference to blocks 2,3 -> they stay Suspended.
    eng.remove(0, 1, 2)
    assert states(eng)[:8] == [IDLE, IDLE, IDLE, IDLE, DEAD, DEAD, IDLE, IDLE]
    # the block dies only once nobody maps it any more (Section 6.1): now the child goes too
    eng.terminate(1)
    assert states(eng)[:8] == [IDLE, IDLE] + [DEAD] * 6
    # execution in one context does not touch the other's message states
    eng.fork(0, 2, 1)
    eng.map_blocks([2], LOOKUP)
    assert states(eng)[:2] == [ACTIVE, ACTIVE]
    eng.map_blocks([2], ADMIT)
    eng.prefill_done(2)
    eng.terminate(2)
    assert states(eng)[:2] == [IDLE, IDLE]               # parent's Suspended reference remains


# ---- one_off: Temporary messages bypass reuse storage (Algorithm 1; Section 5.2 (3)) --------------
def one_off_bypass(make):
    eng = make(n_hbm_blocks=32, n_host_blocks=4, max_contexts=4, **TOY)
    rng = np.random.default_rng(4)
    eng.spawn(0)
    eng.append(0, toks(rng, 64))
    call(eng, 0)
    # compaction pattern (Section 4.2): fork, declare one-off, append the instruction, run
    eng.fork(0, 1, 1)
    eng.one_off(1)
    eng.append(1, toks(rng, 48))
    a, b = call(eng, 1, done=False)
    assert (a["n_blocks"], a["hit_len"], a["n_admissible"]) == (7, 4, 0)
    assert (b["n_admitted"], b["n_held"]) == (0, 4)
    assert eng.get_stats()["occ_hbm"] == 4               # nothing of the temporary context was stored
    assert states(eng)[:4] == [IDLE] * 4                 # Temporary references do not keep KV alive
    eng.prefill_done(1)
    eng.terminate(1)
    # per-message form: a scratch message at the tail; the block it shares with an ordinary message
    # is admissible, blocks made only of temporary tokens are not
    eng.append(0, toks(rng, 24))                         # tokens 64..88
    eng.append(0, toks(rng, 40))                         # tokens 88..128 (scratch)
    eng.one_off(0, 2, 3)
    a, b = call(eng, 0, done=False)
    assert (a["n_blocks"], a["hit_len"], a["n_admissible"]) == (8, 4, 2)   # blocks 4 and 5 (straddles 88)
    assert b["n_held"] == 6
    eng.prefill_done(0)
    # a temporary message in the middle stops admission at its first pure block
    eng.append(0, toks(rng, 64))
    a, b = call(eng, 0, done=False)
    assert (a["hit_len"], a["n_admissible"]) == (6, 0)
    eng.prefill_done(0)


# ---- pin / unpin: explicit retention (Table 3; Section 5.2; Algorithm 1's last branch) ---------------
def pinned_retention(make):
    eng = make(n_hbm_blocks=8, n_host_blocks=4, max_contexts=4, **TOY)
    rng = np.random.default_rng(15)
    eng.spawn(0)
    eng.append(0, toks(rng, 32))                         # system message: blocks 0, 1
    eng.pin(0, 0, 1)                                     # pinned at initialisation (Section 4.2)
    eng.append(0, toks(rng, 32))                         # blocks 2, 3
    a, b = call(eng, 0, done=False)
    assert (a["n_admissible"], a["n_pinned"], b["n_held"]) == (4, 2, 4)
    assert states(eng)[:4] == [PINNED, PINNED, ACTIVE, ACTIVE]
    eng.prefill_done(0)
    assert states(eng)[:4] == [PINNED, PINNED, IDLE, IDLE]      # prefill-done does not touch Pinned messages
    v, s = eng.select_victims(HBM, 8)
    assert list(v) == [3, 2] and list(s) == [1, 1]              # Pinned KV is out of ordinary contention
    v, s = eng.select_victims(HBM, 8, include_pinned=True)
    assert list(v) == [3, 2, 1, 0] and list(s) == [1, 1, 3, 3]  # it competes last, oldest / deepest first
    eng.map_blocks([0], LOOKUP)
    assert states(eng)[:4] == [PINNED, PINNED, ACTIVE, ACTIVE]
    eng.map_blocks([0], ADMIT)
    eng.prefill_done(0)
    # unpin between calls: back to Suspended
    eng.unpin(0, 0, 1)
    assert states(eng)[:4] == [IDLE] * 4
    eng.pin(0, 0, 2)
    assert states(eng)[:4] == [PINNED] * 4
    eng.unpin(0, 1, 2)
    # termination: ordinary messages expire, Pinned ones keep their protection
    eng.terminate(0)
    assert states(eng)[:4] == [PINNED, PINNED, DEAD, DEAD]
    assert eng.get_stats()["n_contexts"] == 1
    assert eng.apply_op_rc(3, 0, tokens=toks(rng, 4)) == E_NOCTX     # (3 = append) the context has ended
    assert eng.apply_op_rc(1, 0) == E_INVAL                          # (1 = spawn) its id is still in use
    assert eng.map_blocks_rc([0], LOOKUP)[0] == E_NOCTX
    # releasing the protection of a terminated context: Expired, and the context goes away
    eng.unpin(0, 0, 1)
    assert states(eng)[:4] == [DEAD] * 4
    assert eng.get_stats()["n_contexts"] == 0
    eng.spawn(0)


def pinned_competes_only_with_pinned(make, run_call, options):
    eng = make(n_hbm_blocks=4, n_host_blocks=4, max_contexts=4, **TOY)
    rng = np.random.default_rng(16)
    eng.spawn(0)
    eng.append(0, toks(rng, 64))
    eng.pin(0, 0, 1)
    run_call(eng, [0], options())                       # 4 pinned blocks fill the pool
    assert states(eng) == [PINNED] * 4
    eng.spawn(1)
    eng.append(1, toks(rng, 32))
    rec = run_call(eng, [1], options())                  # ordinary KV cannot displace Pinned KV
    assert int(rec["admit"][0]["n_admitted"]) == 0 and len(rec["victims"]) == 0
    assert states(eng) == [PINNED] * 4
    eng.spawn(2)
    eng.append(2, toks(rng, 32))
    eng.pin(2, 0, 1)
    rec = run_call(eng, [2], options())                  # Pinned incoming KV competes with Pinned residents
    assert list(rec["victims"]) == [3, 2] and list(rec["vstates"]) == [3, 3]
    assert rec["offload"] == (0, 2, 0)                   # live: moved to the host tier, not dropped
    assert int(rec["admit"][0]["n_admitted"]) == 2
    assert states(eng) == [PINNED] * 4 and states(eng, HOST)[:2] == [PINNED, PINNED]
    # one_off on a context does not strip explicit protection
    eng.one_off(2)
    assert states(eng)[2:] == [PINNED, PINNED]
    eng.one_off(2, 0, 1)                                 # the per-message declaration does
    assert states(eng)[2:] == [DEAD, DEAD]


# ---- "w/o LT" ablation (Section 8.3): no lifecycle information reaches the policy -----------------------
def no_lifecycle_policy(make):
    eng = make(n_hbm_blocks=8, n_host_blocks=8, max_contexts=4, policy_flags=1, **TOY)
    rng = np.random.default_rng(17)
    eng.spawn(0)
    eng.append(0, toks(rng, 64))                         # blocks 0..3, clock 1..2
    call(eng, 0)
    eng.spawn(1)
    eng.one_off(1)
    eng.append(1, toks(rng, 32))                         # a one-off context: its KV would bypass storage
    a, b = call(eng, 1)
    assert (a["n_admissible"], b["n_admitted"]) == (2, 2)    # nothing is known to be Temporary: admitted
    eng.terminate(1)
    eng.remove(0, 0, 1)
    assert states(eng)[:6] == [DEAD] * 6                 # the true states are still reported (for metrics) ...
    v, s = eng.select_victims(HBM, 8)
    assert list(v) == [5, 4, 3, 2, 1, 0] and list(s) == [1] * 6   # ... but the policy sees one tier, newest first
    rc, n_done, n_dropped = eng.offload(v[:3])
    assert (rc, n_done, n_dropped) == (0, 3, 0)          # and cannot reclaim zombies without a copy
    assert eng.get_stats()["occ_host"] == 3
    eng2 = make(n_hbm_blocks=8, n_host_blocks=8, max_contexts=4, policy_flags=1, suspended_order=1, **TOY)
    eng2.debug_load_resident([10, 11, 12], [2, 0, 1], [5, 9, 7], [0, 0, 0], [0, 1, 2], HBM)
    assert list(eng2.select_victims(HBM, 3)[0]) == [0, 2, 1]      # plain LRU


# ---- inclusive tiering: a reloaded block keeps its host copy, a later offload of it needs no copy ----------
SHADOW, HAS_COPY, NONE = 0xFE, 0x80, 0xFFFFFFFF


def inclusive_tiers(make):
    eng = make(n_hbm_blocks=6, n_host_blocks=6, max_contexts=4, policy_flags=2, **TOY)
    rng = np.random.default_rng(18)
    eng.spawn(0)
    eng.append(0, toks(rng, 64))
    call(eng, 0)                                         # blocks 0..3 at HBM slots 0..3
    keys = eng.get_block_map(0)[0]
    for b in range(4):
        eng.write_block(HBM, b, _payload(keys[b], eng.block_bytes))
    assert eng.offload([3, 2]) == (0, 2, 0)              # copied to host slots 0 (block 3) and 1 (block 2)
    a = eng.map_blocks([0], LOOKUP)[0]
    assert (a["hit_len"], a["n_hit_hbm"], a["n_hit_host"]) == (4, 2, 2)
    assert eng.reload([1, 0]) == (0, 2)                  # block 2 -> HBM slot 2, block 3 -> HBM slot 3
    st = eng.get_stats()
    assert (st["occ_hbm"], st["occ_host"], st["bytes_h2d"]) == (4, 2, 2 * eng.block_bytes)   # host copies stay
    assert states(eng, HOST)[:3] == [SHADOW, SHADOW, FREE]
    assert list(eng.get_entries(HBM)["link"][:4]) == [NONE, NONE, 1, 0]
    assert list(eng.get_entries(HOST)["link"][:2]) == [3, 2]
    assert list(eng.get_block_map(0)[1]) == [HBM] * 4    # the block's home is HBM again
    assert eng.reload([0])[0] == E_INVAL                 # a copy is not a resident block of the host tier
    eng.map_blocks([0], ADMIT)
    eng.prefill_done(0)
    v, s = eng.select_victims(HBM, 4)
    assert list(v) == [3, 2, 1, 0] and list(s) == [IDLE | HAS_COPY, IDLE | HAS_COPY, IDLE, IDLE]
    d2h = eng.get_stats()["bytes_d2h"]
    assert eng.offload([3, 2]) == (0, 2, 0)              # handed over to their host copies: nothing is copied
    st = eng.get_stats()
    assert (st["occ_hbm"], st["occ_host"], st["bytes_d2h"], st["offloaded"], st["offloaded_clean"]) == (2, 2, d2h, 4, 2)
    assert states(eng, HOST)[:2] == [IDLE, IDLE] and list(eng.get_entries(HOST)["link"][:2]) == [NONE, NONE]
    k, t, sl = eng.get_block_map(0)
    assert list(t) == [HBM, HBM, HOST, HOST] and list(sl) == [0, 1, 1, 0]
    for b in range(4):
        assert np.array_equal(eng.read_block(int(t[b]), int(sl[b])), _payload(keys[b], eng.block_bytes))
    # copies are the first victims of the host tier (dropping them loses nothing) and may be released
    assert eng.reload([1, 0]) == (0, 2)
    v, s = eng.select_victims(HOST, 6)
    assert list(v) == [0, 1] and list(s) == [SHADOW, SHADOW]     # same stamp: deeper block first
    eng.release(HOST, [0])                               # drop the copy of block 3
    assert list(eng.get_entries(HBM)["link"][:4]) == [NONE, NONE, 1, NONE]
    assert eng.get_stats()["occ_host"] == 1
    eng.release(HBM, [2])                                # drop block 2: its copy goes with it
    st = eng.get_stats()
    assert (st["occ_hbm"], st["occ_host"]) == (3, 0)
    assert list(eng.get_block_map(0)[1]) == [HBM, HBM, 0xFF, HBM]
    # compaction keeps block and copy linked
    assert eng.offload([3]) == (0, 1, 0)                 # block 3 -> host slot 0 (copied again: its copy was dropped)
    assert eng.reload([0]) == (0, 1)                     # back to HBM slot 2, host slot 0 is its copy
    eng.release(HBM, [0])
    assert eng.compact(HBM) == 1                         # 2 occupied: slot 2 moves to slot 0
    assert list(eng.get_entries(HBM)["link"][:3]) == [0, NONE, NONE]
    assert list(eng.get_entries(HOST)["link"][:1]) == [0]
    assert list(eng.get_block_map(0)[2]) == [NONE, 1, NONE, 0]
    # a dead block with a copy: both are reclaimed
    eng.terminate(0)
    v, s = eng.select_victims(HBM, 6)
    assert list(s) == [DEAD | HAS_COPY, DEAD]
    assert eng.offload(v) == (0, 2, 2)
    st = eng.get_stats()
    assert (st["occ_hbm"], st["occ_host"]) == (0, 0)


# ---- exchange: reload and offload in one call, destinations = slots free when the call begins ------------------
def exchange_both_ways(make):
    for flags in (0, 2):
        eng = make(n_hbm_blocks=8, n_host_blocks=8, max_contexts=4, policy_flags=flags, **TOY)
        rng = np.random.default_rng(19)
        keys = {}
        for c in (0, 1):
            eng.spawn(c)
            eng.append(c, toks(rng, 64))
            call(eng, c)                                  # context 0: HBM slots 0..3, context 1: slots 4..7
            k, _t, sl = eng.get_block_map(c)
            keys[c] = k
            for kk, s_ in zip(k, sl):
                eng.write_block(HBM, int(s_), _payload(kk, eng.block_bytes))
        assert eng.offload([7, 6]) == (0, 2, 0)           # context 1's blocks 3, 2 -> host slots 0, 1
        # bring them back while pushing context 0's tail out, as offload then reload would: the outgoing blocks take
        # the host slots that are free now (2, 3; 0 and 1 are still occupied), the incoming ones the lowest free HBM
        # slots, which are the two the victims just left (2, 3), not 6 and 7
        assert eng.exchange([3, 2], [1, 0]) == (0, 2, 0, 2)
        _k, t1, s1 = eng.get_block_map(1)
        assert list(t1) == [HBM] * 4 and list(s1) == [4, 5, 2, 3]
        _k, t0, s0 = eng.get_block_map(0)
        assert list(t0) == [HBM, HBM, HOST, HOST] and list(s0) == [0, 1, 3, 2]
        st = eng.get_stats()
        assert (st["occ_hbm"], st["occ_host"]) == ((6, 2) if flags == 0 else (6, 4))   # inclusive keeps the copies
        for c in (0, 1):
            _k, t, sl = eng.get_block_map(c)
            for b in range(4):
                assert np.array_equal(eng.read_block(int(t[b]), int(sl[b])), _payload(keys[c][b], eng.block_bytes))
        # second exchange: context 0's block 0 goes out and its tail comes back, into the slot block 0 left and
        # into slot 6; the host slots 0, 1 are free again without inclusive tiers, and still hold clean copies with them
        assert eng.exchange([0], [3, 2]) == (0, 1, 0, 2)
        _k, t0, s0 = eng.get_block_map(0)
        assert list(t0) == [HOST, HBM, HBM, HBM] and list(s0) == [0 if flags == 0 else 4, 1, 0, 6]
        # validation covers both lists before anything moves
        watch = ("occ_hbm", "occ_host", "offloaded", "reloaded", "dropped", "bytes_d2h", "bytes_h2d")
        before = {k: eng.get_stats()[k] for k in watch}
        assert eng.exchange([1, 1], [])[0] == E_INVAL and eng.exchange([], [7])[0] == E_INVAL
        assert eng.exchange([9], [])[0] == E_RANGE and eng.exchange([1], [9])[0] == E_RANGE
        assert {k: eng.get_stats()[k] for k in watch} == before
        for c in (0, 1):
            _k, t, sl = eng.get_block_map(c)
            for b in range(4):
                assert np.array_equal(eng.read_block(int(t[b]), int(sl[b])), _payload(keys[c][b], eng.block_bytes))
    # more incoming blocks than free HBM slots: what fits is done, the rest is reported
    eng = make(n_hbm_blocks=4, n_host_blocks=4, max_contexts=4, **TOY)
    rng = np.random.default_rng(20)
    eng.spawn(0)
    eng.append(0, toks(rng, 64))
    call(eng, 0)
    assert eng.offload([3, 2]) == (0, 2, 0)
    eng.spawn(1)
    eng.append(1, toks(rng, 16))
    call(eng, 1)                                          # takes HBM slot 2; slot 3 is the only free one
    assert eng.exchange([], [0, 1]) == (E_NOSPACE, 0, 0, 1)
    assert list(eng.get_block_map(0)[2]) == [0, 1, 1, 3]  # block 3 came back to HBM slot 3, block 2 still at host slot 1
    assert eng.exchange([], []) == (0, 0, 0, 0)
    # a full pool: the incoming blocks can only go where the outgoing ones were; every byte of both survives
    eng = make(n_hbm_blocks=4, n_host_blocks=4, max_contexts=4, **TOY)
    rng = np.random.default_rng(23)
    keys = {}
    for c in (0, 1):
        eng.spawn(c)
        eng.append(c, toks(rng, 32))
        call(eng, c)                                      # context 0 at HBM slots 0, 1; context 1 at slots 2, 3
        keys[c] = eng.get_block_map(c)[0]
        for b in range(2):
            eng.write_block(HBM, 2 * c + b, _payload(keys[c][b], eng.block_bytes))
    assert eng.offload([3, 2]) == (0, 2, 0)               # context 1 -> host slots 0 (block 1), 1 (block 0)
    eng.spawn(2)
    eng.append(2, toks(rng, 32))
    call(eng, 2)                                          # context 2 fills HBM slots 2, 3: the pool is full
    keys[2] = eng.get_block_map(2)[0]
    for b in range(2):
        eng.write_block(HBM, 2 + b, _payload(keys[2][b], eng.block_bytes))
    assert eng.get_stats()["occ_hbm"] == 4
    assert eng.exchange([1, 0], [1, 0]) == (0, 2, 0, 2)   # context 0 out (host slots 2, 3), context 1 into slots 0, 1
    assert [list(x) for x in eng.get_block_map(1)[1:]] == [[HBM, HBM], [0, 1]]
    assert [list(x) for x in eng.get_block_map(0)[1:]] == [[HOST, HOST], [3, 2]]
    for c in (0, 1, 2):
        _k, t, sl = eng.get_block_map(c)
        for b in range(2):
            assert np.array_equal(eng.read_block(int(t[b]), int(sl[b])), _payload(keys[c][b], eng.block_bytes)), (c, b)


# ---- hand-worked lifecycle example (8-block pool) --------------------------------------------------
def worked_example(make):
    eng = make(n_hbm_blocks=8, n_host_blocks=8, max_contexts=4, **TOY)
    rng = np.random.default_rng(0)
    A, B = 0, 1
    eng.spawn(A)
    for n in (20, 30, 14):
        eng.append(A, toks(rng, n))                      # bounds [0,20) [20,50) [50,64): 4 blocks
    a, b = call(eng, A, done=False)                      # clock 1
    assert (b["n_admitted"],) == (4,)
    assert list(eng.get_block_map(A)[2]) == [0, 1, 2, 3] # lowest free slots in chain order
    assert list(eng.get_entries(HBM)["stamp"][:4]) == [1] * 4
    eng.prefill_done(A)                                  # clock 2
    assert list(eng.get_entries(HBM)["stamp"][:4]) == [2] * 4
    eng.fork(A, B, 2)                                    # child maps floor(50/16) = 3 blocks
    assert states(eng)[:4] == [ACTIVE, ACTIVE, ACTIVE, IDLE]
    eng.append(B, toks(rng, 30))
    a, b = call(eng, B, done=False)                      # clock 3; 80 tokens = 5 blocks
    assert (a["n_blocks"], a["hit_len"]) == (5, 3)       # block 3 differs from A's: tokens 50.. differ
    assert list(eng.get_block_map(B)[2]) == [0, 1, 2, 4, 5]
    eng.prefill_done(B)                                  # clock 4
    assert list(eng.get_entries(HBM)["stamp"][:6]) == [4, 4, 4, 2, 4, 4]
    eng.remove(A, 1, 2)                                  # cut = floor(20/16) = 1
    assert states(eng)[:6] == [IDLE, IDLE, IDLE, DEAD, IDLE, IDLE]
    eng.terminate(B)
    assert states(eng)[:6] == [IDLE, DEAD, DEAD, DEAD, DEAD, DEAD]
    v, s = eng.select_victims(HBM, 8)
    # dead tier oldest first (stamp 2), then stamp 4 by depth 4,3,2,1; then the one Suspended block
    assert list(v) == [3, 5, 4, 2, 1, 0] and list(s) == [0, 0, 0, 0, 0, 1]
    assert eng.get_stats()["clock"] == 4


def mixed_pool_example(make, order=0):
    """{slot: (state, stamp, depth, inflight)}; slot 5 is in flight."""
    eng = make(n_hbm_blocks=8, n_host_blocks=8, max_contexts=4, suspended_order=order, **TOY)
    S, D, A = IDLE, DEAD, ACTIVE
    pool = {0: (S, 5, 0), 1: (S, 5, 1), 2: (S, 9, 2), 3: (D, 7, 3), 4: (D, 2, 1), 6: (A, 8, 4), 7: (S, 9, 3)}
    slots = sorted(pool)
    eng.debug_load_resident([100 + s for s in slots], [pool[s][0] for s in slots], [pool[s][1] for s in slots],
                            [pool[s][2] for s in slots], slots, HBM)
    # slot 5: held in flight by a real context
    rng = np.random.default_rng(9)
    eng.spawn(0)
    eng.append(0, toks(rng, 16))
    call(eng, 0, done=False)
    assert list(eng.get_block_map(0)[2]) == [5]
    v, s = eng.select_victims(HBM, 8)
    if order == 0:
        assert list(v) == [4, 3, 7, 2, 1, 0, 6]          # idle tier newest first
    else:
        assert list(v) == [4, 3, 1, 0, 7, 2, 6]          # idle tier oldest first
    assert list(s) == [0, 0, 1, 1, 1, 1, 2]
    v3, _ = eng.select_victims(HBM, 3)
    assert list(v3) == list(v[:3])                       # a prefix of the same order


# ---- victim order = brute-force sort, Algorithm 1 order, LRU special cases ------------------------
def _brute_order(ent, st, mru):
    cands = [s for s in range(len(st)) if st[s] != FREE and ent["inflight"][s] == 0 and st[s] < 3]

    def key(s):
        rec = int(ent["stamp"][s])
        if st[s] == IDLE and mru:
            rec = -rec
        return (int(st[s]), rec, -int(ent["depth"][s]), s)
    return sorted(cands, key=key)


def victim_order_bruteforce(make, seeds=range(30)):
    for seed in seeds:
        rng = np.random.default_rng(seed)
        order = int(seed % 2)
        n = int(rng.integers(1, 65))
        eng = make(n_hbm_blocks=n, n_host_blocks=8, max_contexts=4, suspended_order=order, **TOY)
        k = int(rng.integers(0, n + 1))
        slots = rng.permutation(n)[:k]
        eng.debug_load_resident(rng.integers(2, 1 << 62, k).astype(np.uint64), rng.integers(0, 3, k),
                                rng.integers(0, 6, k), rng.integers(0, 4, k), slots, HBM)  # many ties
        st = eng.get_states(HBM)
        want = _brute_order(eng.get_entries(HBM), st, order == 0)
        for n_req in (0, 1, k // 2, k, k + 5):
            v, s = eng.select_victims(HBM, n_req)
            assert list(v) == want[: n_req], (seed, n_req)
            assert [int(x) for x in s] == [int(st[i]) for i in v]
            # Algorithm 1: no idle victim while a dead candidate remains, no active while idle remains
            if len(v) < len(want):
                rest = [int(st[i]) for i in want[len(v):]]
                assert max([int(x) for x in s], default=0) <= min(rest)


def one_state_pools_reduce_to_lru(make):
    rng = np.random.default_rng(5)
    n = 40
    stamps = rng.permutation(1000)[:n]                   # distinct stamps
    lru = list(np.argsort(stamps))
    for state, order, want in ((DEAD, 0, lru), (ACTIVE, 0, lru), (IDLE, 1, lru), (IDLE, 0, lru[::-1])):
        eng = make(n_hbm_blocks=n, n_host_blocks=8, max_contexts=4, suspended_order=order, **TOY)
        eng.debug_load_resident(np.arange(n) + 50, [state] * n, stamps, np.zeros(n), np.arange(n), HBM)
        v, _ = eng.select_victims(HBM, n)
        assert list(v) == want, (state, order)


# ---- movement ------------------------------------------------------------------------------------
def _payload(key, nbytes):
    rng = np.random.default_rng(int(key))
    return rng.integers(0, 256, nbytes, dtype=np.uint8)


def offload_reload_round_trip(make, geos=None, layouts=(0, 1)):
    geos = geos or [TOY, dict(n_layers=3, n_kv_heads=1, head_dim=16), dict(n_layers=1, n_kv_heads=8, head_dim=128)]
    for geo in geos:
        for layout in layouts:
            eng = make(n_hbm_blocks=12, n_host_blocks=6, max_contexts=4, pool_layout=layout, **geo)
            rng = np.random.default_rng(6)
            eng.spawn(0)
            eng.append(0, toks(rng, 16 * 10))
            call(eng, 0)
            keys, tier, slot = eng.get_block_map(0)
            for k, s in zip(keys, slot):
                eng.write_block(HBM, int(s), _payload(k, eng.block_bytes))
            # suspended blocks are live: offload copies them to the lowest free host slots, in order
            rc, n_done, n_dropped = eng.offload([7, 2, 9, 4])
            assert (rc, n_done, n_dropped) == (0, 4, 0)
            k2, t2, s2 = eng.get_block_map(0)
            assert [int(t2[b]) for b in (7, 2, 9, 4)] == [HOST] * 4 and [int(s2[b]) for b in (7, 2, 9, 4)] == [0, 1, 2, 3]
            for b in (7, 2, 9, 4):
                assert np.array_equal(eng.read_block(HOST, int(s2[b])), _payload(keys[b], eng.block_bytes))
            assert eng.get_stats()["occ_hbm"] == 6 and eng.get_stats()["occ_host"] == 4
            # host tier has 2 slots left: the third live victim does not fit
            rc, n_done, n_dropped = eng.offload([0, 1, 3])
            assert (rc, n_done, n_dropped) == (E_NOSPACE, 2, 0)
            # reload in a different order: lowest free HBM slots
            free_hbm = sorted(set(range(12)) - {int(s) for s, t in zip(*eng.get_block_map(0)[2:0:-1]) if t == HBM})
            hs = [int(eng.get_block_map(0)[2][b]) for b in (9, 0, 7)]
            rc, n_done = eng.reload(hs)
            assert (rc, n_done) == (0, 3)
            k3, t3, s3 = eng.get_block_map(0)
            assert [int(s3[b]) for b in (9, 0, 7)] == free_hbm[:3]
            for b in range(10):
                assert np.array_equal(eng.read_block(int(t3[b]), int(s3[b])), _payload(keys[b], eng.block_bytes)), (geo, layout, b)
            # lookups find blocks in either tier and report where they are
            a = eng.map_blocks([0], LOOKUP)[0]
            assert (a["hit_len"], a["n_hit_hbm"], a["n_hit_host"]) == (10, 7, 3)
            eng.prefill_done(0)


def dead_victims_are_dropped_without_copy(make):
    eng = make(n_hbm_blocks=8, n_host_blocks=4, max_contexts=4, **TOY)
    rng = np.random.default_rng(7)
    eng.spawn(0)
    eng.append(0, toks(rng, 64))
    eng.append(0, toks(rng, 64))
    call(eng, 0)
    eng.remove(0, 1, 2)                                  # blocks 4..7 dead
    v, s = eng.select_victims(HBM, 6)
    assert list(s) == [0, 0, 0, 0, 1, 1]
    rc, n_done, n_dropped = eng.offload(v)
    assert (rc, n_done, n_dropped) == (0, 6, 4)
    st = eng.get_stats()
    assert (st["occ_hbm"], st["occ_host"], st["dropped"], st["offloaded"]) == (2, 2, 4, 2)
    assert st["bytes_d2h"] == 2 * eng.block_bytes
    a = eng.map_blocks([0], LOOKUP)[0]
    assert (a["n_blocks"], a["hit_len"], a["n_hit_hbm"], a["n_hit_host"]) == (4, 4, 2, 2)
    eng.prefill_done(0)


def compaction(make):
    eng = make(n_hbm_blocks=16, n_host_blocks=4, max_contexts=4, **TOY)
    rng = np.random.default_rng(8)
    eng.spawn(0)
    eng.append(0, toks(rng, 16 * 12))
    call(eng, 0)
    keys, _, slot = eng.get_block_map(0)
    for k, s in zip(keys, slot):
        eng.write_block(HBM, int(s), _payload(k, eng.block_bytes))
    eng.release(HBM, [1, 4, 5, 10])
    n_moved = eng.compact(HBM)                           # 8 occupied; movers 8, 9, 11 -> holes 1, 4, 5
    assert n_moved == 3
    ent = eng.get_entries(HBM)
    assert np.all(ent["key"][:8] != 0) and np.all(ent["key"][8:] == 0)
    assert [int(ent["key"][h]) for h in (1, 4, 5)] == [int(keys[m]) for m in (8, 9, 11)]
    assert [int(ent["depth"][h]) for h in (1, 4, 5)] == [8, 9, 11]
    for s in range(8):
        assert np.array_equal(eng.read_block(HBM, s), _payload(int(ent["key"][s]), eng.block_bytes))
    assert eng.compact(HBM) == 0


def raw_copy_blocks(make):
    for layout in (0, 1):
        eng = make(n_hbm_blocks=10, n_host_blocks=10, max_contexts=2, pool_layout=layout, **TOY)
        for s in range(10):
            eng.write_block(HBM, s, _payload(1000 + s, eng.block_bytes))
        eng.copy_blocks(HBM, [3, 9, 0], HOST, [5, 1, 8])
        for s, d in ((3, 5), (9, 1), (0, 8)):
            assert np.array_equal(eng.read_block(HOST, d), _payload(1000 + s, eng.block_bytes))
        eng.copy_blocks(HOST, [5, 8], HBM, [6, 7])
        assert np.array_equal(eng.read_block(HBM, 6), _payload(1003, eng.block_bytes))
        assert np.array_equal(eng.read_block(HBM, 7), _payload(1000, eng.block_bytes))
        eng.copy_blocks(HBM, [1, 2], HBM, [4, 5])
        assert np.array_equal(eng.read_block(HBM, 4), _payload(1001, eng.block_bytes))
        assert np.array_equal(eng.read_block(HBM, 3), _payload(1003, eng.block_bytes))   # untouched
        eng.copy_blocks(HBM, [], HOST, [])                                                # empty list


# ---- admission under a full pool; batch semantics ---------------------------------------------------
def admission_stops_when_full(make):
    eng = make(n_hbm_blocks=6, n_host_blocks=4, max_contexts=4, **TOY)
    rng = np.random.default_rng(10)
    shared = toks(rng, 32)
    for c in (0, 1, 2):
        eng.spawn(c)
        eng.append(c, shared)
        eng.append(c, toks(rng, 48))
    info = eng.map_blocks([0, 1, 2], LOOKUP)
    assert [int(i["n_blocks"]) for i in info] == [5, 5, 5] and [int(i["hit_len"]) for i in info] == [0, 0, 0]
    adm = eng.map_blocks([0, 1, 2], ADMIT)
    # context 0 inserts 5 (slots 0..4); context 1 adopts the 2 shared blocks, inserts 1 (slot 5), then
    # the pool is full; context 2 adopts the 2 shared blocks and stops at its first absent block
    assert [int(i["n_admitted"]) for i in adm] == [5, 3, 2]
    assert [int(i["n_held"]) for i in adm] == [5, 3, 2]
    ent = eng.get_entries(HBM)
    assert list(ent["inflight"]) == [3, 3, 1, 1, 1, 1]
    assert list(ent["depth"]) == [0, 1, 2, 3, 4, 2]
    assert list(eng.get_block_map(1)[2][:3]) == [0, 1, 5]
    st = eng.get_stats()
    assert (st["inserted"], st["adopted"], st["occ_hbm"]) == (6, 4, 6)
    # nothing evictable while everything is in flight; afterwards ADMIT can continue
    assert len(eng.select_victims(HBM, 6)[0]) == 0
    eng.prefill_done(0)
    assert list(eng.get_entries(HBM)["inflight"]) == [2, 2, 0, 0, 0, 1]
    v, s = eng.select_victims(HBM, 2)
    assert list(v) == [4, 3] and list(s) == [1, 1]       # same stamp: chain tail first
    rc, n_done, n_dropped = eng.offload(v)
    assert (rc, n_done, n_dropped) == (0, 2, 0)
    adm = eng.map_blocks([1, 2], ADMIT)
    assert [int(i["n_admitted"]) for i in adm] == [2, 0] and [int(i["n_held"]) for i in adm] == [5, 2]
    eng.prefill_done(1)
    eng.prefill_done(2)
    assert int(eng.get_entries(HBM)["inflight"].sum()) == 0


def lookup_locks_and_orphans(make):
    eng = make(n_hbm_blocks=8, n_host_blocks=4, max_contexts=4, **TOY)
    rng = np.random.default_rng(12)
    eng.spawn(0)
    eng.append(0, toks(rng, 96))                         # 6 blocks
    call(eng, 0)
    eng.release(HBM, [2])                                # hole in the chain: 3,4,5 become unreachable orphans
    a = eng.map_blocks([0], LOOKUP)[0]
    assert (a["hit_len"], a["n_admissible"]) == (2, 4)
    assert list(eng.get_entries(HBM)["inflight"][:6]) == [1, 1, 0, 0, 0, 0]
    b = eng.map_blocks([0], ADMIT)[0]
    assert (b["n_admitted"], b["n_held"]) == (4, 6)      # block 2 re-inserted at slot 2, orphans adopted
    st = eng.get_stats()
    assert (st["inserted"], st["adopted"]) == (7, 3)
    assert list(eng.get_entries(HBM)["inflight"][:6]) == [1] * 6
    # a hit on a dead block is still a hit (content-addressed) and the block revives
    eng.prefill_done(0)
    eng.terminate(0)
    assert states(eng)[:6] == [DEAD] * 6
    eng.spawn(1)
    rng = np.random.default_rng(12)                      # a new context with the same tokens
    eng.append(1, toks(rng, 96))
    a = eng.map_blocks([1], LOOKUP)[0]
    assert a["hit_len"] == 6
    assert states(eng)[:6] == [ACTIVE] * 6
    eng.prefill_done(1)


# ---- error codes -----------------------------------------------------------------------------------
def error_codes(make, op_codes):
    OP = op_codes
    eng = make(n_hbm_blocks=8, n_host_blocks=2, max_contexts=4, **TOY)
    rng = np.random.default_rng(13)
    assert eng.apply_op_rc(OP["APPEND"], 0, tokens=toks(rng, 4)) == E_NOCTX
    assert eng.apply_op_rc(OP["SPAWN"], 9) == E_INVAL    # id out of range
    eng.spawn(0)
    assert eng.apply_op_rc(OP["SPAWN"], 0) == E_INVAL    # id in use
    assert eng.apply_op_rc(77, 0) == E_INVAL and eng.apply_op_rc(0, 0) == E_INVAL
    eng.append(0, toks(rng, 40))
    assert eng.apply_op_rc(OP["REMOVE"], 0, msg_start=0, msg_end=2) == E_RANGE
    assert eng.apply_op_rc(OP["REMOVE"], 0, msg_start=1, msg_end=1) == E_RANGE
    assert eng.apply_op_rc(OP["REPLACE"], 0, msg_start=1, msg_end=2, tokens=toks(rng, 4)) == E_RANGE
    assert eng.apply_op_rc(OP["ONE_OFF"], 0, msg_start=0, msg_end=5) == E_RANGE
    assert eng.apply_op_rc(OP["PIN"], 0, msg_start=0, msg_end=2) == E_RANGE
    assert eng.apply_op_rc(OP["UNPIN"], 0, msg_start=1, msg_end=1) == E_RANGE
    assert eng.apply_op_rc(OP["PIN"], 2, msg_start=0, msg_end=1) == E_NOCTX
    assert eng.apply_op_rc(OP["FORK"], 1, parent=0, msg_end=2) == E_RANGE
    assert eng.apply_op_rc(OP["FORK"], 1, parent=3, msg_end=0) == E_NOCTX
    assert eng.apply_op_rc(OP["FORK"], 0, parent=0, msg_end=0) == E_INVAL
    assert eng.apply_op_rc(OP["PREFILL_DONE"], 0) == E_STATE
    assert eng.map_blocks_rc([0], ADMIT)[0] == E_STATE
    assert eng.map_blocks_rc([0, 0], LOOKUP)[0] == E_INVAL
    assert eng.map_blocks_rc([0, 2], LOOKUP)[0] == E_NOCTX
    assert eng.get_stats()["clock"] == 0                 # rejected calls change nothing
    eng.map_blocks([0], LOOKUP)
    assert eng.map_blocks_rc([0], LOOKUP)[0] == E_STATE
    for op in ("APPEND", "REPLACE", "REMOVE", "ONE_OFF", "PIN", "UNPIN"):
        assert eng.apply_op_rc(OP[op], 0, msg_start=0, msg_end=1, tokens=toks(rng, 4)) == E_STATE
    assert eng.apply_op_rc(OP["FORK"], 1, parent=0, msg_end=1) == E_STATE
    eng.map_blocks([0], ADMIT)                           # 2 blocks at slots 0, 1, in flight
    assert eng.offload([0])[0] == E_STATE
    assert eng.release_rc(HBM, [1]) == E_STATE
    assert eng.offload([5])[0] == E_INVAL                # empty slot
    assert eng.offload([8])[0] == E_RANGE
    eng.prefill_done(0)
    assert eng.offload([0, 0])[0] == E_INVAL             # repeated slot
    assert eng.offload([0, 9, 5])[0] == E_RANGE          # range errors win over the others
    assert eng.reload([0])[0] == E_INVAL
    assert eng.release_rc(HOST, [3]) == E_RANGE
    st = eng.get_stats()
    assert (st["occ_hbm"], st["occ_host"], st["dropped"]) == (2, 0, 0)
    assert eng.debug_load_resident_rc([1], [0], [0], [0], [3], HBM) == E_INVAL        # reserved key value
    assert eng.debug_load_resident_rc([50, 50], [0, 0], [0, 0], [0, 0], [3, 4], HBM) == E_INVAL
    assert eng.debug_load_resident_rc([50], [0], [0], [0], [0], HBM) == E_INVAL       # slot occupied
    assert eng.debug_load_resident_rc([int(eng.get_entries(HBM)["key"][0])], [0], [0], [0], [3], HBM) == E_INVAL
    eng.terminate(0)
    assert eng.apply_op_rc(OP["APPEND"], 0, tokens=toks(rng, 4)) == E_NOCTX
    eng.spawn(0)                                         # a terminated id can be reused


# ---- zero-length and sub-block inputs ----------------------------------------------------------------
def degenerate_inputs(make):
    eng = make(n_hbm_blocks=8, n_host_blocks=2, max_contexts=4, **TOY)
    rng = np.random.default_rng(14)
    eng.spawn(0)
    a, b = call(eng, 0)                                  # empty context
    assert (a["n_blocks"], a["hit_len"], a["n_admissible"], b["n_held"]) == (0, 0, 0, 0)
    eng.append(0, toks(rng, 15))                         # no full block
    a, b = call(eng, 0)
    assert a["n_blocks"] == 0
    eng.append(0, toks(rng, 0))                          # empty message
    eng.append(0, toks(rng, 1))                          # completes block 0
    a, b = call(eng, 0)
    assert (a["n_blocks"], b["n_admitted"]) == (1, 1)
    assert states(eng)[0] == IDLE
    eng.remove(0, 1, 2)                                  # removing the empty message (starts at token 15)
    assert states(eng)[0] == DEAD                        # cut = floor(15/16) = 0
    assert len(eng.select_victims(HBM, 0)[0]) == 0
    assert eng.offload([])[:2] == (0, 0)
    assert eng.reload([])[:2] == (0, 0)
    keys, tier, slot = eng.get_block_map(0)
    assert len(keys) == 1


# ---- reachability-aware classification: blocks behind a missing prefix block are dead ----------------
def orphans_are_dead(make):
    for flags in (0, 4):
        eng = make(n_hbm_blocks=12, n_host_blocks=4, max_contexts=4, policy_flags=flags, **TOY)
        rng = np.random.default_rng(21)
        eng.spawn(0)
        eng.append(0, toks(rng, 96))                     # 6 blocks at slots 0..5
        call(eng, 0)
        eng.fork(0, 1, 1)                                # the child shares all six and adds two of its own (6, 7)
        eng.append(1, toks(rng, 32))
        call(eng, 1)
        eng.pin(1, 1, 2)                                 # the child's own message is pinned
        assert states(eng)[:8] == [IDLE] * 6 + [PINNED] * 2
        assert eng.offload([1]) == (0, 1, 0)             # a block on the host tier still counts as present
        assert states(eng)[:8] == [IDLE, FREE] + [IDLE] * 4 + [PINNED] * 2 and states(eng, HOST)[0] == IDLE
        eng.release(HBM, [2])                            # block 2 is gone from every tier
        want = [IDLE, FREE, FREE] + ([DEAD] * 5 if flags else [IDLE] * 3 + [PINNED] * 2)
        assert states(eng)[:8] == want                   # pinned or not: nothing behind the hole can be hit again
        v, s = eng.select_victims(HBM, 5)
        if flags:
            assert list(v) == [7, 6, 5, 4, 3] and list(s) == [DEAD] * 5      # first victims, deepest first
            assert eng.offload(v[:2]) == (0, 2, 2)       # and dropped, not copied
        else:
            assert list(s) == [IDLE] * 4 and set(v) == {0, 3, 4, 5}
        # the parent's next call re-creates block 2 and adopts what is still there: everything is reachable again
        a = eng.map_blocks([0], LOOKUP)[0]
        assert (a["hit_len"], a["n_hit_hbm"], a["n_hit_host"]) == (2, 1, 1)
        assert states(eng)[:6] == [ACTIVE, FREE, FREE] + ([DEAD] * 3 if flags else [ACTIVE] * 3)
        b = eng.map_blocks([0], ADMIT)[0]
        assert (b["n_admitted"], b["n_held"]) == (4, 6)
        assert states(eng)[:6] == [ACTIVE, ACTIVE, FREE] + [ACTIVE] * 3     # block 2 re-created at the lowest free slot (1)
        eng.prefill_done(0)


# ---- three tiers: HBM, host memory, remote memory (Section 7) ------------------------------------------
REMOTE = 2


def three_tiers(make):
    eng = make(n_hbm_blocks=6, n_host_blocks=3, n_remote_blocks=4, max_contexts=4, **TOY)
    rng = np.random.default_rng(22)
    eng.spawn(0)
    eng.append(0, toks(rng, 96))
    call(eng, 0)                                         # blocks 0..5 at HBM slots 0..5
    keys = eng.get_block_map(0)[0]
    for b in range(6):
        eng.write_block(HBM, b, _payload(keys[b], eng.block_bytes))
    assert eng.offload([5, 4, 3]) == (0, 3, 0)           # host slots 0, 1, 2 hold blocks 5, 4, 3
    v, s = eng.select_victims(HOST, 2)                   # same stamp everywhere: the chain's tail goes first
    assert list(v) == [0, 1] and list(s) == [IDLE, IDLE]
    assert eng.move(HOST, REMOTE, v) == (0, 2, 0)        # remote slots 0 (block 5) and 1 (block 4)
    st = eng.get_stats()
    assert (st["occ_hbm"], st["occ_host"], st["occ_remote"], st["demoted"]) == (3, 1, 2, 2)
    assert states(eng, REMOTE) == [IDLE, IDLE, FREE, FREE]
    a = eng.map_blocks([0], LOOKUP)[0]
    assert (a["hit_len"], a["n_hit_hbm"], a["n_hit_host"], a["n_hit_remote"]) == (6, 3, 1, 2)
    _k, tier, slot = eng.get_block_map(0)
    assert list(tier) == [0, 0, 0, 1, 2, 2] and list(slot) == [0, 1, 2, 2, 1, 0]
    assert states(eng, REMOTE)[:2] == [ACTIVE, ACTIVE]
    assert eng.move(HOST, REMOTE, [2])[0] < 0            # a block in flight does not move down
    assert eng.move(REMOTE, HBM, [1, 0]) == (0, 2, 0)    # straight up: block 4 -> HBM slot 3, block 5 -> slot 4
    assert eng.reload([2]) == (0, 1)                     # block 3 -> HBM slot 5
    _k, tier, slot = eng.get_block_map(0)
    assert list(tier) == [0] * 6 and list(slot) == [0, 1, 2, 5, 3, 4]
    for b in range(6):
        assert np.array_equal(eng.read_block(HBM, int(slot[b])), _payload(keys[b], eng.block_bytes)), b
    st = eng.get_stats()
    assert (st["occ_hbm"], st["occ_host"], st["occ_remote"], st["promoted"], st["reloaded"]) == (6, 0, 0, 2, 1)
    eng.map_blocks([0], ADMIT)
    eng.prefill_done(0)
    # down again, one level at a time, then one level up; dead blocks are dropped on the way down
    assert eng.offload([4, 3]) == (0, 2, 0)              # blocks 5, 4 -> host slots 0, 1
    assert eng.move(HOST, REMOTE, [0, 1]) == (0, 2, 0)   # -> remote slots 0, 1
    assert eng.move(REMOTE, HOST, [1]) == (0, 1, 0)      # block 4 back to host slot 0
    assert states(eng, HOST) == [IDLE, FREE, FREE] and states(eng, REMOTE) == [IDLE, FREE, FREE, FREE]
    assert np.array_equal(eng.read_block(HOST, 0), _payload(keys[4], eng.block_bytes))
    assert np.array_equal(eng.read_block(REMOTE, 0), _payload(keys[5], eng.block_bytes))
    eng.remove(0, 0, 1)                                  # everything dies
    assert eng.move(HOST, REMOTE, [0]) == (0, 1, 1)      # dropped, not copied
    v, s = eng.select_victims(REMOTE, 4)
    assert list(v) == [0] and list(s) == [DEAD]
    eng.release(REMOTE, v)
    st = eng.get_stats()
    assert (st["occ_host"], st["occ_remote"], st["promoted"], st["demoted"]) == (0, 0, 3, 4)
    # pairs that skip a level on the way down, and bad slots, are rejected
    assert eng.move(HBM, REMOTE, [0])[0] < 0 and eng.move(REMOTE, REMOTE, [0])[0] < 0
    assert eng.move(REMOTE, HOST, [0])[0] < 0 and eng.move(REMOTE, HOST, [9])[0] < 0
    # the remote tier fills up: the move stops there and reports how far it got
    eng.release(HBM, [0, 1, 2, 5])                       # the dead blocks 0..3 of the first context
    eng.spawn(1)
    eng.append(1, toks(rng, 96))
    call(eng, 1)                                         # six new blocks at HBM slots 0..5
    assert eng.offload([0, 1, 2]) == (0, 3, 0)
    assert eng.move(HOST, REMOTE, [0, 1, 2]) == (0, 3, 0)
    assert eng.offload([3, 4, 5]) == (0, 3, 0)
    rc, n_done, n_dropped = eng.move(HOST, REMOTE, [0, 1, 2])
    assert rc < 0 and (n_done, n_dropped) == (1, 0)      # one remote slot was left
    assert eng.get_stats()["occ_remote"] == 4


# ---- destinations of a downward move = the slots free when the call begins (hand-worked) -----------------------
def offload_destinations_are_fixed_at_call_begin(make):
    """Inclusive tiers, one offload call that lists a dead block WITH a clean host copy ahead of a live block without
    one. Dropping the dead block frees its copy's host slot (slot 0) in the middle of the call; the live block must
    still go to the lowest slot that was free when the call began (slot 1), not to the slot the call itself freed."""
    eng = make(n_hbm_blocks=6, n_host_blocks=6, max_contexts=4, policy_flags=2, **TOY)
    rng = np.random.default_rng(31)
    eng.spawn(0)
    eng.append(0, toks(rng, 64))
    call(eng, 0)                                         # ctx 0: blocks 0..3 at HBM slots 0..3
    eng.spawn(1)
    eng.append(1, toks(rng, 32))
    call(eng, 1)                                         # ctx 1: blocks 0, 1 at HBM slots 4, 5
    k0 = eng.get_block_map(0)[0]
    k1 = eng.get_block_map(1)[0]
    for s, k in ((3, k0[3]), (4, k1[0]), (5, k1[1])):
        eng.write_block(HBM, s, _payload(k, eng.block_bytes))
    assert eng.offload([3]) == (0, 1, 0)                 # ctx 0's last block -> host slot 0
    a = eng.map_blocks([0], LOOKUP)[0]
    assert (a["hit_len"], a["n_hit_hbm"], a["n_hit_host"]) == (4, 3, 1)
    assert eng.reload([0]) == (0, 1)                     # back to HBM slot 3; host slot 0 keeps the clean copy
    eng.map_blocks([0], ADMIT)
    eng.prefill_done(0)
    eng.terminate(0)                                     # ctx 0's blocks are dead now, slot 3 still has its copy
    assert states(eng) == [DEAD] * 4 + [IDLE] * 2
    assert states(eng, HOST) == [SHADOW] + [FREE] * 5
    # the call: dead-with-copy first, then two live blocks
    assert eng.offload([3, 4, 5]) == (0, 3, 1)
    assert states(eng) == [DEAD] * 3 + [FREE] * 3
    assert states(eng, HOST) == [FREE, IDLE, IDLE, FREE, FREE, FREE]      # slot 0 was not free when the call began
    _k, tier, slot = eng.get_block_map(1)
    assert list(tier) == [HOST, HOST] and list(slot) == [1, 2]
    assert np.array_equal(eng.read_block(HOST, 1), _payload(k1[0], eng.block_bytes))
    assert np.array_equal(eng.read_block(HOST, 2), _payload(k1[1], eng.block_bytes))
    st = eng.get_stats()
    assert (st["occ_hbm"], st["occ_host"], st["dropped"]) == (3, 2, 1)
    # the next call does see slot 0 as free
    eng.spawn(2)
    eng.append(2, toks(rng, 16))
    call(eng, 2)                                         # one block at HBM slot 3 (lowest free)
    assert eng.offload([3]) == (0, 1, 0)
    assert list(eng.get_block_map(2)[1]) == [HOST] and list(eng.get_block_map(2)[2]) == [0]


def move_down_with_a_dead_block_ahead(make):
    """kvt_move(host -> remote) with a dead block listed ahead of live ones: the dead one is dropped without taking a
    remote slot, the live ones take the lowest remote slots in list order. (No drop of such a call can free a remote
    slot, so the slots free at call begin and the slots free at each step are the same set here.)"""
    eng = make(n_hbm_blocks=6, n_host_blocks=4, n_remote_blocks=4, max_contexts=4, **TOY)
    rng = np.random.default_rng(32)
    eng.spawn(0)
    eng.append(0, toks(rng, 32))
    call(eng, 0)                                         # ctx 0: HBM slots 0, 1
    eng.spawn(1)
    eng.append(1, toks(rng, 48))
    call(eng, 1)                                         # ctx 1: HBM slots 2, 3, 4
    k1 = eng.get_block_map(1)[0]
    for b in range(3):
        eng.write_block(HBM, 2 + b, _payload(k1[b], eng.block_bytes))
    assert eng.offload([0, 2, 3, 4]) == (0, 4, 0)        # host slot 0: ctx 0 block 0; slots 1, 2, 3: ctx 1 blocks 0, 1, 2
    assert eng.offload([1]) == (-5, 0, 0)                # host tier full
    eng.release(HBM, [1])
    # a remote slot is taken first so that "lowest free" is not slot 0
    assert eng.move(HOST, REMOTE, [3]) == (0, 1, 0)      # ctx 1 block 2 -> remote slot 0
    eng.terminate(0)                                     # host slot 0 is dead now
    assert states(eng, HOST) == [DEAD, IDLE, IDLE, FREE]
    assert eng.move(HOST, REMOTE, [0, 2, 1]) == (0, 3, 1)    # dead dropped; block 1 -> remote 1, block 0 -> remote 2
    assert states(eng, HOST) == [FREE] * 4
    assert states(eng, REMOTE) == [IDLE, IDLE, IDLE, FREE]
    _k, tier, slot = eng.get_block_map(1)
    assert list(tier) == [REMOTE] * 3 and list(slot) == [2, 1, 0]
    for b in range(3):
        assert np.array_equal(eng.read_block(REMOTE, int(slot[b])), _payload(k1[b], eng.block_bytes))
    st = eng.get_stats()
    assert (st["occ_host"], st["occ_remote"], st["demoted"]) == (0, 3, 3)


# ---- recency stamps of a context that ends while its call is in flight (hand-worked) ----------------------------
def stamps_of_a_call_that_is_terminated_in_flight(make):
    """A block is stamped when a lookup hits it, when an admission inserts or adopts it and at PREFILL_DONE of a holder
    (Section 6.2: the order of cache events). TERMINATE of an in-flight context releases its locks and stamps
    nothing (Section 6.1: reclaimed once in-flight use completes). Clock values are worked out by hand below."""
    eng = make(n_hbm_blocks=16, n_host_blocks=4, max_contexts=4, **TOY)
    rng = np.random.default_rng(33)
    eng.spawn(0)
    eng.append(0, toks(rng, 80))
    call(eng, 0)                                         # lookup: clock 1; done: clock 2. Slots 0..4 stamp 2
    eng.spawn(1)
    eng.append(1, toks(rng, 32))
    call(eng, 1)                                         # clock 3, 4. Slots 5, 6 stamp 4
    assert list(eng.get_entries(HBM)["stamp"][:7]) == [2] * 5 + [4] * 2
    eng.release(HBM, [2])                                # ctx 0's blocks 3, 4 are now behind a hole
    a = eng.map_blocks([0], LOOKUP)[0]                   # clock 5: blocks 0, 1 hit
    assert (a["hit_len"], a["n_admissible"]) == (2, 3)
    assert list(eng.get_entries(HBM)["stamp"][:5]) == [5, 5, 0, 2, 2]
    b = eng.map_blocks([0], ADMIT)[0]                    # block 2 inserted at slot 2, blocks 3, 4 adopted
    assert (b["n_admitted"], b["n_held"]) == (3, 5)
    ent = eng.get_entries(HBM)
    assert list(ent["stamp"][:5]) == [5] * 5 and list(ent["inflight"][:5]) == [1] * 5
    eng.spawn(2)
    eng.append(2, toks(rng, 16))
    call(eng, 2)                                         # clock 6, 7. Slot 7 stamp 7
    eng.spawn(3)
    eng.append(3, toks(rng, 16))
    call(eng, 3)                                         # clock 8, 9. Slot 8 stamp 9
    eng.terminate(0)                                     # in flight: locks released, no stamp, clock stays 9
    ent = eng.get_entries(HBM)
    assert list(ent["stamp"][:9]) == [5, 5, 5, 5, 5, 4, 4, 7, 9]
    assert list(ent["inflight"][:9]) == [0] * 9
    assert eng.get_stats()["clock"] == 9
    eng.terminate(1)
    eng.terminate(2)
    assert states(eng)[:9] == [DEAD] * 8 + [IDLE]
    v, s = eng.select_victims(HBM, 16)
    # dead, oldest stamp first, deeper block first inside one stamp: ctx 1 (stamp 4), ctx 0 (stamp 5), ctx 2 (7); then idle
    assert list(v) == [6, 5, 4, 3, 2, 1, 0, 7, 8]
    assert list(s) == [DEAD] * 8 + [IDLE]


ALL = [state_machine_single_context, suffix_invalidation, fork_and_shared_kv, one_off_bypass, worked_example,
       mixed_pool_example, victim_order_bruteforce, one_state_pools_reduce_to_lru, offload_reload_round_trip,
       dead_victims_are_dropped_without_copy, compaction, raw_copy_blocks, admission_stops_when_full,
       lookup_locks_and_orphans, degenerate_inputs, pinned_retention, no_lifecycle_policy, inclusive_tiers, exchange_both_ways,
       orphans_are_dead, three_tiers, offload_destinations_are_fixed_at_call_begin, move_down_with_a_dead_block_ahead,
       stamps_of_a_call_that_is_terminated_in_flight]
