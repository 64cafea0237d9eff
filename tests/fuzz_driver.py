"""Random differential driver: applies the same seeded stream of API calls (valid and invalid) to one or
two engines and compares every status code and, periodically, every observable piece of state."""
import numpy as np

from paper_2609_39819_b200 import workloads as W

HBM, HOST, REMOTE = 0, 1, 2
OPS = ("append", "append", "append", "replace", "remove", "one_off_ctx", "one_off_msg", "pin", "unpin", "fork", "spawn",
       "terminate", "call", "call", "call", "lookup_only", "admit_only", "prefill_done", "evict", "evict_pinned",
       "release_hbm", "release_host", "reload_some", "compact_hbm", "compact_host", "exchange", "exchange", "bad")
OPS_REMOTE = ("demote", "demote", "promote_host", "promote_hbm", "release_remote", "compact_remote", "bad_move")


def tiers(eng):
    return (HBM, HOST, REMOTE) if getattr(eng, "n_remote_blocks", 0) else (HBM, HOST)


def tier_size(eng, tier):
    return (eng.n_hbm_blocks, eng.n_host_blocks, getattr(eng, "n_remote_blocks", 0))[tier]


def payload(key, nbytes):
    return W.payload_pattern(int(key), nbytes)


def observe(eng):
    """Everything an engine lets a caller see, as a comparable structure."""
    out = {"stats": {k: v for k, v in eng.get_stats().items() if k not in W.GPU_ONLY_STATS}}
    for tier in tiers(eng):
        out[f"states{tier}"] = eng.get_states(tier)
        out[f"entries{tier}"] = eng.get_entries(tier)
    return out


def check_payload(eng):
    """Every occupied slot (blocks and clean copies) holds the payload of its key."""
    if eng.metadata_only:
        return True
    for tier in tiers(eng):
        keys = eng.get_entries(tier)["key"]
        for s in np.nonzero(keys)[0]:
            if not np.array_equal(eng.read_block(tier, int(s)), payload(keys[s], eng.block_bytes)):
                return False
    return True


def check_invariants(eng, inclusive):
    st = eng.get_stats()
    ent = [eng.get_entries(t) for t in tiers(eng)]
    states = [eng.get_states(t) for t in tiers(eng)]
    for tier in tiers(eng):
        occ = int((ent[tier]["key"] != 0).sum())
        assert occ == st[("occ_hbm", "occ_host", "occ_remote")[tier]] <= tier_size(eng, tier)
        assert np.all((states[tier] == 0xFF) == (ent[tier]["key"] == 0))
        assert np.all(ent[tier]["inflight"][ent[tier]["key"] == 0] == 0)
    copies = states[HOST] == 0xFE
    if not inclusive:
        assert not copies.any()
    # a clean copy and its block point at each other and hold the same key; every other key is unique
    for h in np.nonzero(copies)[0]:
        b = int(ent[HOST]["link"][h])
        assert int(ent[HBM]["link"][b]) == h and ent[HBM]["key"][b] == ent[HOST]["key"][h]
    prim = np.concatenate([ent[HBM]["key"][ent[HBM]["key"] != 0], ent[HOST]["key"][(ent[HOST]["key"] != 0) & ~copies]] +
                          [ent[t]["key"][ent[t]["key"] != 0] for t in tiers(eng)[2:]])
    assert len(np.unique(prim)) == len(prim)
    assert st["hits_hbm"] + st["hits_host"] + st["hits_remote"] + st["misses"] == st["blocks_hashed"]
    if hasattr(eng, "classify_bruteforce"):
        for tier in tiers(eng):
            assert np.array_equal(states[tier], eng.classify_bruteforce(tier))


class Fuzzer:
    def __init__(self, engines, seed, max_ctx=6, max_tok=90):
        self.engs = engines
        self.rng = np.random.default_rng([77, seed])
        self.max_ctx = max_ctx
        self.max_tok = max_tok
        self.n_msgs = {}            # mirror: live contexts -> message count (retained contexts excluded)
        self.in_flight = set()
        self.log = []

    def toks(self, lo=1):
        n = int(self.rng.integers(lo, self.max_tok + 1))
        return self.rng.integers(0, 50, n, dtype=np.uint32)  # tiny vocabulary: blocks shared across contexts do occur

    def all_rc(self, fn):
        """Calls fn(engine) on every engine; the results must be equal; returns the first."""
        res = [fn(e) for e in self.engs]
        for r in res[1:]:
            assert W.records_equal(res[0], r) is None, (self.log[-3:], res[0], r)
        return res[0]

    def pick_ctx(self, live=True):
        r = self.rng
        if live and self.n_msgs and r.random() < 0.9:
            return int(r.choice(sorted(self.n_msgs)))
        return int(r.integers(0, self.max_ctx))

    def msg_range(self, c):
        n = self.n_msgs.get(c, 0)
        r = self.rng
        if n == 0 or r.random() < 0.07:
            return int(r.integers(0, 3)), int(r.integers(0, 4))        # possibly invalid
        s = int(r.integers(0, n))
        return s, int(r.integers(s + 1, n + 1))

    def step(self):
        r = self.rng
        op = str(r.choice(OPS + OPS_REMOTE if len(tiers(self.engs[0])) == 3 else OPS))
        self.log.append(op)
        E = self.engs[0]
        if op == "spawn":
            c = self.pick_ctx(live=False)
            rc = self.all_rc(lambda e: e.apply_op_rc(1, c))
            if rc == 0:
                self.n_msgs[c] = 0
        elif op == "fork":
            p, c = self.pick_ctx(), self.pick_ctx(live=False)
            end = int(r.integers(0, self.n_msgs.get(p, 0) + 2))
            rc = self.all_rc(lambda e: e.apply_op_rc(2, c, parent=p, msg_end=end))
            if rc == 0:
                self.n_msgs[c] = end
        elif op == "append":
            c, t = self.pick_ctx(), self.toks(0 if r.random() < 0.05 else 1)
            rc = self.all_rc(lambda e: e.apply_op_rc(3, c, tokens=t))
            if rc == 0:
                self.n_msgs[c] = self.n_msgs.get(c, 0) + 1
        elif op in ("replace", "remove"):
            c = self.pick_ctx()
            s, e_ = self.msg_range(c)
            t = self.toks()
            code = 4 if op == "replace" else 5
            rc = self.all_rc(lambda e: e.apply_op_rc(code, c, msg_start=s, msg_end=e_, tokens=t if code == 4 else None))
            if rc == 0:
                self.n_msgs[c] = self.n_msgs.get(c, 0) + (1 if code == 4 else 0) - (e_ - s)
        elif op == "one_off_ctx":
            c = self.pick_ctx()
            self.all_rc(lambda e: e.apply_op_rc(6, c, msg_start=0, msg_end=0xFFFFFFFF))
        elif op in ("one_off_msg", "pin", "unpin"):
            c = self.pick_ctx() if op != "unpin" or r.random() < 0.7 else int(r.integers(0, self.max_ctx))
            s, e_ = self.msg_range(c)
            code = {"one_off_msg": 6, "pin": 9, "unpin": 10}[op]
            self.all_rc(lambda e: e.apply_op_rc(code, c, msg_start=s, msg_end=e_))
        elif op == "terminate":
            c = self.pick_ctx()
            if r.random() < 0.6:
                return
            rc = self.all_rc(lambda e: e.apply_op_rc(8, c))
            if rc == 0:
                self.n_msgs.pop(c, None)
                self.in_flight.discard(c)
        elif op in ("call", "lookup_only", "admit_only"):
            k = int(r.integers(1, 4))
            ctxs = [self.pick_ctx() for _ in range(k)]
            if r.random() < 0.9:
                ctxs = list(dict.fromkeys(ctxs))
            if op != "admit_only":
                rc, info = self.all_rc(lambda e: e.map_blocks_rc(ctxs, 0))
                if rc == 0:
                    self.in_flight |= set(ctxs)
            if op == "call" and r.random() < 0.7:
                need = int(r.integers(0, 8))
                if need:
                    self.evict(need, False)
            if op == "call" and r.random() < 0.7:        # bring the host-tier part of the prefixes back
                hs, rs = [], []
                for c in ctxs:
                    if c in self.n_msgs:
                        try:
                            _k, tier, slot = E.get_block_map(c)
                        except Exception:
                            continue
                        hs += [int(x) for x, t in zip(slot, tier) if t == HOST]
                        rs += [int(x) for x, t in zip(slot, tier) if t == REMOTE]
                if hs:
                    hs = list(dict.fromkeys(hs))
                    self.all_rc(lambda e: e.reload(hs))
                if rs:
                    rs = list(dict.fromkeys(rs))
                    self.all_rc(lambda e: e.move(REMOTE, HBM, rs))
            if op != "lookup_only":
                rc, info = self.all_rc(lambda e: e.map_blocks_rc(ctxs, 1))
                if rc == 0:
                    self.write_new(ctxs, info)
            if op == "call":
                for c in ctxs:
                    if self.all_rc(lambda e: e.apply_op_rc(7, c)) == 0:
                        self.in_flight.discard(c)
        elif op == "prefill_done":
            c = self.pick_ctx()
            if self.all_rc(lambda e: e.apply_op_rc(7, c)) == 0:
                self.in_flight.discard(c)
        elif op in ("evict", "evict_pinned"):
            self.evict(int(r.integers(0, 12)), op == "evict_pinned")
        elif op in ("release_hbm", "release_host"):
            tier = HBM if op == "release_hbm" else HOST
            n = E.n_hbm_blocks if tier == HBM else E.n_host_blocks
            slots = r.integers(0, n + 1, int(r.integers(0, 4)))
            occ = np.nonzero(E.get_entries(tier)["key"])[0]
            if len(occ) and r.random() < 0.7:
                slots = r.choice(occ, size=min(len(occ), int(r.integers(1, 4))), replace=False)
            self.all_rc(lambda e: e.release_rc(tier, slots))
        elif op == "reload_some":
            slots = r.integers(0, E.n_host_blocks + 1, int(r.integers(0, 5)))
            occ = np.nonzero(E.get_entries(HOST)["key"])[0]
            if len(occ) and r.random() < 0.8:
                slots = r.choice(occ, size=min(len(occ), int(r.integers(1, 6))), replace=False)
            self.all_rc(lambda e: e.reload(slots))
        elif op == "exchange":
            occ_h = np.nonzero(E.get_entries(HBM)["key"])[0]
            occ_s = np.nonzero(E.get_entries(HOST)["key"])[0]
            out = r.choice(occ_h, size=min(len(occ_h), int(r.integers(0, 5))), replace=False) if len(occ_h) else []
            inn = r.choice(occ_s, size=min(len(occ_s), int(r.integers(0, 5))), replace=False) if len(occ_s) else []
            if r.random() < 0.1:
                out = list(out) + [int(r.integers(0, E.n_hbm_blocks + 2))]
            self.all_rc(lambda e: e.exchange(out, inn))
        elif op in ("compact_hbm", "compact_host", "compact_remote"):
            tier = {"compact_hbm": HBM, "compact_host": HOST, "compact_remote": REMOTE}[op]
            self.all_rc(lambda e: e.compact(tier))
        elif op in ("demote", "promote_host", "promote_hbm"):
            src, dst = {"demote": (HOST, REMOTE), "promote_host": (REMOTE, HOST), "promote_hbm": (REMOTE, HBM)}[op]
            n = tier_size(E, src)
            slots = r.integers(0, n + 1, int(r.integers(0, 4)))
            occ = np.nonzero(E.get_entries(src)["key"])[0]
            if len(occ) and r.random() < 0.85:
                slots = r.choice(occ, size=min(len(occ), int(r.integers(1, 6))), replace=False)
            if op == "demote" and r.random() < 0.5:       # the usual way down: the host tier's own victims
                k = int(r.integers(1, 6))
                slots, _s = self.all_rc(lambda e: e.select_victims(HOST, k))
            self.all_rc(lambda e: e.move(src, dst, slots))
        elif op == "release_remote":
            occ = np.nonzero(E.get_entries(REMOTE)["key"])[0]
            slots = r.choice(occ, size=min(len(occ), int(r.integers(1, 4))), replace=False) if len(occ) else [0]
            self.all_rc(lambda e: e.release_rc(REMOTE, slots))
        elif op == "bad_move":
            src, dst = [(HBM, REMOTE), (REMOTE, REMOTE), (HBM, HBM), (3, 0), (HOST, HOST)][int(r.integers(0, 5))]
            self.all_rc(lambda e: e.move(src, dst, [0]))
        elif op == "bad":
            which = int(r.integers(0, 4))
            if which == 0:
                self.all_rc(lambda e: e.apply_op_rc(int(r.integers(11, 40)), 0))
            elif which == 1:
                self.all_rc(lambda e: e.offload([0, 0]))
            elif which == 2:
                self.all_rc(lambda e: e.map_blocks_rc([0, 0], 0)[0])
            else:
                self.all_rc(lambda e: e.offload([E.n_hbm_blocks + 3]))

    def evict(self, n, pinned):
        v, s = self.all_rc(lambda e: e.select_victims(HBM, n, include_pinned=pinned))
        if len(v) == 0:
            return
        E = self.engs[0]
        need_host = int((((s & 0x7F) > 0) & ((s & 0x80) == 0)).sum())
        free_host = E.n_host_blocks - E.get_stats()["occ_host"]
        if need_host > free_host and self.rng.random() < 0.8:
            hv, hs = self.all_rc(lambda e: e.select_victims(HOST, need_host - free_host))
            if len(hv):
                self.all_rc(lambda e: e.release_rc(HOST, hv))
        self.all_rc(lambda e: e.offload(v))

    def write_new(self, ctxs, info):
        for e in self.engs:
            if e.metadata_only:
                continue
            for c, inf in zip(ctxs, info):
                keys, tier, slot = e.get_block_map(c)
                for b in range(int(inf["n_held"]) - int(inf["n_admitted"]), int(inf["n_held"])):
                    if tier[b] == HBM:
                        e.write_block(HBM, int(slot[b]), payload(keys[b], e.block_bytes))


def run(engines, seed, steps=250, inclusive=False, check_every=10, invariants=True, max_tok=90):
    f = Fuzzer(engines, seed, max_tok=max_tok)
    for i in range(steps):
        f.step()
        if (i + 1) % check_every == 0 or i == steps - 1:
            obs = [observe(e) for e in engines]
            for o in obs[1:]:
                d = W.records_equal(obs[0], o, f"seed {seed} step {i} after {f.log[-check_every:]}")
                assert d is None, d
            for e in engines:
                assert check_payload(e), (seed, i, f.log[-check_every:])
            if invariants:
                check_invariants(engines[-1], inclusive)
    return f
