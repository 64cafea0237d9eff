"""ctypes front end of the CPU oracle (oracle/kvt_oracle.cpp).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only tests, the smoke check and the benchmark's CPU-baseline
leg may import this module. It imports nothing from the CUDA package and the CUDA package imports
nothing from here. Payload pools are numpy arrays in ordinary host memory.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kvt_oracle.cpp")
# KVT_ORACLE_SANITIZE=1: a separate build with AddressSanitizer and UndefinedBehaviorSanitizer (the process must
# then run with the ASan runtime preloaded; the sanitizer test starts such a process)
_SANITIZE = os.environ.get("KVT_ORACLE_SANITIZE") == "1"
_LIB = os.path.join(_HERE, "libkvt_oracle_asan.so" if _SANITIZE else "libkvt_oracle.so")

OK, E_INVAL, E_NOCTX, E_RANGE, E_STATE, E_NOSPACE, E_BUFSZ = 0, -1, -2, -3, -4, -5, -6
TIER_HBM, TIER_HOST, TIER_REMOTE, TIER_NONE = 0, 1, 2, 0xFF
LAYOUT_LAYER_MAJOR, LAYOUT_BLOCK_MAJOR = 0, 1
ORDER_MRU, ORDER_LRU = 0, 1
POLICY_NO_LIFECYCLE, POLICY_INCLUSIVE = 1, 2
(OP_SPAWN, OP_FORK, OP_APPEND, OP_REPLACE, OP_REMOVE, OP_ONE_OFF, OP_PREFILL_DONE, OP_TERMINATE,
 OP_PIN, OP_UNPIN) = range(1, 11)
MAP_LOOKUP, MAP_ADMIT = 0, 1


class OracleError(RuntimeError):
    def __init__(self, code, what):
        super().__init__(f"{what}: status {code}")
        self.code = code


def build(force: bool = False) -> str:
    """Compiles the oracle with g++ (plain -O2, one thread) if the library is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        flags = ["-O1", "-g", "-fsanitize=address,undefined", "-fno-sanitize-recover=undefined", "-fno-omit-frame-pointer"] \
            if _SANITIZE else ["-O2"]
        subprocess.check_call(["g++"] + flags + ["-std=c++17", "-shared", "-fPIC", "-pthread", "-o", _LIB, _SRC])
    return _LIB


class _Config(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("n_layers", "n_kv_heads", "head_dim", "elem_bytes", "pool_layout",
                                           "n_hbm_blocks", "n_host_blocks", "max_contexts", "suspended_order",
                                           "policy_flags")] + \
               [("hash_seed", C.c_uint64), ("hbm_pool", C.c_void_p), ("host_pool", C.c_void_p),
                ("n_remote_blocks", C.c_uint32), ("pad", C.c_uint32), ("remote_pool", C.c_void_p)]


class _Op(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("op", "ctx", "parent", "msg_start", "msg_end", "n_tokens", "flags",
                                           "reserved")] + [("tokens", C.c_void_p)]


CALL_INFO_DTYPE = np.dtype([(n, np.uint32) for n in ("n_blocks", "hit_len", "n_hit_hbm", "n_hit_host",
                                                       "n_admissible", "n_admitted", "n_held", "n_pinned",
                                                       "n_hit_remote")])
STATS_FIELDS = ("clock", "n_contexts", "occ_hbm", "occ_host", "blocks_hashed", "hits_hbm", "hits_host", "misses",
                "inserted", "adopted", "dropped", "offloaded", "reloaded", "compacted", "bytes_d2h", "bytes_h2d",
                "bytes_d2d", "table_rebuilds", "tombstones", "kernel_launches", "mover_launches", "mover_ns",
                "mover_bytes", "lookup_ns", "lookup_blocks", "select_ns", "select_slots", "offloaded_clean",
                "blocks_rehashed", "occ_remote", "hits_remote", "demoted", "promoted", "classify_ns", "classify_items")

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.kvto_hash_tokens.argtypes = [C.c_void_p, C.c_uint64, C.c_uint64, C.c_void_p]
        _lib.kvto_hash_constants.argtypes = [C.c_uint64, C.c_uint64, C.c_void_p]
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def _u32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.uint32))


def hash_tokens(tokens, seed: int = 0) -> np.ndarray:
    """Chained block keys of one token sequence (one key per full 16-token block)."""
    tok = _u32(tokens)
    keys = np.zeros(len(tok) // 16, dtype=np.uint64)
    rc = lib().kvto_hash_tokens(_p(tok), len(tok), seed, _p(keys))
    if rc:
        raise OracleError(rc, "hash_tokens")
    return keys


def par_digests(tokens, seed: int = 0, n_threads: int = 1) -> np.ndarray:
    """Block digests d_b of a token sequence, blocks spread over n_threads threads (timing helper)."""
    tok = _u32(tokens)
    out = np.zeros(len(tok) // 16, dtype=np.uint64)
    lib().kvto_par_digests.argtypes = [C.c_void_p, C.c_uint64, C.c_uint64, C.c_void_p, C.c_uint32]
    rc = lib().kvto_par_digests(_p(tok), len(tok), seed, _p(out), n_threads)
    if rc:
        raise OracleError(rc, "par_digests")
    return out


def par_copy_blocks(dst, src, block_bytes, src_ids, dst_ids, n_threads: int = 1):
    """dst[dst_ids[i]] = src[src_ids[i]] for whole blocks (uint8 arrays), over n_threads threads (timing helper)."""
    s, d = _u32(src_ids), _u32(dst_ids)
    lib().kvto_par_copy_blocks.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_void_p, C.c_uint32, C.c_uint32]
    rc = lib().kvto_par_copy_blocks(_p(dst), _p(src), block_bytes, _p(s), _p(d), len(s), n_threads)
    if rc:
        raise OracleError(rc, "par_copy_blocks")


def hash_constants(seed: int = 0, x: int = 0):
    """(K[0..15], P, H0, mix64(x)) as Python ints."""
    out = np.zeros(19, dtype=np.uint64)
    lib().kvto_hash_constants(seed, x, _p(out))
    o = [int(v) for v in out]
    return o[:16], o[16], o[17], o[18]


class OracleEngine:
    """CPU engine with the same method names as the CUDA binding."""

    def __init__(self, n_layers, n_kv_heads, head_dim, elem_bytes=2, pool_layout=LAYOUT_LAYER_MAJOR,
                 n_hbm_blocks=128, n_host_blocks=512, max_contexts=64, hash_seed=0,
                 suspended_order=ORDER_MRU, metadata_only=False, policy_flags=0, n_remote_blocks=0, **_ignored):
        self.L = lib()
        self.n_layers, self.n_kv_heads, self.head_dim, self.elem_bytes = n_layers, n_kv_heads, head_dim, elem_bytes
        self.pool_layout = pool_layout
        self.n_hbm_blocks, self.n_host_blocks, self.n_remote_blocks = n_hbm_blocks, n_host_blocks, n_remote_blocks
        self.chunk_bytes = 16 * n_kv_heads * head_dim * elem_bytes
        self.n_chunks = 2 * n_layers
        self.block_bytes = self.chunk_bytes * self.n_chunks
        self.metadata_only = metadata_only
        if metadata_only:
            self.hbm_pool = self.host_pool = self.remote_pool = None
        else:
            self.hbm_pool = np.zeros(n_hbm_blocks * self.block_bytes, dtype=np.uint8)
            self.host_pool = np.zeros(max(n_host_blocks, 1) * self.block_bytes, dtype=np.uint8)
            self.remote_pool = np.zeros(max(n_remote_blocks, 1) * self.block_bytes, dtype=np.uint8)
        cfg = _Config(n_layers, n_kv_heads, head_dim, elem_bytes, pool_layout, n_hbm_blocks, n_host_blocks,
                      max_contexts, suspended_order, policy_flags, hash_seed,
                      None if metadata_only else self.hbm_pool.ctypes.data,
                      None if metadata_only else self.host_pool.ctypes.data,
                      n_remote_blocks, 0, None if metadata_only else self.remote_pool.ctypes.data)
        h = C.c_void_p()
        rc = self.L.kvto_create(C.byref(cfg), C.byref(h))
        if rc:
            raise OracleError(rc, "create")
        self.h = h

    def close(self):
        if self.h:
            self.L.kvto_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- primitives ---------------------------------------------------------------------------
    def apply_op_rc(self, op, ctx, parent=0, msg_start=0, msg_end=0, tokens=None) -> int:
        tok = _u32(tokens) if tokens is not None else None
        o = _Op(op, ctx, parent, msg_start, msg_end, 0 if tok is None else len(tok), 0, 0,
                None if tok is None else tok.ctypes.data)
        return self.L.kvto_apply_op(self.h, C.byref(o))

    def _op(self, what, *a, **k):
        rc = self.apply_op_rc(*a, **k)
        if rc:
            raise OracleError(rc, what)

    def spawn(self, ctx): self._op("spawn", OP_SPAWN, ctx)
    def fork(self, parent, child, end): self._op("fork", OP_FORK, child, parent=parent, msg_end=end)
    def append(self, ctx, tokens): self._op("append", OP_APPEND, ctx, tokens=_u32(tokens))
    def replace(self, ctx, s, e, tokens): self._op("replace", OP_REPLACE, ctx, msg_start=s, msg_end=e, tokens=_u32(tokens))
    def remove(self, ctx, s, e): self._op("remove", OP_REMOVE, ctx, msg_start=s, msg_end=e)

    def one_off(self, ctx, s=0, e=None):
        self._op("one_off", OP_ONE_OFF, ctx, msg_start=s, msg_end=0xFFFFFFFF if e is None else e)

    def pin(self, ctx, s, e): self._op("pin", OP_PIN, ctx, msg_start=s, msg_end=e)
    def unpin(self, ctx, s, e): self._op("unpin", OP_UNPIN, ctx, msg_start=s, msg_end=e)
    def prefill_done(self, ctx): self._op("prefill_done", OP_PREFILL_DONE, ctx)
    def terminate(self, ctx): self._op("terminate", OP_TERMINATE, ctx)

    # ---- hash / lookup / admit ---------------------------------------------------------------
    def map_blocks_rc(self, ctx_ids, phase):
        ids = _u32(ctx_ids)
        out = np.zeros(len(ids), dtype=CALL_INFO_DTYPE)
        rc = self.L.kvto_map_blocks(self.h, _p(ids), len(ids), phase, _p(out))
        return rc, out

    def map_blocks(self, ctx_ids, phase):
        rc, out = self.map_blocks_rc(ctx_ids, phase)
        if rc:
            raise OracleError(rc, "map_blocks")
        return out

    def get_block_map(self, ctx):
        n = C.c_uint32(0)
        rc = self.L.kvto_get_block_map(self.h, ctx, None, None, None, 0, C.byref(n))
        if rc not in (OK, E_BUFSZ):
            raise OracleError(rc, "get_block_map")
        nb = n.value
        keys = np.zeros(nb, np.uint64); tier = np.zeros(nb, np.uint8); slot = np.zeros(nb, np.uint32)
        rc = self.L.kvto_get_block_map(self.h, ctx, _p(keys), _p(tier), _p(slot), nb, C.byref(n))
        if rc:
            raise OracleError(rc, "get_block_map")
        return keys, tier, slot

    # ---- classify / select ----------------------------------------------------------------------
    def classify(self):
        pass  # the oracle derives states from the definition whenever they are asked for

    def _tier_size(self, tier):
        sizes = (self.n_hbm_blocks, self.n_host_blocks, self.n_remote_blocks)
        return sizes[tier] if 0 <= tier < 3 else 0      # an unknown tier is for the library to reject

    def get_states(self, tier):
        st = np.zeros(self._tier_size(tier), np.uint8)
        rc = self.L.kvto_get_states(self.h, tier, _p(st), len(st))
        if rc:
            raise OracleError(rc, "get_states")
        return st

    def classify_bruteforce(self, tier):
        st = np.zeros(self._tier_size(tier), np.uint8)
        rc = self.L.kvto_classify_bruteforce(self.h, tier, _p(st), len(st))
        if rc:
            raise OracleError(rc, "classify_bruteforce")
        return st

    def select_victims(self, tier, n_req, include_pinned=False):
        cap = min(n_req, self._tier_size(tier))
        slots = np.zeros(cap, np.uint32); states = np.zeros(cap, np.uint8)
        n = C.c_uint32(0)
        rc = self.L.kvto_select_victims(self.h, tier, n_req, 1 if include_pinned else 0, _p(slots), _p(states), cap,
                                        C.byref(n))
        if rc:
            raise OracleError(rc, "select_victims")
        return slots[:n.value].copy(), states[:n.value].copy()

    # ---- movement -------------------------------------------------------------------------------
    def offload(self, slots):
        s = _u32(slots); nd = C.c_uint32(0); nx = C.c_uint32(0)
        rc = self.L.kvto_offload(self.h, _p(s), len(s), C.byref(nd), C.byref(nx))
        return rc, nd.value, nx.value

    def reload(self, slots):
        s = _u32(slots); nd = C.c_uint32(0)
        rc = self.L.kvto_reload(self.h, _p(s), len(s), C.byref(nd))
        return rc, nd.value

    def move(self, src_tier, dst_tier, slots):
        s = _u32(slots); nd = C.c_uint32(0); nx = C.c_uint32(0)
        rc = self.L.kvto_move(self.h, src_tier, dst_tier, _p(s), len(s), C.byref(nd), C.byref(nx))
        return rc, nd.value, nx.value

    def exchange(self, out_slots, in_slots):
        o, i = _u32(out_slots), _u32(in_slots)
        a, b, c = C.c_uint32(0), C.c_uint32(0), C.c_uint32(0)
        rc = self.L.kvto_exchange(self.h, _p(o), len(o), _p(i), len(i), C.byref(a), C.byref(b), C.byref(c))
        return rc, a.value, b.value, c.value

    def release_rc(self, tier, slots):
        s = _u32(slots)
        return self.L.kvto_release(self.h, tier, _p(s), len(s))

    def release(self, tier, slots):
        rc = self.release_rc(tier, slots)
        if rc:
            raise OracleError(rc, "release")

    def compact(self, tier):
        n = C.c_uint32(0)
        rc = self.L.kvto_compact(self.h, tier, C.byref(n))
        if rc:
            raise OracleError(rc, "compact")
        return n.value

    def copy_blocks(self, src_tier, src, dst_tier, dst):
        s, d = _u32(src), _u32(dst)
        rc = self.L.kvto_copy_blocks(self.h, src_tier, _p(s), dst_tier, _p(d), len(s))
        if rc:
            raise OracleError(rc, "copy_blocks")

    # ---- introspection --------------------------------------------------------------------------
    def get_stats(self):
        out = np.zeros(len(STATS_FIELDS), np.uint64)
        self.L.kvto_get_stats(self.h, _p(out))
        return {k: int(v) for k, v in zip(STATS_FIELDS, out)}

    def get_entries(self, tier):
        n = self._tier_size(tier)
        keys = np.zeros(n, np.uint64); stamp = np.zeros(n, np.uint32)
        depth = np.zeros(n, np.uint32); infl = np.zeros(n, np.uint32); link = np.zeros(n, np.uint32)
        rc = self.L.kvto_get_entries(self.h, tier, _p(keys), _p(stamp), _p(depth), _p(infl), _p(link), n)
        if rc:
            raise OracleError(rc, "get_entries")
        return {"key": keys, "stamp": stamp, "depth": depth, "inflight": infl, "link": link}

    def debug_load_resident_rc(self, keys, state, stamp, depth, slot, tier):
        k = np.ascontiguousarray(np.asarray(keys, np.uint64)); st = np.ascontiguousarray(np.asarray(state, np.uint8))
        sp, dp, sl = _u32(stamp), _u32(depth), _u32(slot)
        return self.L.kvto_debug_load_resident(self.h, _p(k), _p(st), _p(sp), _p(dp), _p(sl), tier, len(k))

    def debug_load_resident(self, *a):
        rc = self.debug_load_resident_rc(*a)
        if rc:
            raise OracleError(rc, "debug_load_resident")

    # ---- payload access for the harness (the "prefill" that produces KV is not the engine's job) --
    def _chunks(self, tier, slot):
        if tier == TIER_HBM and self.pool_layout == LAYOUT_LAYER_MAJOR:
            v = self.hbm_pool.reshape(self.n_chunks, self.n_hbm_blocks, self.chunk_bytes)
            return v[:, slot, :]
        pool = (self.hbm_pool, self.host_pool, self.remote_pool)[tier]
        return pool.reshape(-1, self.n_chunks, self.chunk_bytes)[slot]

    def write_block(self, tier, slot, payload):
        self._chunks(tier, slot)[...] = np.asarray(payload, np.uint8).reshape(self.n_chunks, self.chunk_bytes)

    def read_block(self, tier, slot):
        return np.array(self._chunks(tier, slot)).reshape(-1)
