"""Thin ctypes binding of libkvt.so: argument marshalling only. Every stage of the path (hashing,
table lookup, classification, victim selection, block movement) runs in the library's CUDA kernels.
PyTorch is used for device / pinned memory and streams, nothing else. There is no CPU fallback:
loading fails loudly when the library or a CUDA device is missing."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libkvt.so")
# KVT_LIB=<path>: load another build of the same sources instead (the checked build libkvt_debug.so, a traced build)
ALT_LIB = os.environ.get("KVT_LIB")

OK, E_INVAL, E_NOCTX, E_RANGE, E_STATE, E_NOSPACE, E_BUFSZ, E_DEVICE, E_CUDA = 0, -1, -2, -3, -4, -5, -6, -7, -8
TIER_HBM, TIER_HOST, TIER_REMOTE, TIER_NONE = 0, 1, 2, 0xFF
LAYOUT_LAYER_MAJOR, LAYOUT_BLOCK_MAJOR = 0, 1
ORDER_MRU, ORDER_LRU = 0, 1
POLICY_NO_LIFECYCLE, POLICY_INCLUSIVE, POLICY_ORPHANS_DEAD = 1, 2, 4
(OP_SPAWN, OP_FORK, OP_APPEND, OP_REPLACE, OP_REMOVE, OP_ONE_OFF, OP_PREFILL_DONE, OP_TERMINATE,
 OP_PIN, OP_UNPIN) = range(1, 11)
OPF_TOKENS_ON_DEVICE = 1
MAP_LOOKUP, MAP_ADMIT = 0, 1
IDS_ON_DEVICE = 1

EXPORTS = ("kvt_query_sizes", "kvt_create", "kvt_destroy", "kvt_apply_op", "kvt_map_blocks", "kvt_get_block_map",
           "kvt_classify", "kvt_get_states", "kvt_select_victims", "kvt_offload", "kvt_reload", "kvt_release",
           "kvt_compact", "kvt_copy_blocks", "kvt_hash_scratch_bytes", "kvt_hash_tokens", "kvt_get_stats",
           "kvt_last_error", "kvt_get_entries", "kvt_debug_load_resident", "kvt_set_profiling",
           "kvt_hash_tokens_noalloc", "kvt_debug_set_mover_variant", "kvt_exchange", "kvt_debug_set_lookup_variant", "kvt_move", "kvt_set_mover_ctas",
           "kvt_debug_set_wait_limit", "kvt_debug_set_classify_mode", "kvt_set_l2_residency", "kvt_debug_set_copy_delay")


class KvtError(RuntimeError):
    def __init__(self, code, what, detail=""):
        super().__init__(f"{what}: status {code} {detail}".strip())
        self.code = code


class Config(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("abi_version", "block_tokens", "n_layers", "n_kv_heads", "head_dim",
                                           "elem_bytes", "pool_layout", "n_hbm_blocks", "n_host_blocks",
                                           "table_capacity", "max_contexts", "max_messages", "max_batch_blocks",
                                           "policy_flags")] + \
               [("max_tokens", C.c_uint64), ("max_key_blocks", C.c_uint64), ("hash_seed", C.c_uint64),
                ("suspended_order", C.c_uint32), ("n_remote_blocks", C.c_uint32),
                ("hbm_pool", C.c_void_p), ("hbm_pool_bytes", C.c_uint64),
                ("host_pool", C.c_void_p), ("host_pool_bytes", C.c_uint64),
                ("dev_meta", C.c_void_p), ("dev_meta_bytes", C.c_uint64),
                ("dev_tokens", C.c_void_p), ("dev_tokens_bytes", C.c_uint64),
                ("remote_pool", C.c_void_p), ("remote_pool_bytes", C.c_uint64),
                ("stage_buf", C.c_void_p), ("stage_bytes", C.c_uint64)]


class Op(C.Structure):
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


def load_library():
    """Loads libkvt.so (built in-tree by paper_2609_39819_b200.build). Raises if it is missing."""
    global _lib
    if _lib is None:
        if ALT_LIB:
            if not os.path.exists(ALT_LIB):
                raise RuntimeError(f"KVT_LIB={ALT_LIB} does not exist")
            lib_path = ALT_LIB
        else:
            lib_path = LIB_PATH
        try:                                       # a build step, not a fallback: (re)compile the CUDA library
            from . import build                    # in-tree when it is missing or older than its sources
            if not ALT_LIB:
                build.build_lib()
        except Exception as exc:
            if not os.path.exists(LIB_PATH):
                raise RuntimeError(f"{LIB_PATH} is missing and could not be built with nvcc ({exc}); "
                                   "there is no CPU fallback") from exc
            import warnings
            warnings.warn(f"libkvt.so could not be rebuilt ({exc}); loading the existing binary")
        lib = C.CDLL(lib_path)
        vp, u32, u64, i32 = C.c_void_p, C.c_uint32, C.c_uint64, C.c_int32
        sig = {
            "kvt_query_sizes": [vp, vp, vp],
            "kvt_create": [vp, vp, vp],
            "kvt_destroy": [vp],
            "kvt_apply_op": [vp, vp, vp],
            "kvt_map_blocks": [vp, vp, u32, u32, vp, vp],
            "kvt_get_block_map": [vp, u32, vp, vp, vp, u32, vp, vp],
            "kvt_classify": [vp, vp],
            "kvt_get_states": [vp, u32, vp, u32, vp],
            "kvt_select_victims": [vp, u32, u32, u32, vp, vp, u32, vp, vp],
            "kvt_offload": [vp, vp, u32, vp, vp, vp],
            "kvt_reload": [vp, vp, u32, vp, vp],
            "kvt_exchange": [vp, vp, u32, vp, u32, vp, vp, vp, vp],
            "kvt_move": [vp, u32, u32, vp, u32, vp, vp, vp],
            "kvt_release": [vp, u32, vp, u32, vp],
            "kvt_compact": [vp, u32, vp, vp],
            "kvt_copy_blocks": [vp, u32, vp, u32, vp, u32, u32, vp],
            "kvt_hash_tokens": [vp, u64, u64, vp, vp, u64, vp],
            "kvt_hash_tokens_noalloc": [vp, u64, u64, vp, vp],
            "kvt_get_stats": [vp, vp],
            "kvt_last_error": [vp, vp, u32],
            "kvt_set_profiling": [vp, u32],
            "kvt_debug_set_mover_variant": [vp, u32],
            "kvt_debug_set_lookup_variant": [vp, u32],
            "kvt_set_mover_ctas": [vp, u32],
            "kvt_debug_set_wait_limit": [vp, u32],
            "kvt_debug_set_classify_mode": [vp, u32],
            "kvt_set_l2_residency": [vp, u32],
            "kvt_debug_set_copy_delay": [vp, u32],
            "kvt_get_entries": [vp, u32, vp, vp, vp, vp, vp, u32, vp],
            "kvt_debug_load_resident": [vp, vp, vp, vp, vp, vp, u32, u32, vp],
        }
        for name, args in sig.items():
            fn = getattr(lib, name)
            fn.argtypes = args
            fn.restype = i32
        lib.kvt_hash_scratch_bytes.argtypes = [u64]
        lib.kvt_hash_scratch_bytes.restype = u64
        _lib = lib
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def _u32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.uint32))


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def hash_tokens(tokens_dev, seed: int = 0):
    """Chained block keys of a device token tensor (int32/uint32 view, 16-byte aligned) -> int64 tensor
    whose bit patterns are the unsigned 64-bit keys."""
    import torch
    lib = load_library()
    n = tokens_dev.numel()
    keys = torch.empty(n // 16, dtype=torch.int64, device=tokens_dev.device)
    sb = lib.kvt_hash_scratch_bytes(n)
    scratch = torch.empty(sb, dtype=torch.uint8, device=tokens_dev.device)
    rc = lib.kvt_hash_tokens(tokens_dev.data_ptr(), n, seed, keys.data_ptr(), scratch.data_ptr(), sb, _stream())
    if rc:
        raise KvtError(rc, "hash_tokens")
    return keys


HASH_NOALLOC_MAX_TOKENS = 1 << 22


def hash_tokens_noalloc(tokens_dev, keys_out, seed: int = 0) -> int:
    """Block keys of a device token tensor written into the caller's `keys_out` (int64, >= n // 16
    elements) with the library's built-in scratch: for callers that must not allocate. Returns the
    status code (KVT_E_NOSPACE beyond HASH_NOALLOC_MAX_TOKENS)."""
    lib = load_library()
    return lib.kvt_hash_tokens_noalloc(tokens_dev.data_ptr(), tokens_dev.numel(), seed, keys_out.data_ptr(), _stream())


class Engine:
    """One cache engine on the current CUDA device. Allocates the pools and arenas with torch and
    hands raw pointers to the library."""

    def __init__(self, n_layers, n_kv_heads, head_dim, elem_bytes=2, pool_layout=LAYOUT_LAYER_MAJOR,
                 n_hbm_blocks=128, n_host_blocks=512, max_contexts=64, hash_seed=0, suspended_order=ORDER_MRU,
                 metadata_only=False, table_capacity=None, max_messages=1 << 16, max_batch_blocks=None,
                 max_tokens=1 << 22, max_key_blocks=None, host_pool_on_device=False, zero_pools=True, policy_flags=0,
                 n_remote_blocks=0, stage_mib=256, device="cuda"):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2609_39819_b200 needs a CUDA device (there is no CPU fallback)")
        self.torch = torch
        self.L = load_library()
        self.device = torch.device(device)
        self.n_layers, self.n_kv_heads, self.head_dim, self.elem_bytes = n_layers, n_kv_heads, head_dim, elem_bytes
        self.pool_layout = pool_layout
        self.n_hbm_blocks, self.n_host_blocks, self.n_remote_blocks = n_hbm_blocks, n_host_blocks, n_remote_blocks
        self.chunk_bytes = 16 * n_kv_heads * head_dim * elem_bytes
        self.n_chunks = 2 * n_layers
        self.block_bytes = self.chunk_bytes * self.n_chunks
        self.metadata_only = metadata_only
        n_total = n_hbm_blocks + n_host_blocks + n_remote_blocks
        if table_capacity is None:
            table_capacity = 1 << max(4, (2 * n_total - 1).bit_length())
        if max_batch_blocks is None:
            max_batch_blocks = max(max_tokens // 16, 1)
        if max_key_blocks is None:
            max_key_blocks = max(max_tokens // 8, 64)
        cfg = Config()
        cfg.abi_version, cfg.block_tokens = 3, 16
        cfg.n_layers, cfg.n_kv_heads, cfg.head_dim, cfg.elem_bytes = n_layers, n_kv_heads, head_dim, elem_bytes
        cfg.pool_layout, cfg.n_hbm_blocks, cfg.n_host_blocks = pool_layout, n_hbm_blocks, n_host_blocks
        cfg.n_remote_blocks = n_remote_blocks
        cfg.table_capacity, cfg.max_contexts, cfg.max_messages = table_capacity, max_contexts, max_messages
        cfg.max_batch_blocks, cfg.max_tokens, cfg.max_key_blocks = max_batch_blocks, max_tokens, max_key_blocks
        cfg.hash_seed, cfg.suspended_order, cfg.policy_flags = hash_seed, suspended_order, policy_flags
        mb, tb = C.c_uint64(0), C.c_uint64(0)
        rc = self.L.kvt_query_sizes(C.byref(cfg), C.byref(mb), C.byref(tb))
        if rc:
            raise KvtError(rc, "query_sizes")
        self.meta = torch.empty(mb.value + 256, dtype=torch.uint8, device=self.device)
        self.tokens = torch.empty(tb.value + 256, dtype=torch.uint8, device=self.device)
        cfg.dev_meta, cfg.dev_meta_bytes = self._align(self.meta), mb.value
        cfg.dev_tokens, cfg.dev_tokens_bytes = self._align(self.tokens), tb.value
        if metadata_only:
            self.hbm_pool = self.host_pool = self.remote_pool = None
        else:
            new = torch.zeros if zero_pools else torch.empty
            self.hbm_pool = new(n_hbm_blocks * self.block_bytes, dtype=torch.uint8, device=self.device)
            nh = max(n_host_blocks, 1) * self.block_bytes
            if host_pool_on_device:   # second tier kept in HBM (in-device measurements)
                self.host_pool = new(nh, dtype=torch.uint8, device=self.device)
            else:
                self.host_pool = new(nh, dtype=torch.uint8, pin_memory=True)
            cfg.hbm_pool, cfg.hbm_pool_bytes = self.hbm_pool.data_ptr(), self.hbm_pool.numel()
            cfg.host_pool, cfg.host_pool_bytes = self.host_pool.data_ptr(), self.host_pool.numel()
            # the remote tier is stood in for by one more buffer of the same kind as the host tier
            nr = max(n_remote_blocks, 1) * self.block_bytes
            if host_pool_on_device:
                self.remote_pool = new(nr, dtype=torch.uint8, device=self.device)
            else:
                self.remote_pool = new(nr, dtype=torch.uint8, pin_memory=True)
            if n_remote_blocks:
                cfg.remote_pool, cfg.remote_pool_bytes = self.remote_pool.data_ptr(), self.remote_pool.numel()
            # staging ring for copy-engine transfers between HBM and a host-memory tier (large blocks only)
            self.stage_buf = None
            if stage_mib and not host_pool_on_device and (n_host_blocks or n_remote_blocks):
                self.stage_buf = torch.empty(stage_mib << 20, dtype=torch.uint8, device=self.device)
                cfg.stage_buf, cfg.stage_bytes = self.stage_buf.data_ptr(), self.stage_buf.numel()
        self.cfg = cfg
        h = C.c_void_p()
        rc = self.L.kvt_create(C.byref(cfg), _stream(), C.byref(h))
        if rc:
            raise KvtError(rc, "create")
        self.h = h

    @staticmethod
    def _align(t):
        return (t.data_ptr() + 255) // 256 * 256

    def close(self):
        if getattr(self, "h", None):
            self.L.kvt_destroy(self.h)
            self.h = None
            self.hbm_pool = self.host_pool = self.remote_pool = self.meta = self.tokens = self.stage_buf = None   # release the memory

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_profiling(self, on=True):
        self._check(self.L.kvt_set_profiling(self.h, 1 if on else 0), "set_profiling")

    def set_mover_variant(self, variant):
        self._check(self.L.kvt_debug_set_mover_variant(self.h, variant), "set_mover_variant")

    def set_mover_ctas(self, max_ctas):
        self._check(self.L.kvt_set_mover_ctas(self.h, max_ctas), "set_mover_ctas")

    def set_lookup_variant(self, variant):
        self._check(self.L.kvt_debug_set_lookup_variant(self.h, variant), "set_lookup_variant")

    def set_copy_delay(self, delay_ns):
        self._check(self.L.kvt_debug_set_copy_delay(self.h, int(delay_ns)), "set_copy_delay")

    def set_l2_residency(self, on=True):
        self._check(self.L.kvt_set_l2_residency(self.h, 1 if on else 0), "set_l2_residency")

    def set_classify_mode(self, mode):
        self._check(self.L.kvt_debug_set_classify_mode(self.h, mode), "set_classify_mode")

    def set_wait_limit(self, polls):
        self._check(self.L.kvt_debug_set_wait_limit(self.h, polls), "set_wait_limit")

    def last_error(self):
        buf = C.create_string_buffer(256)
        self.L.kvt_last_error(self.h, buf, 256)
        return buf.value.decode()

    def _check(self, rc, what):
        if rc:
            raise KvtError(rc, what, self.last_error())

    # ---- primitives ---------------------------------------------------------------------------
    def apply_op_rc(self, op, ctx, parent=0, msg_start=0, msg_end=0, tokens=None) -> int:
        flags, ptr, n = 0, None, 0
        keep = None
        if tokens is not None:
            if hasattr(tokens, "data_ptr"):      # torch tensor: device memory, or (pinned) host memory
                keep = tokens
                flags, ptr, n = (OPF_TOKENS_ON_DEVICE if tokens.is_cuda else 0), tokens.data_ptr(), tokens.numel()
            else:
                keep = _u32(tokens)
                ptr, n = keep.ctypes.data, len(keep)
        o = Op(op, ctx, parent, msg_start, msg_end, n, flags, 0, ptr)
        return self.L.kvt_apply_op(self.h, C.byref(o), _stream())

    def _op(self, what, *a, **k):
        self._check(self.apply_op_rc(*a, **k), what)

    def spawn(self, ctx): self._op("spawn", OP_SPAWN, ctx)
    def fork(self, parent, child, end): self._op("fork", OP_FORK, child, parent=parent, msg_end=end)
    def append(self, ctx, tokens): self._op("append", OP_APPEND, ctx, tokens=tokens)
    def replace(self, ctx, s, e, tokens): self._op("replace", OP_REPLACE, ctx, msg_start=s, msg_end=e, tokens=tokens)
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
        rc = self.L.kvt_map_blocks(self.h, _p(ids), len(ids), phase, _p(out), _stream())
        return rc, out

    def map_blocks(self, ctx_ids, phase):
        rc, out = self.map_blocks_rc(ctx_ids, phase)
        self._check(rc, "map_blocks")
        return out

    def get_block_map(self, ctx):
        n = C.c_uint32(0)
        rc = self.L.kvt_get_block_map(self.h, ctx, None, None, None, 0, C.byref(n), _stream())
        if rc not in (OK, E_BUFSZ):
            self._check(rc, "get_block_map")
        nb = n.value
        keys = np.empty(nb, np.uint64); tier = np.empty(nb, np.uint8); slot = np.empty(nb, np.uint32)
        self._check(self.L.kvt_get_block_map(self.h, ctx, _p(keys), _p(tier), _p(slot), nb, C.byref(n), _stream()),
                    "get_block_map")
        return keys, tier, slot

    # ---- classify / select ----------------------------------------------------------------------
    def classify(self):
        self._check(self.L.kvt_classify(self.h, _stream()), "classify")

    def _tier_size(self, tier):
        sizes = (self.n_hbm_blocks, self.n_host_blocks, self.n_remote_blocks)
        return sizes[tier] if 0 <= tier < 3 else 0      # an unknown tier is for the library to reject

    def get_states(self, tier):
        st = np.zeros(self._tier_size(tier), np.uint8)
        self._check(self.L.kvt_get_states(self.h, tier, _p(st), len(st), _stream()), "get_states")
        return st

    def victim_buffers(self, n):
        """A pair of pinned host arrays (slots, states) for `out=` of select_victims: the selection's last kernel
        writes the list straight into them instead of staging it for a CPU copy."""
        import torch
        ts = torch.empty(n, dtype=torch.int32, pin_memory=True); tt = torch.empty(n, dtype=torch.uint8, pin_memory=True)
        self._victim_bufs = getattr(self, "_victim_bufs", []) + [(ts, tt)]     # the arrays below do not own the memory
        return ts.numpy().view(np.uint32), tt.numpy()

    def select_victims(self, tier, n_req, include_pinned=False, out=None):
        cap = min(n_req, self._tier_size(tier))
        if out is None:
            slots = np.empty(cap, np.uint32); states = np.empty(cap, np.uint8)     # filled by the call up to n
        else:
            slots, states = out
            if len(slots) < cap or len(states) < cap or slots.dtype != np.uint32 or states.dtype != np.uint8:
                raise ValueError("select_victims: out arrays too small or of the wrong type")
        n = C.c_uint32(0)
        self._check(self.L.kvt_select_victims(self.h, tier, n_req, 1 if include_pinned else 0, _p(slots), _p(states),
                                              cap, C.byref(n), _stream()), "select_victims")
        return slots[:n.value], states[:n.value]

    # ---- movement -------------------------------------------------------------------------------
    def offload(self, slots):
        s = _u32(slots); nd = C.c_uint32(0); nx = C.c_uint32(0)
        rc = self.L.kvt_offload(self.h, _p(s), len(s), C.byref(nd), C.byref(nx), _stream())
        return rc, nd.value, nx.value

    def reload(self, slots):
        s = _u32(slots); nd = C.c_uint32(0)
        rc = self.L.kvt_reload(self.h, _p(s), len(s), C.byref(nd), _stream())
        return rc, nd.value

    def move(self, src_tier, dst_tier, slots):
        s = _u32(slots)
        nd, nx = C.c_uint32(0), C.c_uint32(0)
        rc = self.L.kvt_move(self.h, src_tier, dst_tier, _p(s), len(s), C.byref(nd), C.byref(nx), _stream())
        return rc, nd.value, nx.value

    def exchange(self, out_slots, in_slots):
        o, i = _u32(out_slots), _u32(in_slots)
        a, b, c = C.c_uint32(0), C.c_uint32(0), C.c_uint32(0)
        rc = self.L.kvt_exchange(self.h, _p(o), len(o), _p(i), len(i), C.byref(a), C.byref(b), C.byref(c), _stream())
        return rc, a.value, b.value, c.value

    def release_rc(self, tier, slots):
        s = _u32(slots)
        return self.L.kvt_release(self.h, tier, _p(s), len(s), _stream())

    def release(self, tier, slots):
        self._check(self.release_rc(tier, slots), "release")

    def compact(self, tier):
        n = C.c_uint32(0)
        self._check(self.L.kvt_compact(self.h, tier, C.byref(n), _stream()), "compact")
        return n.value

    def copy_blocks(self, src_tier, src, dst_tier, dst):
        """src / dst: host sequences, or device int32 tensors (ids stay on the device)."""
        if hasattr(src, "data_ptr"):
            rc = self.L.kvt_copy_blocks(self.h, src_tier, src.data_ptr(), dst_tier, dst.data_ptr(), src.numel(),
                                        IDS_ON_DEVICE, _stream())
        else:
            s, d = _u32(src), _u32(dst)
            rc = self.L.kvt_copy_blocks(self.h, src_tier, _p(s), dst_tier, _p(d), len(s), 0, _stream())
        self._check(rc, "copy_blocks")

    # ---- introspection --------------------------------------------------------------------------
    def get_stats(self):
        out = np.zeros(len(STATS_FIELDS), np.uint64)
        self._check(self.L.kvt_get_stats(self.h, _p(out)), "get_stats")
        return dict(zip(STATS_FIELDS, out.tolist()))

    def get_entries(self, tier):
        n = self._tier_size(tier)
        keys = np.zeros(n, np.uint64); stamp = np.zeros(n, np.uint32)
        depth = np.zeros(n, np.uint32); infl = np.zeros(n, np.uint32); link = np.zeros(n, np.uint32)
        self._check(self.L.kvt_get_entries(self.h, tier, _p(keys), _p(stamp), _p(depth), _p(infl), _p(link), n,
                                           _stream()), "get_entries")
        return {"key": keys, "stamp": stamp, "depth": depth, "inflight": infl, "link": link}

    def debug_load_resident_rc(self, keys, state, stamp, depth, slot, tier):
        k = np.ascontiguousarray(np.asarray(keys, np.uint64)); st = np.ascontiguousarray(np.asarray(state, np.uint8))
        sp, dp, sl = _u32(stamp), _u32(depth), _u32(slot)
        return self.L.kvt_debug_load_resident(self.h, _p(k), _p(st), _p(sp), _p(dp), _p(sl), tier, len(k), _stream())

    def debug_load_resident(self, *a):
        self._check(self.debug_load_resident_rc(*a), "debug_load_resident")

    # ---- payload access for the harness (producing KV is the model's job, not the engine's) -------
    def _chunks(self, tier, slot):
        if tier == TIER_HBM and self.pool_layout == LAYOUT_LAYER_MAJOR:
            return self.hbm_pool.view(self.n_chunks, self.n_hbm_blocks, self.chunk_bytes)[:, slot, :]
        pool = (self.hbm_pool, self.host_pool, self.remote_pool)[tier]
        return pool.view(-1, self.n_chunks, self.chunk_bytes)[slot]

    # Device-side counterpart of workloads.payload_pattern for large blocks (harness helpers, torch ops only).
    def _pattern(self, key):
        torch = self.torch
        if getattr(self, "_pat_base", None) is None:
            self._pat_base = (torch.arange(self.block_bytes // 4, dtype=torch.int64, device=self.device) * 0x9E3779B1) & 0xFFFFFFFF
        w = ((self._pat_base + (int(key) & 0xFFFFFFFF)) & 0xFFFFFFFF) ^ (int(key) >> 32)
        return w.to(torch.int32).view(torch.uint8).view(self.n_chunks, self.chunk_bytes)

    def fill_block_pattern(self, tier, slot, key):
        dst = self._chunks(tier, slot)
        dst.copy_(self._pattern(key).to(dst.device))

    def check_block_pattern(self, tier, slot, key) -> bool:
        self.torch.cuda.current_stream().synchronize()
        got = self._chunks(tier, slot).to(self.device)
        return bool(self.torch.equal(got, self._pattern(key)))

    def write_block(self, tier, slot, payload):
        t = self.torch.from_numpy(np.ascontiguousarray(np.asarray(payload, np.uint8))).view(self.n_chunks, self.chunk_bytes)
        dst = self._chunks(tier, slot)
        dst.copy_(t.to(dst.device))

    def read_block(self, tier, slot):
        self.torch.cuda.current_stream().synchronize()
        return self._chunks(tier, slot).contiguous().cpu().numpy().reshape(-1)
