"""The C-ABI library builds for sm_100a, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    from paper_2609_39819_b200 import build, binding
    lib_path = build.build_lib()
    header = open(os.path.join(ROOT, "include", "kvt.h")).read()
    declared = set(re.findall(r"^(?:int32_t|uint64_t)\s+(kvt_\w+)\s*\(", header, flags=re.M))
    assert len(declared) >= 20 and {"kvt_apply_op", "kvt_map_blocks", "kvt_classify", "kvt_select_victims",
                                    "kvt_offload", "kvt_reload"} <= declared
    lib = ctypes.CDLL(lib_path)
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(binding.EXPORTS)


def test_query_sizes_needs_no_gpu():
    from paper_2609_39819_b200 import binding
    lib = binding.load_library()
    cfg = binding.Config()
    cfg.abi_version, cfg.block_tokens = 3, 16
    cfg.n_layers, cfg.n_kv_heads, cfg.head_dim, cfg.elem_bytes = 2, 2, 64, 2
    cfg.n_hbm_blocks, cfg.n_host_blocks, cfg.table_capacity = 128, 512, 2048
    cfg.max_contexts, cfg.max_messages, cfg.max_batch_blocks = 64, 1024, 4096
    cfg.max_tokens, cfg.max_key_blocks = 1 << 16, 1 << 13
    mb, tb = ctypes.c_uint64(0), ctypes.c_uint64(0)
    assert lib.kvt_query_sizes(ctypes.byref(cfg), ctypes.byref(mb), ctypes.byref(tb)) == 0
    assert mb.value > 2048 * 16 and tb.value == (1 << 16) * 4
    assert lib.kvt_query_sizes(None, ctypes.byref(mb), ctypes.byref(tb)) == binding.E_INVAL
    assert lib.kvt_hash_scratch_bytes(16 * 1000) == (2 * 4 + 1) * 8


def test_struct_sizes_match_the_header():
    from paper_2609_39819_b200 import binding
    assert ctypes.sizeof(binding.Config) == 14 * 4 + 3 * 8 + 2 * 4 + 12 * 8
    assert ctypes.sizeof(binding.Op) == 8 * 4 + 8
    assert binding.CALL_INFO_DTYPE.itemsize == 9 * 4


def test_stats_and_call_info_fields_follow_the_header():
    """The bindings unpack kvt_stats / kvt_call_info by position: their field lists must be the header's, in order."""
    import re
    from paper_2609_39819_b200 import binding
    from oracle import kvt_oracle
    text = open(os.path.join(ROOT, "include", "kvt.h")).read()

    def fields(struct, ctype):
        body = text[text.index(f"typedef struct {struct}"):text.index(f"}} {struct};")]
        out = []
        for decl in re.findall(ctype + r"\s+([^;]+);", body):
            out += [x.strip() for x in decl.split(",")]
        return out

    stats = fields("kvt_stats", "uint64_t")
    assert stats == list(binding.STATS_FIELDS) == list(kvt_oracle.STATS_FIELDS)
    info = fields("kvt_call_info", "uint32_t")
    assert info == list(binding.CALL_INFO_DTYPE.names) == list(kvt_oracle.CALL_INFO_DTYPE.names)
