"""Random differential test: the same random stream of API calls (valid and invalid, every policy switch) goes to
the CUDA engine and to the CPU oracle; every status code, every returned list and, every few calls, all metadata,
states, statistics and payload bytes must be identical."""
import pytest

import fuzz_driver as F
from paper_2609_39819_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", range(24))
@pytest.mark.parametrize("flags", [0, 1, 2, 3, 4, 7])
@pytest.mark.parametrize("pools", [(24, 16), (8, 4), (40, 0)], ids=lambda p: f"hbm{p[0]}-host{p[1]}")
def test_random_api_streams_match_the_oracle(oracle, seed, flags, pools):
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_39819_b200 import binding as B
    kw = dict(n_hbm_blocks=pools[0], n_host_blocks=pools[1], max_contexts=6, policy_flags=flags, suspended_order=seed % 2,
              pool_layout=seed % 2, **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=1 << 16, max_messages=2048, stage_mib=1, **kw)
    gpu.set_classify_mode((2, 1, 0)[seed % 3])    # event-driven counts cross-checked / recomputed in full / on their own
    if seed % 2:
        gpu.set_mover_variant(4)                  # payload through the staging ring and the copy engines (8 blocks per stage)
    cpu = oracle.OracleEngine(**kw)
    F.run([gpu, cpu], seed, steps=300, inclusive=bool(flags & 2), check_every=10)


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("flags", [0, 2])
def test_random_api_streams_with_long_messages(oracle, seed, flags):
    """Messages of up to 6,000 tokens: contexts span several 256-block hash chunks, so edits, forks and repeated
    calls exercise the incremental hasher's resume points inside the random stream."""
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_39819_b200 import binding as B
    kw = dict(n_hbm_blocks=1500, n_host_blocks=600, max_contexts=6, policy_flags=flags, metadata_only=True,
              **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=1 << 20, max_messages=4096, **kw)
    gpu.set_lookup_variant(1 + seed % 4)      # every form of the hash + probe stage
    gpu.set_l2_residency(seed % 5 != 0)       # with and without the L2 window on the metadata kernels
    gpu.set_classify_mode((2, 0, 1)[seed % 3])
    cpu = oracle.OracleEngine(**kw)
    F.run([gpu, cpu], seed, steps=200, inclusive=bool(flags & 2), check_every=10, invariants=False, max_tok=6000)
    st = gpu.get_stats()
    assert st["blocks_rehashed"] < st["blocks_hashed"]


@pytest.mark.parametrize("seed", range(12))
@pytest.mark.parametrize("flags", [0, 1, 2, 4])
@pytest.mark.parametrize("pools", [(24, 12, 16), (8, 4, 3), (16, 0, 8)], ids=lambda p: f"hbm{p[0]}-host{p[1]}-remote{p[2]}")
def test_random_api_streams_with_three_tiers(oracle, seed, flags, pools):
    """The same with a remote tier behind the host tier: blocks travel down level by level and up again,
    straight into HBM too."""
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_39819_b200 import binding as B
    kw = dict(n_hbm_blocks=pools[0], n_host_blocks=pools[1], n_remote_blocks=pools[2], max_contexts=6, policy_flags=flags,
              suspended_order=seed % 2, pool_layout=seed % 2, **W.GEO_TOY.kwargs())
    gpu = B.Engine(max_tokens=1 << 16, max_messages=2048, stage_mib=1, **kw)
    gpu.set_classify_mode((2, 1, 0)[seed % 3])    # event-driven counts cross-checked / recomputed in full / on their own
    if seed % 2:
        gpu.set_mover_variant(4)                  # payload through the staging ring and the copy engines (8 blocks per stage)
    cpu = oracle.OracleEngine(**kw)
    F.run([gpu, cpu], seed, steps=300, inclusive=bool(flags & 2), check_every=10)


@pytest.mark.parametrize("seed", range(8))
@pytest.mark.parametrize("long_messages", [False, True], ids=["short", "long"])
def test_results_do_not_depend_on_when_control_records_arrive(oracle, seed, long_messages):
    """The descriptors, message tables and status words of a call are carried by small kernels, and the kernels
    behind them are dependent launches that may start early. With those copies held back by 0.2 ms, a kernel that
    looked at a record before its wait would see the previous call's: every result must still equal the oracle's."""
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_39819_b200 import binding as B
    if long_messages:
        kw = dict(n_hbm_blocks=1500, n_host_blocks=600, max_contexts=6, policy_flags=(0, 2)[seed % 2], metadata_only=True,
                  **W.GEO_TOY.kwargs())
        gpu = B.Engine(max_tokens=1 << 20, max_messages=4096, **kw)
    else:
        kw = dict(n_hbm_blocks=24, n_host_blocks=16, max_contexts=6, policy_flags=(0, 1, 2, 4)[seed % 4], suspended_order=seed % 2,
                  **W.GEO_TOY.kwargs())
        gpu = B.Engine(max_tokens=1 << 16, max_messages=2048, stage_mib=1, **kw)
    gpu.set_copy_delay(200_000)
    gpu.set_classify_mode((0, 2)[seed % 2])
    cpu = oracle.OracleEngine(**kw)
    if long_messages:
        F.run([gpu, cpu], 1000 + seed, steps=120, inclusive=bool(kw["policy_flags"] & 2), check_every=10, invariants=False, max_tok=6000)
    else:
        F.run([gpu, cpu], 1000 + seed, steps=200, inclusive=bool(kw["policy_flags"] & 2), check_every=10)
