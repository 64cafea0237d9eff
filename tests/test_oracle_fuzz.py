"""Random API streams on the CPU oracle alone: after every few calls the global invariants hold, the
classification equals the literal double loop, and every occupied slot holds its key's payload."""
import pytest

import fuzz_driver as F

MOVED = {}
from paper_2609_39819_b200 import workloads as W


@pytest.mark.parametrize("seed", range(8))
@pytest.mark.parametrize("flags", [0, 1, 2, 3, 4, 6])
@pytest.mark.parametrize("pools", [(24, 16), (8, 4), (40, 0)], ids=lambda p: f"hbm{p[0]}-host{p[1]}")
def test_oracle_survives_random_api_streams(oracle, seed, flags, pools):
    eng = oracle.OracleEngine(n_hbm_blocks=pools[0], n_host_blocks=pools[1], max_contexts=6, policy_flags=flags,
                              suspended_order=seed % 2, pool_layout=seed % 2, **W.GEO_TOY.kwargs())
    f = F.run([eng], seed, steps=300, inclusive=bool(flags & 2), check_every=5)
    st = eng.get_stats()
    assert st["blocks_hashed"] > 0 and st["inserted"] > 0


@pytest.mark.parametrize("seed", range(8))
@pytest.mark.parametrize("flags", [0, 1, 2, 4])
@pytest.mark.parametrize("pools", [(24, 12, 16), (8, 4, 3), (16, 0, 8)], ids=lambda p: f"hbm{p[0]}-host{p[1]}-remote{p[2]}")
def test_oracle_survives_random_api_streams_with_three_tiers(oracle, seed, flags, pools):
    eng = oracle.OracleEngine(n_hbm_blocks=pools[0], n_host_blocks=pools[1], n_remote_blocks=pools[2], max_contexts=6,
                              policy_flags=flags, suspended_order=seed % 2, pool_layout=seed % 2, **W.GEO_TOY.kwargs())
    F.run([eng], seed, steps=300, inclusive=bool(flags & 2), check_every=5)
    st = eng.get_stats()
    assert st["blocks_hashed"] > 0 and st["inserted"] > 0
    MOVED[pools] = MOVED.get(pools, 0) + st["demoted"] + st["promoted"]
    if seed == 7 and pools[1]:
        assert MOVED[pools] > 0      # over the seeds of a pool shape, blocks did travel to and from the remote tier
