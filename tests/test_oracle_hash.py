"""Pins of the oracle's block hash against things other than itself: the published SplitMix64
stream, an exact-integer closed form, the inverse of the mixing function, and the structural
properties the chain must have."""
import os

import numpy as np
import pytest

from oracle import hash_ref

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
M64 = (1 << 64) - 1


def _read(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_mix64_is_splitmix64_output_function(oracle):
    stream = [int(r[0], 16) for r in _read("splitmix64_seed0.txt")]
    gold = 0x9E3779B97F4A7C15
    K, P, H0, _ = oracle.hash_constants(0, 0)
    for n, want in enumerate(stream, start=1):
        assert oracle.hash_constants(0, (gold * n) & M64)[3] == want
    for t in range(5):
        assert K[t] == stream[t] | 1  # lane multipliers come from the same stream, forced odd


def test_constants_and_vectors_match_exact_integer_form(oracle):
    rows = _read("hash_vectors.txt")
    for r in rows:
        if r[0] == "constants":
            K, P, H0, m1 = oracle.hash_constants(0, 1)
            assert [K[0], K[1], K[15], P, H0, m1] == [int(x, 16) for x in r[3:]]
    cases = {
        "range48": np.arange(48), "zeros32": np.zeros(32), "max16": np.full(16, 151551),
        "range48_tok20_999": np.where(np.arange(48) == 20, 999, np.arange(48)), "range40": np.arange(40),
        "range48_seed1": np.arange(48),
    }
    seen = 0
    for r in rows:
        if r[0] in cases:
            keys = oracle.hash_tokens(cases[r[0]], int(r[1]))
            assert [int(k) for k in keys] == [int(x, 16) for x in r[3:]], r[0]
            seen += 1
    assert seen == len(cases)


def test_mix64_inverse_round_trip(oracle):
    rng = np.random.default_rng(7)
    for x in [0, 1, 2, M64] + [int(v) for v in rng.integers(0, 1 << 63, 50)]:
        y = oracle.hash_constants(0, x)[3]
        assert hash_ref.unmix64(y) == x  # mix64 is a bijection and the oracle computes exactly it


@pytest.mark.parametrize("seed", [0, 1, 0xDEADBEEFCAFEF00D])
def test_matches_closed_form_on_random_tokens(oracle, seed):
    rng = np.random.default_rng(seed & 0xFFFF)
    for n in (0, 15, 16, 17, 160, 1000):
        tok = rng.integers(0, 151552, n)
        want, _ = hash_ref.hash_tokens(tok, seed)
        got = oracle.hash_tokens(tok, seed)
        assert len(got) == n // 16                      # only full blocks have keys
        assert [int(k) for k in got] == want


def test_chain_is_affine_in_the_previous_state(oracle):
    """h_b - P*h_{b-1} depends only on block b's tokens; recovered through the inverse of mix64."""
    rng = np.random.default_rng(3)
    _, P, H0, _ = oracle.hash_constants(0, 0)
    blk = rng.integers(0, 151552, 16)
    ds = []
    for _ in range(4):
        prefix = rng.integers(0, 151552, 16 * int(rng.integers(1, 6)))
        keys = oracle.hash_tokens(np.concatenate([prefix, blk]))
        h = [hash_ref.unmix64(int(k)) for k in keys]
        ds.append((h[-1] - P * h[-2]) & M64)
    assert len(set(ds)) == 1
    # first block: h_0 = P*H0 + d_0 with the same d
    h0 = hash_ref.unmix64(int(oracle.hash_tokens(blk)[0]))
    assert (h0 - P * H0) & M64 == ds[0]


def test_difference_propagates_with_powers_of_P(oracle):
    """Two sequences differing only in block j: h_b - h'_b = P^(b-j) (d_j - d'_j) for b >= j."""
    rng = np.random.default_rng(5)
    _, P, _, _ = oracle.hash_constants(0, 0)
    a = rng.integers(0, 151552, 16 * 12)
    b = a.copy()
    j = 4
    b[16 * j + 3] ^= 1
    ha = [hash_ref.unmix64(int(k)) for k in oracle.hash_tokens(a)]
    hb = [hash_ref.unmix64(int(k)) for k in oracle.hash_tokens(b)]
    assert ha[:j] == hb[:j]
    d = (ha[j] - hb[j]) & M64
    assert d != 0
    for k in range(j, 12):
        assert (ha[k] - hb[k]) & M64 == (pow(P, k - j, 1 << 64) * d) & M64


def test_prefix_suffix_position_seed_properties(oracle):
    rng = np.random.default_rng(11)
    tok = rng.integers(0, 151552, 16 * 40 + 9)
    keys = oracle.hash_tokens(tok)
    # equal token prefixes hash identically (fork sharing); one-shot = prefix-by-prefix
    for cut in (16, 160, 333, 640):
        assert np.array_equal(oracle.hash_tokens(tok[:cut]), keys[: cut // 16])
    # a change inside block j changes every key from j on and none before
    for j in (0, 7, 39):
        t2 = tok.copy()
        t2[16 * j + 5] = (t2[16 * j + 5] + 1) % 151552
        k2 = oracle.hash_tokens(t2)
        assert np.array_equal(k2[:j], keys[:j]) and np.all(k2[j:] != keys[j:])
    # position inside the block matters (every lane has its own multiplier)
    for p in range(15):
        t2 = tok.copy()
        if t2[p] == t2[p + 1]:
            continue
        t2[p], t2[p + 1] = t2[p + 1], t2[p]
        assert oracle.hash_tokens(t2)[0] != keys[0]
    # keys never take the two reserved table values; the seed changes every key
    assert np.all(keys >= 2)
    assert np.all(oracle.hash_tokens(tok, 1) != keys)
    # no collisions in a modest sample
    big = oracle.hash_tokens(rng.integers(0, 151552, 16 * 20000))
    assert len(np.unique(big)) == len(big)


def test_parallel_digests_and_copies_match_the_plain_ones(oracle):
    """The all-cores timing helpers compute the same things: the chain over their digests gives the block keys, and
    the threaded block copy equals a plain gather."""
    rng = np.random.default_rng(11)
    tok = rng.integers(0, 151552, 16 * 1000 + 9, dtype=np.uint32)
    for seed in (0, 5):
        _K, P, H0, _ = oracle.hash_constants(seed)
        d = oracle.par_digests(tok, seed, n_threads=3)
        h, keys = H0, []
        for x in d:
            h = (P * h + int(x)) & (2**64 - 1)
            k = oracle.hash_constants(seed, h)[3]
            keys.append(k + 2 if k < 2 else k)
        assert keys == [int(k) for k in oracle.hash_tokens(tok, seed)]
    src = rng.integers(0, 256, 64 * 4096, dtype=np.uint8)
    dst = np.zeros(32 * 4096, dtype=np.uint8)
    si, di = rng.permutation(64)[:32], rng.permutation(32)
    oracle.par_copy_blocks(dst, src, 4096, si, di, n_threads=4)
    want = np.zeros_like(dst).reshape(32, 4096)
    want[di] = src.reshape(64, 4096)[si]
    assert np.array_equal(dst.reshape(32, 4096), want)
