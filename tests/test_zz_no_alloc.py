"""The allocation-free hasher entry point, for callers that may not allocate device memory (a plug-in
inside a serving engine that owns the whole memory budget, a request loop where an allocation would
stall the device). Collected last on purpose. It must give exactly the keys of the ordinary entry
point, call after call, although every call reuses the same built-in scratch array."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def test_noalloc_hasher_matches_the_ordinary_one_twice_in_a_row():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_39819_b200 import binding as B
    B.load_library()
    rng = np.random.default_rng(2024)
    from oracle import kvt_oracle
    # first a long input (many chunks), then shorter ones: stale scratch of an earlier call must not matter. Also an
    # exact multiple of the 256-block chunk and a single block.
    for n_tokens, seed in ((16 * 5000 + 11, 0), (16 * 300 + 5, 7), (16 * 256 * 3, 1), (16, 5)):
        host = rng.integers(0, 151552, n_tokens, dtype=np.uint32)
        tok = torch.from_numpy(host.view(np.int32)).cuda()
        want = B.hash_tokens(tok, seed)                       # existing entry point, caller-provided scratch
        got = torch.zeros(n_tokens // 16, dtype=torch.int64, device="cuda")
        assert B.hash_tokens_noalloc(tok, got, seed) == B.OK  # through the C ABI, built-in scratch
        torch.cuda.synchronize()
        assert torch.equal(got, want)                         # integer keys: bit-exact
        assert np.array_equal(got.cpu().numpy().view(np.uint64), kvt_oracle.hash_tokens(host, seed))   # and the CPU definition
    # sizes beyond the built-in scratch are refused, nothing is written
    big = torch.empty(B.HASH_NOALLOC_MAX_TOKENS + 16, dtype=torch.int32, device="cuda")
    out = torch.full((1,), 123, dtype=torch.int64, device="cuda")
    assert B.hash_tokens_noalloc(big, out, 0) == B.E_NOSPACE
    torch.cuda.synchronize()
    assert int(out[0]) == 123
    # the largest accepted size works
    tok = torch.from_numpy(rng.integers(0, 151552, B.HASH_NOALLOC_MAX_TOKENS, dtype=np.uint32).view(np.int32)).cuda()
    got = torch.zeros(B.HASH_NOALLOC_MAX_TOKENS // 16, dtype=torch.int64, device="cuda")
    assert B.hash_tokens_noalloc(tok, got, 3) == B.OK
    assert torch.equal(got, B.hash_tokens(tok, 3))
