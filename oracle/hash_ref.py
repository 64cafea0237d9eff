"""Second, independent statement of the chained block hash, in pure Python integers.

TEST INFRASTRUCTURE (see kvt_oracle.cpp). Where the C++ oracle loops h_b = P*h_{b-1} + d_b, this file
evaluates the closed form  h_b = P^(b+1)*H0 + sum_{i<=b} P^(b-i)*d_i  with arbitrary-precision
integers and reduces mod 2^64 only at the end, so a mistake in either the recurrence or the
wrap-around arithmetic of the C++ code shows up as a difference. Small inputs only.
"""
M64 = (1 << 64) - 1
GOLD = 0x9E3779B97F4A7C15


def mix64(z: int) -> int:
    z &= M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
    return z ^ (z >> 31)


def _unxorshift(y: int, s: int) -> int:
    x = y
    for _ in range(64 // s + 1):
        x = y ^ (x >> s)
    return x


def unmix64(y: int) -> int:
    """Inverse of mix64 (each step of mix64 is invertible: xor-shift and odd multiplication)."""
    y = _unxorshift(y, 31)
    y = (y * pow(0x94D049BB133111EB, -1, 1 << 64)) & M64
    y = _unxorshift(y, 27)
    y = (y * pow(0xBF58476D1CE4E5B9, -1, 1 << 64)) & M64
    return _unxorshift(y, 30)


def constants(seed: int = 0):
    K = [mix64(GOLD * (t + 1)) | 1 for t in range(16)]
    P = mix64(GOLD * 17) | 1
    H0 = mix64((seed & M64) ^ ((GOLD * 18) & M64))
    return K, P, H0


def block_digests(tokens, K):
    out = []
    for b in range(len(tokens) // 16):
        s = sum((int(tokens[16 * b + t]) + 1) * K[t] for t in range(16))  # exact, no wrap-around
        out.append(mix64(s))
    return out


def hash_tokens(tokens, seed: int = 0):
    """Returns (keys, h) per full block using the closed form with exact integers."""
    K, P, H0 = constants(seed)
    d = block_digests(tokens, K)
    keys, hs = [], []
    for b in range(len(d)):
        h = pow(P, b + 1) * H0 + sum(pow(P, b - i) * d[i] for i in range(b + 1))
        h &= M64
        key = mix64(h)
        if key < 2:
            key += 2
        hs.append(h)
        keys.append(key)
    return keys, hs
