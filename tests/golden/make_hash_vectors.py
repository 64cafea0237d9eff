"""Writes tests/golden/hash_vectors.txt from the pure-Python exact-integer statement of the block
hash (oracle/hash_ref.py). Calls nothing outside oracle/. Run from the repository root:
    python tests/golden/make_hash_vectors.py
"""
import os
import sys

sys.path.insert(0, os.path.join(os.path.dirname(os.path.abspath(__file__)), "..", ".."))
from oracle import hash_ref  # noqa: E402

CASES = [
    ("range48", 0, list(range(48))),
    ("zeros32", 0, [0] * 32),
    ("max16", 0, [151551] * 16),
    ("range48_tok20_999", 0, [999 if i == 20 else i for i in range(48)]),
    ("range40", 0, list(range(40))),
    ("range48_seed1", 1, list(range(48))),
]


def main():
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "hash_vectors.txt")
    with open(out, "w") as f:
        f.write("# Block keys of the chained 16-token block hash for small inputs, computed with exact Python\n"
                "# integers from the closed form (oracle/hash_ref.py). The paper does not define a hash; the\n"
                "# definition is this build's reading. Format: name seed n_tokens key0 key1 ...\n")
        for name, seed, toks in CASES:
            keys, _ = hash_ref.hash_tokens(toks, seed)
            f.write(f"{name} {seed} {len(toks)} " + " ".join(f"{k:016x}" for k in keys) + "\n")
        K, P, H0 = hash_ref.constants(0)
        f.write(f"constants 0 0 {K[0]:016x} {K[1]:016x} {K[15]:016x} {P:016x} {H0:016x} {hash_ref.mix64(1):016x}\n")


if __name__ == "__main__":
    main()
