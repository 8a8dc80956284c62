"""Writes tests/golden/sampler_vectors.txt from the CPU oracle alone.

Known-answer vectors for the random-sentinel sampler (Section 3.1 item 2): raw 32-bit
draws and complete sentinel draws.  The CUDA library implements the same counter-based
generator independently; its host-callable copy is checked against this file.

    python tests/golden/make_sampler_vectors.py
"""
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import routerelay_oracle as O  # noqa: E402


def main():
    lines = ["# written by tests/golden/make_sampler_vectors.py (oracle only)",
             "# U seed g layer t -> u32"]
    for seed in (0, 1, 0xDEADBEEFCAFEF00D):
        for g in (0, 1, 1023, 262143, 2 ** 31 - 1):
            for layer in (0, 7, 31):
                for t in (0, 1, 2, 1000):
                    lines.append(f"U {seed} {g} {layer} {t} {O.draw_u32(seed, g, layer, t)}")
    lines.append("# S seed g layer v r n_excluded excluded... -> drawn...")
    cases = [
        (0, 5, 0, 128, 4, list(range(12))),
        (0, 127, 3, 128, 4, [1, 5, 9, 100, 101, 102, 77, 3, 2, 0, 64, 65]),
        (9, 4000, 8, 1024, 16, list(range(0, 96, 2))),
        (9, 4001, 8, 50, 16, list(range(48))),          # pool of 2 < r: whole pool
        (9, 4002, 8, 66, 16, list(range(48))),          # pool of 18, tight
        (2, 70000, 30, 2048, 32, list(range(100, 196))),
    ]
    for seed, g, layer, v, r, ex in cases:
        out = O.draw_random_sentinels(ex, v, r, seed, g, layer)
        lines.append("S %d %d %d %d %d %d %s -> %s" % (
            seed, g, layer, v, r, len(ex), " ".join(map(str, ex)), " ".join(map(str, out))))
    with open(os.path.join(HERE, "sampler_vectors.txt"), "w") as f:
        f.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()
