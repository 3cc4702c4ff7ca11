"""Writes oracle_patterns.txt from the oracle alone (no CUDA code involved)."""
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import pattern  # noqa: E402

K8 = [0.30, 0.20, 0.10, 0.10, 0.10, 0.10, 0.05, 0.05]


def main():
    cdf = pattern.quantise_K(K8)
    lines = ["# K = " + " ".join(repr(k) for k in K8),
             "# cdf = " + " ".join(str(c) for c in cdf),
             "# seed iteration stream -> dp b"]
    for seed in (0, 1, 0x123456789ABCDEF):
        for it in (0, 1, 2, 3, (1 << 32) + 5):
            for stream in (0, 1, 7):
                dp, b = pattern.draw(cdf, seed, it, stream)
                lines.append(f"{seed} {it} {stream} -> {dp} {b}")
    with open(os.path.join(HERE, "oracle_patterns.txt"), "w") as f:
        f.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()
