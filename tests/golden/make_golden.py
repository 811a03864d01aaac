"""Writes the frozen golden vectors of the hash family and the Random Mask
generator.  Calls only ``oracle/``; run from the repository root:

    python tests/golden/make_golden.py

The files guard against silent changes of the family (the paper does not fix
one, Section 3.1 only says each entry picks s random outputs and a sign).
"""
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402


def main():
    rows = []
    for seed in (0, 1, 0x5EED + 1, 0x5EED + 2, 0x5EED + 3, 0xFFFFFFFFFFFFFFFF):
        for s in (1, 2, 4):
            for k in (1, 7, 1024, 2048, 4096, 1000003, (1 << 32) - 1):
                for j in (0, 1, 2, 31, 4095, 65535, 16777215, (1 << 32) - 2):
                    r = (j + k) % s
                    h = oracle.sjlt_hash(seed, s, j, r)
                    bucket = ((h >> 32) * k) >> 32
                    sign = -1 if h & 1 else 1
                    rows.append(f"{seed} {s} {k} {j} {r} {h} {bucket} {sign}")
    with open(os.path.join(HERE, "sjlt_hash.txt"), "w") as f:
        f.write("# seed s k j r H bucket sign  -- this project's hash family (SplitMix64 stream,\n"
                "# multiply-shift bucket, low bit sign); written by make_golden.py from oracle/ only\n")
        f.write("\n".join(rows) + "\n")

    rows = []
    for (p, kp, seed) in ((65536, 8192, 0), (4194304, 65536, 0), (768, 128, 3), (3072, 128, 4),
                          (4096, 64, 5), (14336, 64, 6), (100, 100, 7), (1000, 1, 8)):
        idx = oracle.random_mask(p, kp, seed)
        head = " ".join(str(int(v)) for v in idx[:32])
        rows.append(f"{p} {kp} {seed} {int(idx.astype('uint64').sum())} {head}")
    with open(os.path.join(HERE, "random_mask.txt"), "w") as f:
        f.write("# p kprime seed sum(idx) first<=32 ascending indices -- Random Mask (Section 3.2),\n"
                "# Floyd subset sampling on the SplitMix64 stream; written by make_golden.py from oracle/ only\n")
        f.write("\n".join(rows) + "\n")


if __name__ == "__main__":
    main()
