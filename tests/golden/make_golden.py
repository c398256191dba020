"""Writes the golden Z vectors of the A definition.  Calls only the CPU oracle.

Usage: python tests/golden/make_golden.py   (from the repository root)
Output: tests/golden/z_seed0.txt, z_seed1.txt : 32x32 blocks at (row0, col0) = (0, 0) and one block
far into the index space, as hex of the binary16 bit patterns (every Z is a binary16 number by definition), plus an XOR
checksum and a sum of the patterns of a 2^20-entry block.  There is no printed example in the paper to take these from; the paper fixes
only the distribution (Section 3.3), which tests/test_oracle_a_matrix.py checks separately.
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
import oracle  # noqa: E402

BLOCKS = [(0, 0), (16352, 45088736)]   # (row0, col0)


def main():
    here = os.path.dirname(os.path.abspath(__file__))
    for seed in (0, 1, 0x123456789ABCDEF):
        name = "z_seed%x.txt" % seed
        with open(os.path.join(here, name), "w") as f:
            f.write("# Z(seed=%d) golden blocks; rows of 32 hex binary16 bit patterns\n" % seed)
            for (r0, c0) in BLOCKS:
                z = oracle.z_block(seed, r0, 32, c0, 32)
                zh = z.astype(np.float16)
                assert np.array_equal(zh.astype(np.float32), z)
                f.write("block %d %d\n" % (r0, c0))
                for r in range(32):
                    f.write(" ".join("%04x" % v for v in zh[r].view(np.uint16)) + "\n")
            big = oracle.z_block(seed, 0, 1024, 1000, 1024).astype(np.float16).view(np.uint16)
            f.write("xor1M %04x\n" % int(np.bitwise_xor.reduce(big.ravel())))
            f.write("sum1M %d\n" % int(big.ravel().astype(np.uint64).sum()))


if __name__ == "__main__":
    main()
