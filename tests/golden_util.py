"""Reader for tests/golden/z_seed*.txt (written by tests/golden/make_golden.py from the oracle): binary16 bit patterns."""
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_z_golden(seed):
    blocks = {}
    xor = total = None
    cur = None
    with open(os.path.join(GOLDEN, "z_seed%x.txt" % seed)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if line.startswith("block"):
                _, r0, c0 = line.split()
                cur = (int(r0), int(c0))
                blocks[cur] = []
            elif line.startswith("xor1M"):
                xor = int(line.split()[1], 16)
            elif line.startswith("sum1M"):
                total = int(line.split()[1])
            else:
                blocks[cur].append([int(v, 16) for v in line.split()])
    return {k: np.array(v, dtype=np.uint16) for k, v in blocks.items()}, xor, total
