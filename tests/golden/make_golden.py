"""Writes tests/golden/config1_hashes.txt from the CPU oracle ONLY (never from the
CUDA path).  The file freezes the oracle's chained hashes of the tiny
configuration's stored session (500 tokens) and its 560-token continuation, so
an accidental change to the oracle's arithmetic is caught.  The paper prints no
hash values to compare with (Sec. 4.3 names only a "cumulative prefix hash").

    python -m tests.golden.make_golden
"""
import os

import numpy as np

from oracle import oracle as orc
from paper_2607_17181_b200 import workloads as wl


def config1_streams():
    g = wl.rng(1)
    _s1 = wl.tokens(g, 300)
    s2 = wl.tokens(g, 500)
    cont = wl.continuation(g, s2, 560, 350)
    return s2, cont


def main():
    sess, cont = config1_streams()
    hs = orc.block_hash(sess, 16, wl.HASH_SEED)
    hc = orc.block_hash(cont, 16, wl.HASH_SEED)
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "config1_hashes.txt")
    with open(path, "w") as f:
        f.write("# oracle chained hashes, tiny configuration: 31 stored-session blocks then 35 continuation blocks\n")
        f.write("# (B=16, seed 0x54414C41524941); written by tests/golden/make_golden.py from oracle/ only\n")
        for h in np.concatenate([hs, hc]):
            f.write(f"{int(h):016x}\n")
    print("wrote", path, hs.size, hc.size)


if __name__ == "__main__":
    main()
