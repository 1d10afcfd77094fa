"""Writes the stored expected values under tests/golden/ by calling the CPU oracle only.

    python tests/golden/make_golden.py

cfg1_kept_idx.txt : kept indices of the tiny configuration (L 2048, 2 KV heads, group 4, 16 soft
                    tokens, budget 256, pool 7), one line per KV head, from oracle.evict_layer on
                    jq_workloads.CFG1 layer 0.  First line: CRC32 of the K, V, Qwin bit patterns, so a
                    drift of the seeded generator is told apart from a drift of the oracle.
The paper prints no worked example of the eviction pass (Eq. 3 and the inference section give
definitions only), so no value here is the paper's.
"""
import os
import sys
import zlib

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402
import jq_workloads as W  # noqa: E402


def cfg1_lines():
    wl = W.CFG1
    K, V, Q, _ = W.make_layer(wl)
    crc = [zlib.crc32(a.tobytes()) for a in (K, V, Q)]
    _, _, idx = oracle.evict_layer(K, V, Q, wl.budget, wl.pool)
    lines = ["crc32 %d %d %d" % tuple(crc)]
    lines += [" ".join(str(int(j)) for j in row) for row in idx]
    return lines


if __name__ == "__main__":
    with open(os.path.join(HERE, "cfg1_kept_idx.txt"), "w") as f:
        f.write("\n".join(cfg1_lines()) + "\n")
    print("written")
