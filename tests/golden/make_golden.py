"""Writes the stored expected values under tests/golden/.  Calls ONLY the CPU oracle.

    python -m tests.golden.make_golden

appc_3groups.txt -- the layout of the paper's App. C example ("Detailed Planning Example"):
a navigation map of three object groups, of which Group 2 and Group 3 are retrieved, then
the instruction and trajectory as new tokens.  The paper prints the layout only; the token
counts (group lengths 9, 14, 6; 5 new tokens) and the seeded bf16 values are made up here.
"""
import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import enl_oracle as orc  # noqa: E402

HERE = os.path.dirname(os.path.abspath(__file__))


def appc_case():
    Hq, Hkv, D = 4, 2, 16
    lens = [9, 14, 6]
    g = torch.Generator().manual_seed(20251018)
    cache = orc.OracleCache(1, Hq, Hkv, D)
    for gid, n in enumerate(lens):
        k = torch.randn(n, Hkv, D, generator=g).to(torch.bfloat16)
        v = torch.randn(n, Hkv, D, generator=g).to(torch.bfloat16)
        cache.group_store(gid, 0, k, v)
    q = torch.randn(5, Hq, D, generator=g).to(torch.bfloat16)
    kn = torch.randn(5, Hkv, D, generator=g).to(torch.bfloat16)
    vn = torch.randn(5, Hkv, D, generator=g).to(torch.bfloat16)
    return cache, [1, 2], q, kn, vn


def main():
    cache, sel, q, kn, vn = appc_case()
    out, mass, off = cache.attend(0, sel, q, kn, vn)
    with open(os.path.join(HERE, "appc_3groups.txt"), "w") as f:
        f.write("# App. C layout: pool of 3 groups, Group 2 and Group 3 selected (ids 1, 2), 5 new tokens.\n")
        f.write("# Lengths and values are synthetic (seed 20251018); written by make_golden.py from the oracle.\n")
        f.write("sel_off = " + " ".join(str(int(x)) for x in off) + "\n")
        f.write("mass_row_last_head0 = " + " ".join(float(x).hex() for x in mass[-1, 0]) + "\n")
        f.write("out_row_last_head0_first4 = " + " ".join(float(x).hex() for x in out[-1, 0, :4]) + "\n")


if __name__ == "__main__":
    main()
