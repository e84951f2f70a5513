"""Exhaustive check of the row encoder against the oracle's quantizer over ALL 2^32 float32 bit
patterns (every finite value, both zeros, infinities, every NaN payload), plane by plane.

Not collected by pytest (about 17 minutes on a B200 host, dominated by the CPU side):
    python tests/exhaustive_encode.py [first_chunk last_chunk]
Each of the 32 chunks covers 2^27 consecutive bit patterns; widths 1, 2, 4, 8, both range limiters,
ranges 1.0 and 0.37.  Exit status 0 means no plane word differed.
"""
import os
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import oracle                                              # noqa: E402
from paper_1905_13389_b200 import binding as mpq          # noqa: E402


def main(first=0, last=31):
    dev = torch.device("cuda:0")
    torch.cuda.set_device(0)
    k, chunk = 1 << 20, 1 << 27
    rows = chunk // k
    combos = [(s, a, b) for s in (1.0, 0.37) for a in (0, 1) for b in (1, 2, 4, 8)]
    bad, t0 = 0, time.time()
    for c in range(first, last + 1):
        x = np.arange(c * chunk, (c + 1) * chunk, dtype=np.uint64).astype(np.uint32).view(np.float32).reshape(rows, k)
        xd = torch.from_numpy(x).to(dev)
        for (scale, act, bits) in combos:
            sd = torch.tensor([scale], dtype=torch.float32, device=dev)
            planes = mpq.encode(xd, sd, bits, 0, act).cpu().numpy().view(np.uint32)
            u = oracle.levels(oracle.quantize(x, np.float32(scale), bits, act=act), bits)
            for p in range(bits):
                ref = np.packbits(((u >> p) & 1).astype(np.uint8), axis=1, bitorder="little").view(np.uint32)
                if not np.array_equal(ref, planes[p]):
                    bad += 1
                    print("MISMATCH chunk", c, "range", scale, "act", act, "bits", bits, "plane", p,
                          int((ref != planes[p]).sum()), "words", flush=True)
        print("chunk", c, "done", round(time.time() - t0), "s; mismatching planes so far:", bad, flush=True)
    print("mismatching planes:", bad)
    return 1 if bad else 0


if __name__ == "__main__":
    a = [int(v) for v in sys.argv[1:3]]
    sys.exit(main(*a) if a else main())
