"""Writes tests/golden/sample_hash.txt: frozen values of the sampling hash (seed, layer, dst, k).
Calls only the oracle.  Run from the repository root: python tests/golden/make_sample_hash.py"""
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
import oracle  # noqa: E402

out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "sample_hash.txt")
with open(out, "w") as f:
    f.write("# seed layer dst k hash64(hex) -- sampling hash of the neighbour sampler (Sect. 3.9, sampling paragraph)\n")
    for seed in (0, 1, 2**63 + 5):
        for layer in (0, 2):
            for dst in (0, 1, 110_999_999):
                for k in (0, 14):
                    h = oracle._lib().to_sample_hash(seed, layer, dst, k)
                    f.write("%d %d %d %d %016x\n" % (seed, layer, dst, k, h))
