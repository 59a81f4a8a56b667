"""Writes tests/golden/certified_seeds.json: for the full-size configurations c2, c3, c4 the first seed
(0, 1000, 2000, ...) that the ORACLE ALONE certifies, with the oracle's margin and a SHA-256 of its Z.

Calls only oracle/ (the plain-C nested sweep, Algorithm 5, on the oracle's own factors) and the seeded
input generators; nothing here touches the CUDA path.  The nested sweep is sequential: c2 takes seconds,
c3 minutes, c4 a good part of an hour on one core, which is why the result is stored instead of being
recomputed by every test run.  The GPU parity test hashes its own Z the same way (int32, row-major,
little-endian) and compares.

    python tests/golden/make_certified_seeds.py [2 3 4]
"""
import hashlib
import json
import os
import sys
import time

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
sys.path.insert(0, ROOT)

import oracle as O                      # noqa: E402
from oracle import cref                 # noqa: E402
from paper_2607_27042_b200 import workloads as W   # noqa: E402  (generators only: no method arithmetic)

MARGIN = 1e-9
OUT = os.path.join(HERE, "certified_seeds.json")


def z_digest(Z):
    return hashlib.sha256(np.ascontiguousarray(Z, dtype="<i4").tobytes()).hexdigest()


def certify(index):
    for t in range(6):
        seed = 1000 * t
        t0 = time.time()
        X, A, B = W.make_config(index, seed=seed)
        L, U, _, _ = O.feedback_factors(A, B)
        ref = cref.nested(X, L, U)
        rec = {"seed": seed, "margin": ref["margin"], "shape": list(X.shape), "z_sha256": z_digest(ref["Z"]),
               "z_abs_max": int(np.max(np.abs(ref["Z"]))), "seconds": round(time.time() - t0, 1),
               "oracle": "cref.nested (Algorithm 5) on oracle.feedback_factors"}
        print("c%d seed %d: margin %.3e (%s)" % (index, seed, ref["margin"], rec["seconds"]), flush=True)
        if ref["margin"] >= MARGIN:
            return rec
    raise SystemExit("c%d: no certified seed" % index)


if __name__ == "__main__":
    which = [int(a) for a in sys.argv[1:]] or [2, 3, 4]
    for index in which:
        rec = certify(index)
        table = json.load(open(OUT)) if os.path.exists(OUT) else {}     # re-read: another run may have added rows
        table["c%d" % index] = rec
        json.dump(table, open(OUT, "w"), indent=1, sort_keys=True)
