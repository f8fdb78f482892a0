"""Writes the full-depth golden digests under tests/golden/ from the CPU oracle alone.

    python tests/golden/make_golden.py [--only bvn5 mw4 ...] [--threads T]

For a sample of the matrices of the large workload configurations the oracle runs the
COMPLETE decomposition (Birkhoff-von Neumann until the balanced matrix is exhausted, paper
Sec. 3.1; greedy max-weight with the configuration's largest budget, Sec. 3.2) and one line
per matrix is stored:  row  count  sha256.  The digest covers, in this order, count as a
little-endian int32, the first `count` permutations (count * N bytes) and the first `count`
coefficients / durations (little-endian int32). A GPU test hashes its own output the same
way; a single differing destination anywhere in the tens of thousands of matchings of a
schedule changes the digest. This script imports the oracle and the seeded input generator
and nothing else of the repository; a complete pass costs minutes per matrix at N = 256,
which is why the values are stored instead of being recomputed by every test run.
"""
from __future__ import annotations

import argparse
import hashlib
import os
import sys
import time

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2605_26845_b200.workload import CONFIGS, SEED, bvn_capacity, make_demand  # noqa: E402

# what is stored: (kind, configuration) -> number of matrices, spread evenly over the batch
PLAN = {
    ("bvn", 3): 512,
    ("bvn", 4): 64,
    ("bvn", 5): 8,
    ("mw", 4): 1024,
    ("mw", 5): 256,
}


def sample_rows(B: int, n: int) -> np.ndarray:
    return np.arange(0, B, max(1, B // n))[:n]


def digest(count: int, perm: np.ndarray, val: np.ndarray) -> str:
    """perm: [k_max, N] uint8, val: [k_max] int32 of one matrix."""
    h = hashlib.sha256()
    h.update(np.int32(count).astype("<i4").tobytes())
    h.update(np.ascontiguousarray(perm[:count]).tobytes())
    h.update(np.ascontiguousarray(val[:count]).astype("<i4").tobytes())
    return h.hexdigest()


def golden_path(kind: str, cfg: int) -> str:
    return os.path.join(HERE, f"{kind}_full_depth_config{cfg}.txt")


def write_one(kind: str, cfg: int, threads: int, group: int) -> None:
    c = CONFIGS[cfg]
    N, B = c["N"], c["B"]
    rows = sample_rows(B, PLAN[(kind, cfg)])
    D = make_demand(cfg)
    k_max = bvn_capacity(N) if kind == "bvn" else max(c["k_max"])
    lines = []
    t0 = time.perf_counter()
    for g0 in range(0, len(rows), group):               # a few matrices at a time keeps memory small
        part = rows[g0:g0 + group]
        if kind == "bvn":
            ref = oracle.bvn_decompose(D[part], k_max, threads=threads, want_aug=False)
            val = ref["coef"]
        else:
            ref = oracle.mw_decompose(D[part], k_max, threads=threads, want_residual=False)
            val = ref["dur"]
        for q, r in enumerate(part):
            st = int(ref["status"][q])
            assert st == 0 or (kind == "mw" and st == 1), (kind, cfg, int(r), st)
            lines.append(f"{int(r)} {int(ref['count'][q])} {digest(int(ref['count'][q]), ref['perm'][q], val[q])}")
        print(f"{kind} config {cfg}: {g0 + len(part)}/{len(rows)} matrices, "
              f"{time.perf_counter() - t0:.0f} s", flush=True)
    what = ("Birkhoff-von Neumann decomposition run to completion (paper Sec. 3.1)" if kind == "bvn" else
            f"greedy max-weight decomposition with budget k_max = {k_max} (paper Sec. 3.2)")
    with open(golden_path(kind, cfg), "w") as f:
        f.write(f"# {what} of workload configuration {cfg}\n"
                f"# (N = {N}, B = {B}, seed {SEED}), computed by the CPU oracle alone:\n"
                f"# written by tests/golden/make_golden.py. Columns: matrix index, number of matchings,\n"
                f"# sha256 over (count as int32, count*N permutation bytes, count int32 values), little endian.\n")
        f.write("\n".join(lines) + "\n")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--only", nargs="*", default=None, help="e.g. bvn5 mw4 (default: everything in PLAN)")
    ap.add_argument("--threads", type=int, default=oracle.hardware_threads())
    args = ap.parse_args()
    oracle.build()
    for (kind, cfg) in PLAN:
        if args.only and f"{kind}{cfg}" not in args.only:
            continue
        write_one(kind, cfg, args.threads, group=max(args.threads, 8))


if __name__ == "__main__":
    main()
