"""Writes tests/golden/deep_rows.npz: fp64-oracle outputs of the full-depth block stacks, sampled rows.

The long requests of the benchmark configurations (2 x 1024^2 through 4 blocks, 2048^2 through 4
blocks, and the 1024^2 / 2048^2 requests of the mixed batch through 8 blocks) take the CPU oracle
minutes each, too long for a test run.  This script runs them once, request by request, through
`oracle.dit_oracle.block_forward` (every row of the request at every block: attention needs all
keys), and stores a fixed sample of output rows per request.  The GPU parity tests load the file and
compare the library's output on the same seeded inputs.

It imports only the oracle and the seeded input generators; nothing here touches the CUDA path, so
every stored number is the oracle's.

Stored per (configuration, request):
  rows      int32  [n]      row indices inside the request (0, 127, 128, L-1 and seeded random ones)
  out       float32 [n, H]  the oracle's fp64 output rows, rounded once to fp32 for storage
                            (relative 6e-8, five orders below the parity bar)
  rms_full  float64         sqrt(mean(out^2)) over ALL L x H outputs of the request
  rms_rows  float64         the same over the stored rows only
and, for the whole file, the seed and a SHA-256 of the oracle and generator sources that made it.

Usage:  python tests/golden/make_deep_rows.py            (all entries; about 25 minutes on 8 cores)
        python tests/golden/make_deep_rows.py cfg2_512    (only the named configurations, merged
                                                           into the existing file)
"""
from __future__ import annotations

import hashlib
import math
import os
import sys
import time

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import dit_oracle as O                      # noqa: E402
from paper_2510_01565_b200 import workloads as W        # noqa: E402

OUT_PATH = os.path.join(HERE, "deep_rows.npz")
SEED = 0
N_ROWS = 64
ROW_SEED = 20251001

# configuration -> requests whose full-depth output is stored
ENTRIES = {
    "cfg2_512": [0],
    "cfg3_1024x2": [0, 1],
    "cfg4_2048": [0],
    "cfg5_mixed8": [0, 5],        # a 1024^2 request and the 2048^2 request of the seeded mix
}

HASHED_SOURCES = ("oracle/dit_oracle.py", "paper_2510_01565_b200/workloads.py")


def source_hash() -> str:
    h = hashlib.sha256()
    for rel in HASHED_SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def sample_rows(length: int, cfg: str, r: int) -> np.ndarray:
    """Fixed rows (first, both sides of the first 128-row tile edge, last) plus seeded random ones."""
    fixed = sorted({i for i in (0, 127, 128, length - 1) if 0 <= i < length})
    rng = np.random.default_rng([ROW_SEED, sum(cfg.encode()), r])
    rest = [i for i in rng.permutation(length).tolist() if i not in fixed]
    return np.array(sorted(fixed + rest[:max(0, min(N_ROWS, length) - len(fixed))]), dtype=np.int32)


def oracle_request(wl: W.Workload, r: int) -> np.ndarray:
    """The oracle's output for request r of the workload through all its blocks, fp64 [L_r, H]."""
    x = W.bf16_to_f64(wl.tokens[r])
    cond = W.bf16_to_f64(wl.cond[r])
    for b in range(wl.n_blocks):
        w = {k: W.bf16_to_f64(v) for k, v in wl.weights[b].items()}     # one block widened at a time
        x = O.block_forward(x, cond, w, wl.dims.n_heads, wl.dims.ln_eps)
    return x


def make_entry(cfg: str, requests) -> dict:
    wl = W.make_workload(cfg, seed=SEED)
    res = {}
    for r in requests:
        t0 = time.time()
        y = oracle_request(wl, r)
        rows = sample_rows(y.shape[0], cfg, r)
        key = f"{cfg}/r{r}"
        res[key + "/rows"] = rows
        res[key + "/out"] = y[rows].astype(np.float32)
        res[key + "/rms_full"] = np.float64(math.sqrt(np.mean(y ** 2)))
        res[key + "/rms_rows"] = np.float64(math.sqrt(np.mean(y[rows] ** 2)))
        res[key + "/n_tokens"] = np.int32(y.shape[0])
        res[key + "/n_blocks"] = np.int32(wl.n_blocks)
        print(f"{key}: L = {y.shape[0]}, {wl.n_blocks} blocks, {time.time() - t0:.0f} s", flush=True)
    return res


def main(argv) -> None:
    names = argv or list(ENTRIES)
    data = {}
    if argv and os.path.exists(OUT_PATH):
        with np.load(OUT_PATH) as old:
            data = {k: old[k] for k in old.files}
        if str(data["source_sha256"]) != source_hash():
            raise SystemExit("the stored file was made by other oracle/generator sources: regenerate all entries")
    for cfg in names:
        data.update(make_entry(cfg, ENTRIES[cfg]))
    data["seed"] = np.int32(SEED)
    data["source_sha256"] = np.array(source_hash())
    np.savez(OUT_PATH, **data)
    print("wrote", OUT_PATH)


if __name__ == "__main__":
    main(sys.argv[1:])
