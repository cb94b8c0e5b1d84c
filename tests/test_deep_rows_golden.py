"""The stored full-depth oracle rows (tests/golden/deep_rows.npz) still belong to the oracle as it stands.

The file is written by tests/golden/make_deep_rows.py from `oracle/` and the seeded generators only.
Here: the hash of those sources inside the file equals the current one, every entry the GPU parity
tests read is present and well formed, and the cheapest entry (the 512^2 request through 4 blocks) is
regenerated through the same script and equals the stored one.
"""
import importlib.util
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))


def _script():
    spec = importlib.util.spec_from_file_location("make_deep_rows", os.path.join(HERE, "golden", "make_deep_rows.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_stored_rows_match_the_current_oracle_sources_and_are_complete():
    M = _script()
    with np.load(M.OUT_PATH) as z:
        assert str(z["source_sha256"]) == M.source_hash(), "oracle or generator sources changed: regenerate deep_rows.npz"
        assert int(z["seed"]) == M.SEED
        expect = {"cfg2_512": (1536, 4), "cfg3_1024x2": (4608, 4), "cfg4_2048": (16896, 4), "cfg5_mixed8": (None, 8)}
        for cfg, reqs in M.ENTRIES.items():
            for r in reqs:
                key = f"{cfg}/r{r}"
                rows, out = z[key + "/rows"], z[key + "/out"]
                L, nb = int(z[key + "/n_tokens"]), int(z[key + "/n_blocks"])
                assert nb == expect[cfg][1] and (expect[cfg][0] is None or L == expect[cfg][0])
                assert rows.shape == (M.N_ROWS,) and out.shape == (M.N_ROWS, 3072) and out.dtype == np.float32
                assert {0, 127, 128, L - 1} <= set(rows.tolist()) and rows.max() == L - 1 and len(set(rows.tolist())) == M.N_ROWS
                assert np.isfinite(out).all()
                # the stored rows are a fair sample of the request: their rms is that of the whole output
                assert abs(float(z[key + "/rms_rows"]) / float(z[key + "/rms_full"]) - 1.0) < 0.1
        assert int(z["cfg5_mixed8/r0/n_tokens"]) == 4608 and int(z["cfg5_mixed8/r5/n_tokens"]) == 16896


def test_cheapest_entry_regenerates_to_the_stored_values():
    M = _script()
    fresh = M.make_entry("cfg2_512", [0])
    with np.load(M.OUT_PATH) as z:
        for k, v in fresh.items():
            stored = z[k]
            if k.endswith("/out"):
                # fp64 results rounded once to fp32: a different BLAS thread count may move the last fp64
                # bits, which can flip an fp32 rounding; anything beyond that is a changed oracle
                rms = float(z["cfg2_512/r0/rms_full"])
                assert np.abs(stored.astype(np.float64) - v.astype(np.float64)).max() <= 1e-6 * rms
            elif k.endswith("/rows") or k.endswith("/n_tokens") or k.endswith("/n_blocks"):
                np.testing.assert_array_equal(stored, v)
            else:
                assert abs(float(stored) - float(v)) <= 1e-9 * abs(float(v))
