"""Host-side checks of the C-ABI library that need no GPU.

The library must load, export every symbol include/dit.h declares, and its
host-only entry points (the packer, size queries, argument validation) must
agree bit for bit with the oracle's integer results.
"""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import dit_oracle as O
from paper_2510_01565_b200 import binding as B
from paper_2510_01565_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return B.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "dit.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(dit_[a-z_0-9]+)\s*\(", header))
    assert {"dit_ctx_create", "dit_load_block_weights", "dit_step_forward", "dit_pack_requests"} <= declared
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in include/dit.h but not exported"
    assert set(B.EXPORTS) == declared


def test_pack_requests_bit_exact_against_oracle(lib):
    rng = np.random.default_rng(0)
    cases = [[(256, 256, 0)], [(1024, 1024, 512), (1024, 1024, 512)], [(16, 16, 0)],
             [(2048, 2048, 512), (256, 256, 512), (512, 512, 512), (1024, 1024, 512)], []]
    for _ in range(5):
        n = int(rng.integers(1, 9))
        cases.append([(int(rng.integers(1, 40)) * 16, int(rng.integers(1, 40)) * 16, int(rng.integers(0, 600))) for _ in range(n)])
    for reqs in cases:
        got = B.dit_pack_requests(reqs)
        lens, cu, row_req, row_local = O.pack_requests(reqs)
        assert got["token_lens"].dtype == np.int32 and got["cu_seqlens"].dtype == np.int32
        np.testing.assert_array_equal(got["token_lens"], lens)
        np.testing.assert_array_equal(got["cu_seqlens"], cu)
        np.testing.assert_array_equal(got["row_req"], row_req)
        np.testing.assert_array_equal(got["row_local"], row_local)
        assert got["total_tokens"] == int(cu[-1])


def test_pack_requests_rejects_bad_shapes(lib):
    for bad in [[(250, 256, 0)], [(256, 0, 0)], [(256, 256, -1)], [(-16, 16, 0)]]:
        with pytest.raises(B.DitError) as e:
            B.dit_pack_requests(bad)
        assert e.value.status == 2           # DIT_ERR_SHAPE
    total = C.c_int32()
    assert lib.dit_pack_requests(None, 1, None, None, None, None, C.byref(total)) == 1   # DIT_ERR_INVALID_ARG


def test_workspace_bytes_and_config_validation(lib):
    def ws(**kw):
        base = dict(hidden=3072, n_heads=24, head_dim=128, mlp_hidden=12288, cond_dim=3072, max_blocks=4,
                    max_total_tokens=9216, max_requests=2, ln_eps=1e-6, flags=0)
        base.update(kw)
        return lib.dit_workspace_bytes(C.byref(B.DitConfig(*base.values())))
    full = ws()
    # weights: 12 H^2 + 6 H C 16-bit parameters per block (C = H here), plus activations
    assert full > 4 * 18 * 3072 * 3072 * 2
    assert ws(max_blocks=8) - full >= 4 * 18 * 3072 * 3072 * 2
    assert ws(max_total_tokens=2 * 9216) > full
    for bad in [dict(hidden=3000), dict(head_dim=96, n_heads=32), dict(n_heads=23), dict(mlp_hidden=100),
                dict(max_requests=65), dict(max_requests=0), dict(max_blocks=0), dict(flags=16), dict(hidden=8192, n_heads=64),
                dict(flags=8 | 1), dict(flags=8 | 2), dict(flags=8 | 4),     # bf16 operands: plain blocks only
                dict(ln_eps=-1.0)]:
        assert ws(**bad) == 0, bad
    assert ws(flags=3) == full        # the QK variant bits are accepted and cost no workspace
    # the e4m3 mode adds the quantised copy [T, H + F] of the tile-produced operands and their row scales
    assert 9216 * (3072 + 12288) <= ws(flags=7) - full <= 9216 * (3072 + 12288) + 9216 * 4 + 4096
    assert ws(flags=8) == full        # so is the bf16-operand mode (same element sizes)
    assert lib.dit_workspace_bytes(None) == 0


def test_null_arguments_and_status_strings(lib):
    assert lib.dit_ctx_create(None, None, 0, None) == 1
    out = C.c_void_p()
    cfg = B.DitConfig(384, 6, 64, 1536, 384, 1, 256, 1, 1e-6, 0)
    assert lib.dit_ctx_create(C.byref(cfg), None, 0, C.byref(out)) == 1 and not out.value
    assert lib.dit_ctx_destroy(None) == 1
    assert lib.dit_step_forward(None, None, None, 0, None, 1, None, None) == 1
    assert lib.dit_last_launch_count(None) == 0
    assert lib.dit_last_error(None) == b""
    names = [lib.dit_status_string(i).decode() for i in range(9)]
    assert names[0] == "ok" and len(set(names)) == 9 and lib.dit_status_string(99) == b"unknown status"
