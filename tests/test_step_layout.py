"""How the one-kernel step deals a logit block to its CTAs, checked on the host through the C-ABI (no GPU needed):
the shares partition the block, the inverse map agrees with them, the per-CTA bounds the kernel's tables rely on hold,
and the rules for small blocks (whole rows, or rows with CTAs of their own) do what they say."""
import ctypes

import numpy as np
import pytest

SMS = 148
GRANULE = 512


@pytest.fixture(scope="module")
def lib():
    import __graft_entry__ as entry
    entry.build()
    from paper_2602_10273_b200 import build as bld
    L = ctypes.CDLL(bld.LIB)
    i32p = ctypes.POINTER(ctypes.c_int32)
    L.psmc_step_layout.restype = ctypes.c_int
    L.psmc_step_layout.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, i32p, i32p, ctypes.c_int]
    L.psmc_step_share_of.restype = ctypes.c_int
    L.psmc_step_share_of.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int]
    return L


def layout(L, R, V, dt):
    out = (ctypes.c_int32 * 8)()
    shares = (ctypes.c_int32 * (SMS * 4 + 2))()
    rc = L.psmc_step_layout(R, V, dt, out, shares, len(shares))
    assert rc == 0
    d = dict(zip(("fits", "grid", "W", "gpr", "seg_cap", "per_row", "row_bytes16", "tail"), list(out)))
    return d, np.array(shares[: d["grid"] + 1], dtype=np.int64)


def shapes():
    rng = np.random.default_rng(5)
    fixed = [(4, 1024, 0), (8, 32000, 1), (16, 151936, 1), (32, 151936, 1), (512, 128256, 1), (64, 151936, 1),
             (100, 151936, 1), (148, 151936, 1), (149, 151936, 1), (1, 7, 0), (1, 8, 1), (3000, 16, 0), (4096, 128256, 1),
             (40, 1000, 0), (330, 2048, 1), (74, 50264, 1), (75, 50264, 1)]
    rand = [(int(rng.integers(1, 3000)), int(rng.choice([16, 96, 1000, 4096, 32000, 50264, 128256, 151936, 262144])),
             int(rng.integers(0, 2))) for _ in range(200)]
    return fixed + [s for s in rand if s[0] * s[1] < 1 << 29]


@pytest.mark.parametrize("R,V,dt", shapes())
def test_shares_partition_the_block(lib, R, V, dt):
    d, first = layout(lib, R, V, dt)
    esize = 2 if dt == 1 else 4
    per16 = 16 // esize
    assert d["row_bytes16"] == (V // per16) * 16 and d["tail"] == V % per16
    assert d["gpr"] == max(1, -(-d["row_bytes16"] // GRANULE))
    total = R * d["gpr"]
    assert 1 <= d["grid"] <= SMS and 1 <= d["W"] <= 23
    assert first[0] == 0 and first[-1] == total and (np.diff(first) > 0).all()       # a partition, no empty share
    if not d["fits"]:
        return
    rows_met = (first[1:] - 1) // d["gpr"] - first[:-1] // d["gpr"] + 1
    assert rows_met.max() <= d["seg_cap"] <= 48                                          # what the kernel's tables hold
    probe = np.unique(np.concatenate([first[:-1], first[1:] - 1, np.random.default_rng(R + V).integers(0, total, 64)]))
    for q in probe:
        b = lib.psmc_step_share_of(R, V, dt, int(q))
        assert 0 <= b < d["grid"] and first[b] <= q < first[b + 1], (q, b)
    assert lib.psmc_step_share_of(R, V, dt, total) == -1 and lib.psmc_step_share_of(R, V, dt, -1) == -1
    if R <= SMS:                                                                         # rows are never shared across rows
        assert (rows_met == 1).all()
        if d["gpr"] <= 256:
            assert d["grid"] == R and d["per_row"] == 0                                  # one whole row per CTA
        elif d["per_row"]:
            assert d["per_row"] == SMS // R and d["grid"] == R * d["per_row"]
            sizes = np.diff(first).reshape(R, d["per_row"])
            assert (sizes.sum(axis=1) == d["gpr"]).all() and sizes.max() - sizes.min() <= 1
    else:
        assert np.diff(first).max() - np.diff(first).min() <= 1                          # the even deal


def test_layout_argument_checks(lib):
    out = (ctypes.c_int32 * 8)()
    few = (ctypes.c_int32 * 4)()
    assert lib.psmc_step_layout(0, 10, 1, out, None, 0) != 0
    assert lib.psmc_step_layout(4, 10, 7, out, None, 0) != 0
    assert lib.psmc_step_layout(512, 128256, 1, out, few, 4) != 0          # array too short for 148 shares
    assert lib.psmc_step_layout(512, 128256, 1, out, None, 0) == 0 and out[1] == SMS
