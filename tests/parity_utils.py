"""Shared machinery of the GPU parity tests: runs the oracle window by window on
the seeded workload, keeps its state (incremental representative table), and
compares the CUDA path's outputs with the tolerances the project states:

  * selected block sets: identical, except blocks whose oracle score lies within
    1e-3 (relative) of the cut-off score -- those are counted separately;
  * activation bias, probe-query, scores (fp32): |a - b| <= 1e-4 * max(|b|, floor),
    floor = 1 for cosines, 1e-3 * max|b| for phi (phi -> 0 where q = mean), 1e-2 * max|b| for
    probe channels (signed sums that cancel);
  * attention (bf16 in, fp32 accumulate): max abs err <= 2e-2, mean abs err <= 2e-3.
"""
from __future__ import annotations

import numpy as np

from oracle import actqkv_oracle as orc
from paper_2502_13542_b200 import workloads as wl

REL_TOL = 1e-4
ATT_MAX_ABS = 2e-2
ATT_MEAN_ABS = 2e-3
NEAR_TIE_REL = 1e-3


def rel_err_floor(got, want, floor):
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    return float(np.max(np.abs(got - want) / np.maximum(np.abs(want), floor))) if want.size else 0.0


def assert_rel(got, want, floor, what, tol=REL_TOL):
    e = rel_err_floor(got, want, floor)
    assert e <= tol, f"{what}: rel err {e:.3e} > {tol:.1e}"
    return e


def assert_phi_like(got, want, what, floor_frac=1e-3):
    want = np.asarray(want, np.float64)
    floor = floor_frac * max(float(np.max(np.abs(want))), 1e-30)
    return assert_rel(got, want, floor, what)


def assert_probe(got, want, what):
    """A probe channel is a signed sum of W terms that largely cancel, so an fp32 sum cannot
    be relatively accurate in its small channels: 1e-4 relative for channels above 1% of the
    largest, 1e-6 of the largest (a few fp32 ulps) below."""
    return assert_phi_like(got, want, what, floor_frac=1e-2)


def attention_errors(got, want):
    d = np.abs(np.asarray(got, np.float64) - np.asarray(want, np.float64))
    return float(d.max()), float(d.mean())


def assert_attention(got, want, what, dtype="bf16"):
    """fp32-stored output against the raw fp64 oracle: max abs <= 2e-2, mean abs <= 2e-3."""
    mx, mean = attention_errors(got, want)
    assert mx <= ATT_MAX_ABS and mean <= ATT_MEAN_ABS, f"{what}: max abs {mx:.3e}, mean abs {mean:.3e}"
    return mx, mean


def assert_attention_bf16_out(got, want, what):
    """bf16-stored output: storing alone costs up to |o| * 2^-9 (outlier value channels reach
    |o| ~ 30), so the bound is the stated one plus one bf16 half-ulp of the stored value."""
    d = np.abs(np.asarray(got, np.float64) - np.asarray(want, np.float64))
    bound = ATT_MAX_ABS + np.abs(np.asarray(want, np.float64)) * 2.0 ** -8
    assert np.all(d <= bound), f"{what}: worst excess {float((d - bound).max()):.3e}"
    assert d.mean() <= ATT_MEAN_ABS + np.abs(want).mean() * 2.0 ** -9, f"{what}: mean abs {d.mean():.3e}"
    return float(d.max()), float(d.mean())


def compare_selection(got_idx, got_count, oracle_res, what):
    """got_idx [Hkv, cap] int32 (-1 padded), got_count int.  Returns number of near-tie
    differences; asserts everything else is identical."""
    near_diffs = 0
    c = oracle_res["c"]
    if got_count != c:
        assert oracle_res["fragile"], f"{what}: count {got_count} != oracle {c} (B={oracle_res['b_real']})"
        return -1
    for g, want in enumerate(oracle_res["sel"]):
        got = got_idx[g][:got_count]
        assert np.all(got_idx[g][got_count:] == -1), f"{what}: head {g} tail not -1"
        assert np.all(np.diff(got) > 0), f"{what}: head {g} not strictly ascending"
        if np.array_equal(got, want):
            continue
        diff = set(got.tolist()) ^ set(want.tolist())
        near = set(oracle_res["near"][g].tolist())
        assert diff <= near, (f"{what}: head {g} differs outside the near-tie band: "
                              f"{sorted(diff - near)} tau={oracle_res['tau'][g]}")
        near_diffs += len(diff)
    return near_diffs


from oracle.runner import OracleRunner  # noqa: E402,F401  (re-exported for the tests)


# host <-> device plumbing lives with the input generators
to_device = wl.to_device
to_numpy = wl.to_numpy
