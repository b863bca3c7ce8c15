"""The comparison helper of the GPU parity tests, exercised on the CPU with a stand-in for the CUDA export.

A hybrid group whose two candidates have (nearly) equal L1 error may get either mask from an implementation that
sums in float32; the helper then demands the stored form of the oracle's other candidate, bit for bit.
"""
import copy

import numpy as np
import pytest

from oracle import innerq_oracle as O
from tests import _parity as P


def _cache_with_tied_groups():
    # 1 unit, G = 32, 2 bits, hybrid.  Key token 0 of the packed part is constant inside every group (both
    # candidates reconstruct it exactly: a tie, which the oracle gives to symmetric); the rest is random.
    rng = np.random.default_rng(3)
    N, D = 4 + 96 + 16, 128
    K = rng.standard_normal((1, 1, N, D)).astype(np.float16)
    V = rng.standard_normal((1, 1, N, D)).astype(np.float16)
    K[0, 0, 4] = np.repeat(np.array([1.5, -0.75, 2.0, 0.5], dtype=np.float16), 32)
    oc = O.OracleCache(1, 1, 1, D, N + 8, 32, 2, 2, w_sink=4, w_recent=16, k_normalize=0)
    oc.prefill(K, V)
    return oc


def test_a_contested_group_resolved_the_other_way_must_hold_the_other_candidate():
    o = _cache_with_tied_groups().export()
    assert not (o["k_scale"][0, 0] & 0x8000).any()            # ties went to symmetric
    g = copy.deepcopy(o)
    assert P.assert_export_equal(g, o, O.INNER, 32) == 0
    # the stand-in chooses asymmetric for group 1 of that token and stores the asymmetric candidate: accepted
    g["k_scale"][0, 0, 1] = o["k_alt_scale"][0, 0, 1]
    g["k_zero"][0, 0, 1] = o["k_alt_zero"][0, 0, 1]
    g["k_code"][0, 0, 32:64] = o["k_alt_code"][0, 0, 32:64]
    assert (g["k_scale"][0, 0, 1] & 0x8000) and g["k_zero"][0, 0, 1] == np.array(-0.75, np.float16).view(np.uint16)
    assert P.assert_export_equal(g, o, O.INNER, 32) == 1
    # ... but not with the symmetric candidate's codes left in place, nor with another zero-point
    bad = copy.deepcopy(g)
    bad["k_code"][0, 0, 32:64] = o["k_code"][0, 0, 32:64]
    with pytest.raises(AssertionError, match="k_code"):
        P.assert_export_equal(bad, o, O.INNER, 32)
    bad = copy.deepcopy(g)
    bad["k_zero"][0, 0, 1] ^= 1
    with pytest.raises(AssertionError, match="k_zero"):
        P.assert_export_equal(bad, o, O.INNER, 32)


def test_an_uncontested_group_must_keep_the_oracles_mask():
    o = _cache_with_tied_groups().export()
    g = copy.deepcopy(o)
    clear = np.argwhere(np.abs(o["v_err_asym"] - o["v_err_sym"]) > 1e-2 * np.maximum(o["v_err_asym"], o["v_err_sym"]))[0]
    u, j, c = clear
    g["v_scale"][u, j, c] = o["v_alt_scale"][u, j, c]
    g["v_zero"][u, j, c] = o["v_alt_zero"][u, j, c]
    g["v_code"][u, 32 * j:32 * j + 32, c] = o["v_alt_code"][u, 32 * j:32 * j + 32, c]
    with pytest.raises(AssertionError, match="uncontested"):
        P.assert_export_equal(g, o, O.INNER, 32)
