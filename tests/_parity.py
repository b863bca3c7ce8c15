"""Helpers for comparing the CUDA path with the CPU oracle (test infrastructure)."""
from __future__ import annotations

import numpy as np

from oracle import innerq_oracle as O

# Attention outputs: |err| <= OUT_RTOL * max|out_row| + OUT_ATOL per (batch, query head) row
OUT_RTOL, OUT_ATOL = 2e-3, 1e-3
# A hybrid group is "contested" when the two candidates' L1 errors differ by less than this
# relative margin in the oracle's float64 sums; the CUDA path sums in float32 in another order,
# so either mask value is correct there.
CONTEST_RTOL = 1e-4
# Largest share of a tensor's groups that may be contested AND resolved the other way (observed: 1e-5 .. 2e-4)
MAX_FLIP_SHARE = 4e-4


def assert_outputs_close(out_gpu, out_ref, what=""):
    out_gpu = np.asarray(out_gpu, dtype=np.float64)
    out_ref = np.asarray(out_ref, dtype=np.float64)
    assert out_gpu.shape == out_ref.shape
    assert np.all(np.isfinite(out_gpu)), f"{what}: non-finite output"
    tol = OUT_RTOL * np.abs(out_ref).max(axis=-1, keepdims=True) + OUT_ATOL
    err = np.abs(out_gpu - out_ref)
    worst = float((err / tol).max())
    assert worst <= 1.0, f"{what}: max err/tol = {worst:.3f}"
    return worst


def _contested(e_a, e_s):
    return np.abs(e_a - e_s) <= CONTEST_RTOL * np.maximum(e_a, e_s)


def assert_store_equal(g, o, name, kind, G, hybrid):
    """Compare one tensor's canonical arrays (g: CUDA export, o: oracle export).  Returns #contested flips.

    Where both sides chose the same mask, codes, scale bits and zero bits must be identical.  Where they chose
    differently the group must be contested, and the CUDA path's codes, scale bits and zero bits must be identical to
    the oracle's OTHER candidate (the one its mask did not select), so every stored bit of every group is checked."""
    sc_g, sc_o = g[f"{name}_scale"], o[f"{name}_scale"]
    assert sc_g.shape == sc_o.shape, (name, sc_g.shape, sc_o.shape)
    flag_g, flag_o = (sc_g & 0x8000) != 0, (sc_o & 0x8000) != 0
    flips = flag_g != flag_o
    n_flips = int(flips.sum())
    if n_flips:
        assert hybrid, f"{name}: mask differs in a non-hybrid mode"
        cont = _contested(o[f"{name}_err_asym"], o[f"{name}_err_sym"])
        assert np.all(cont[flips]), f"{name}: {int((flips & ~cont).sum())} uncontested groups chose another mode"
        assert n_flips <= max(2, int(MAX_FLIP_SHARE * flips.size)), f"{name}: too many contested flips ({n_flips})"
    # expected stored form per group: the oracle's chosen candidate, or its other one where the masks differ
    sc_e = np.where(flips, o[f"{name}_alt_scale"], sc_o)
    ze_e = np.where(flips, o[f"{name}_alt_zero"], o[f"{name}_zero"])
    assert np.array_equal(sc_g, sc_e), f"{name}_scale"
    assert np.array_equal(g[f"{name}_zero"], ze_e), f"{name}_zero"
    # zero-point is 0 wherever the mask is 0
    assert not np.any(g[f"{name}_zero"][~flag_g])
    cg, co = g[f"{name}_code"], o[f"{name}_code"]
    assert cg.shape == co.shape
    U, n, D = cg.shape
    if kind == "row":
        flips_e = np.repeat(flips, G, axis=-1).reshape(U, n, D)
    else:
        flips_e = np.repeat(flips, G, axis=1).reshape(U, n, D)
    assert np.array_equal(cg, np.where(flips_e, o[f"{name}_alt_code"], co)), f"{name}_code"
    return n_flips


def assert_export_equal(g, o, grouping, G, k_hybrid=True, v_hybrid=True):
    """Whole-cache comparison: counts, windows and norm bit-exact; packed stores via assert_store_equal."""
    for key in ("n_tokens", "n_sink", "n_qk", "n_qv", "n_k_recent", "n_v_recent"):
        assert int(g[key]) == int(o[key]), (key, g[key], o[key])
    assert np.array_equal(g["norm"].view(np.uint32), o["norm"].view(np.uint32)), "norm"
    for key in ("k_sink", "v_sink", "k_recent", "v_recent"):
        assert np.array_equal(g[key].view(np.uint16), o[key].view(np.uint16)), key
    k_kind, v_kind = ("row", "block") if grouping == O.INNER else ("block", "row")
    flips = assert_store_equal(g, o, "k", k_kind, G, k_hybrid)
    flips += assert_store_equal(g, o, "v", v_kind, G, v_hybrid)
    return flips
