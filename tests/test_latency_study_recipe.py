"""The latency study's mask-ablation inputs: the oracle's hybrid rule flags the wanted fraction of value groups."""
import numpy as np
import pytest

from oracle import innerq_oracle as O
from paper_2602_23200_b200 import latency_study as LS
from paper_2602_23200_b200 import synth


@pytest.mark.parametrize("density", LS.MASK_DENSITIES)
def test_values_with_mask_density_hits_the_wanted_fraction(density):
    w = LS.layer_workload(32 + 32 * 16 + 96, **LS.MASK_PRESET).with_(n_kv_heads=2, n_q_heads=8)
    K, V = synth.kv_all(w)
    Vm = LS.values_with_mask_density(V, w.w_sink, w.group, density)
    assert Vm.dtype == np.float16 and Vm.shape == V.shape
    # tokens in the sink and behind the last whole group are untouched
    assert np.array_equal(Vm[:, :, :w.w_sink], V[:, :, :w.w_sink])
    oc = O.from_workload(w)
    oc.prefill(K, Vm)
    e = oc.export()
    frac = float(((e["v_scale"] & 0x8000) != 0).mean())
    n = e["v_scale"].size
    assert abs(frac - density) <= 4 * np.sqrt(density * (1 - density) / n) + 1e-3
    # the groups built for the symmetric candidate are reproduced exactly by it (L1 error zero); a shifted group
    # that happens to prefer it as well is the rare exception
    sym = (e["v_scale"] & 0x8000) == 0
    if sym.any():
        assert np.mean(e["v_err_sym"][sym] == 0.0) > 0.9
