"""The decode entry point that runs on the library's built-in scratch array (needs a B200).

Collected last on purpose: a run that stops at the first failure has then already run everything else.
It checks the variant against the regular entry point AND against the CPU oracle on two calls in a row (the
shared array keeps the first call's contents when the second starts), and that an over-sized configuration
is refused.
"""
import numpy as np
import pytest

from oracle import innerq_oracle as O
from paper_2602_23200_b200 import synth
from tests import _parity as P

pytestmark = pytest.mark.gpu


def _setup(w):
    import torch
    from paper_2602_23200_b200 import binding as B
    K, V = synth.kv_all(w)
    gc = B.InnerQCache(B.make_config(w, max_tokens=w.n_tokens + 8))
    gc.innerq_quantize_prefill(torch.from_numpy(K).cuda(), torch.from_numpy(V).cuda())
    return gc


@pytest.mark.parametrize("w", [synth.tiny(n_tokens=700), synth.config1().with_(n_tokens=1500)], ids=["gqa", "single_head"])
def test_static_scratch_decode_matches_regular_decode_twice(w):
    import torch
    gc = _setup(w)
    oc = O.from_workload(w)
    oc.prefill(*synth.kv_all(w))
    for call in range(2):
        qh = synth.query(w, call)
        q = torch.from_numpy(qh).cuda()
        ref = gc.innerq_decode_attention(q).cpu().numpy()
        got = gc.innerq_decode_attention_static(q).cpu().numpy()
        assert np.isfinite(got).all()
        P.assert_outputs_close(got, ref, f"static scratch against the regular entry point, call {call}")
        P.assert_outputs_close(got, oc.decode(qh), f"static scratch against the oracle, call {call}")
        assert gc.innerq_read_device_error() == 0      # covers the error word inside the shared array as well
    # a different cache on the same device shares the array: its call must not be disturbed by the leftovers
    w2 = synth.tiny(n_tokens=333, group=64, k_bits=4, v_bits=4)
    gc2 = _setup(w2)
    q2 = torch.from_numpy(synth.query(w2, 7)).cuda()
    P.assert_outputs_close(gc2.innerq_decode_attention_static(q2).cpu().numpy(),
                           gc2.innerq_decode_attention(q2).cpu().numpy(), "static scratch, second cache")
    torch.cuda.synchronize()


def test_static_scratch_refuses_configurations_beyond_its_size():
    import torch
    from paper_2602_23200_b200 import binding as B
    w = synth.tiny(batch=64, n_q_heads=64, n_kv_heads=8, n_tokens=40)      # 4096 query heads of partial slots
    cfg = B.make_config(w, max_tokens=48)
    _, ws_bytes = B.innerq_cache_bytes(cfg)
    assert ws_bytes > 4 << 20
    gc = _setup(w)
    q = torch.from_numpy(synth.query(w)).cuda()
    with pytest.raises(B.InnerQError) as ei:
        gc.innerq_decode_attention_static(q)
    assert ei.value.status == -4
    out = gc.innerq_decode_attention(q)          # the regular entry point still serves it
    assert torch.isfinite(out.float()).all()
