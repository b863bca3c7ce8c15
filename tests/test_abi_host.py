"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, validates arguments, and its packed layout has the paper's effective bit-widths."""
import ctypes as C
import os
import re

import pytest

from paper_2602_23200_b200 import binding as B
from paper_2602_23200_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "innerq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(innerq_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert len(names) >= 10
    assert sorted(B.EXPORTED_SYMBOLS) == names
    lib = C.CDLL(B.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings():
    for code in range(-5, 1):
        assert B.status_string(code) not in ("", "unknown status")
    assert B.status_string(-99) == "unknown status"


def test_config_validation_without_gpu():
    ok = B.make_config(synth.config1())
    cb, wb = B.innerq_cache_bytes(ok)
    assert cb > 0 and wb > 0 and cb % 256 == 0
    for field, bad, status in [("head_dim", 64, -2), ("group", 48, -2), ("k_bits", 5, -2), ("batch", 0, -1),
                               ("n_q_heads", 3, -1), ("max_tokens", 0, -1), ("k_mode", 7, -1), ("grouping", 3, -1)]:
        cfg = B.make_config(synth.config1().with_(n_q_heads=2, n_kv_heads=2), **{field: bad})
        with pytest.raises(B.InnerQError) as ei:
            B.innerq_cache_bytes(cfg)
        assert ei.value.status == status, field
    with pytest.raises(B.InnerQError):      # the outer-grouped method has no key normalisation
        B.innerq_cache_bytes(B.make_config(synth.config1(), grouping=B.GROUPING_OUTER, k_normalize=1))


def test_step_staging_size_without_gpu():
    # device staging of innerq_decode_step_host: k_new, v_new, q and out, each rounded up to 256 bytes
    need = C.c_size_t()
    cfg = B.make_config(batch=3, n_q_heads=8, n_kv_heads=2, max_tokens=64)
    assert B.lib().innerq_step_staging_bytes(C.byref(cfg), C.byref(need)) == 0
    kv, q = 3 * 2 * 128 * 2, 3 * 8 * 128 * 2
    assert need.value == 2 * ((kv + 255) // 256 * 256) + 2 * ((q + 255) // 256 * 256)
    bad = B.make_config(batch=3, n_q_heads=8, n_kv_heads=3, max_tokens=64)
    assert B.lib().innerq_step_staging_bytes(C.byref(bad), C.byref(need)) == -1
    assert B.lib().innerq_step_staging_bytes(C.byref(cfg), None) == -1


def test_multi_query_scratch_size_without_gpu():
    # partials of four query rows per (batch, KV head) unit: the per-row size is the single-query workspace's
    need, ws, cb = C.c_size_t(), C.c_size_t(), C.c_size_t()
    cfg1 = B.make_config(batch=1, n_q_heads=1, n_kv_heads=1, max_tokens=64)
    cfg8 = B.make_config(batch=2, n_q_heads=8, n_kv_heads=4, max_tokens=64)
    sizes = []
    for cfg in (cfg1, cfg8):
        assert B.lib().innerq_multi_query_scratch_bytes(C.byref(cfg), C.byref(need)) == 0
        assert need.value > 0 and need.value % 256 == 0
        sizes.append(need.value)
    assert B.lib().innerq_multi_query_scratch_bytes(C.byref(cfg1), None) == -1
    bad = B.make_config(batch=1, n_q_heads=3, n_kv_heads=2, max_tokens=64)
    assert B.lib().innerq_multi_query_scratch_bytes(C.byref(bad), C.byref(need)) == -1


def test_packed_payload_matches_table_bits():
    # Table "bits" (G = 32, head dim 128): effective bits per cached number = payload bytes * 8 / 128.
    rows = [l.split() for l in open(os.path.join(ROOT, "tests", "golden", "table_bits.txt"))
            if l.strip() and not l.startswith("#")]
    for name, kb, kz, vb, vz, eff in rows:
        if name == "KIVI":
            cfg = B.make_config(synth.config1(), k_bits=int(kb), v_bits=int(vb), grouping=B.GROUPING_OUTER,
                                k_normalize=0, k_mode=B.MODE_ASYM, v_mode=B.MODE_ASYM)
        else:
            cfg = B.make_config(synth.config1(), k_bits=int(kb), v_bits=int(vb),
                                k_mode=B.MODE_HYBRID if int(kz) else B.MODE_SYM,
                                v_mode=B.MODE_HYBRID if int(vz) else B.MODE_SYM)
        k_bytes, v_bytes = B.innerq_token_payload_bytes(cfg)
        assert (k_bytes + v_bytes) * 8 / (2 * 128) == pytest.approx(float(eff)), name


def test_cache_size_tracks_payload():
    # the buffer the caller must provide is the payload plus windows, norms and alignment: within 2 %
    # for a long context
    w = synth.config4()
    cfg = B.make_config(w)
    cb, _ = B.innerq_cache_bytes(cfg)
    k_bytes, v_bytes = B.innerq_token_payload_bytes(cfg)
    payload = w.n_units * w.n_tokens * (k_bytes + v_bytes)
    assert payload <= cb <= 1.02 * payload
    assert cb < 0.16 * (2 * w.n_units * w.n_tokens * 128 * 2)      # 2.25 bits vs 16 bits per number


def test_paged_sizes_without_gpu():
    # a page holds page_tokens tokens of every unit, at exactly the payload the effective-bits table counts;
    # the cache buffer of a paged cache keeps only what does not grow with the context
    for w in (synth.config2(), synth.config3(4), synth.config4()):
        for kw in ({}, dict(grouping=B.GROUPING_OUTER, k_normalize=0, k_mode=B.MODE_ASYM, v_mode=B.MODE_ASYM)):
            cfg = B.make_config(w, **kw)
            k_bytes, v_bytes = B.innerq_token_payload_bytes(cfg)
            full, _ = B.innerq_cache_bytes(cfg)
            for page in (128, 1024, 4096):
                cb, wb, pb, mp = B.innerq_paged_cache_bytes(cfg, page)
                assert pb == page * w.n_units * (k_bytes + v_bytes), (w.name, page)
                packed_tokens = w.n_tokens - w.w_sink - w.w_recent
                assert mp * page >= packed_tokens and (mp - 1) * page < packed_tokens + 32 + 128
                assert cb < 0.02 * full + 2 * w.n_units * (w.w_sink + w.w_recent + w.group + 1) * 128 * 2 + 4 * mp + 4096
                assert wb == B.innerq_cache_bytes(cfg)[1]
    cfg = B.make_config(synth.config2())
    for bad in (0, 100, 64, 384, -1024):
        with pytest.raises(B.InnerQError) as ei:
            B.innerq_paged_cache_bytes(cfg, bad)
        assert ei.value.status == -1
    with pytest.raises(B.InnerQError) as ei:
        B.innerq_paged_cache_bytes(B.make_config(synth.config2(), grouping=B.GROUPING_FP16), 1024)
    assert ei.value.status == -2
