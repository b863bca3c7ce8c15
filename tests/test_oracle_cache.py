"""Pins for the oracle's cache bookkeeping and decode attention (CPU only).

Checks against things other than the oracle itself: torch's scaled_dot_product_attention
in float64, a pure-Python brute force on tiny shapes, exactness on representable grids,
window/eviction invariants from Sections "High-precision Window" and "Latency".
"""
import math

import numpy as np
import pytest
import torch

from oracle import innerq_oracle as O
from paper_2602_23200_b200 import synth

f32 = np.float32


def sdpa64(q, K, V, scale):
    """Library reference: q [Hq, D], K/V [Hq, N, D] float64."""
    qt = torch.from_numpy(np.asarray(q, dtype=np.float64))[None, :, None, :]
    Kt = torch.from_numpy(np.asarray(K, dtype=np.float64))[None]
    Vt = torch.from_numpy(np.asarray(V, dtype=np.float64))[None]
    o = torch.nn.functional.scaled_dot_product_attention(qt, Kt, Vt, scale=scale)
    return o[0, :, 0, :].numpy()


def test_dense_attention_matches_library():
    g = np.random.default_rng(0)
    q, K, V = g.standard_normal(24), g.standard_normal((57, 24)), g.standard_normal((57, 24))
    ref = sdpa64(q[None], K[None], V[None], 1 / math.sqrt(24))[0]
    assert np.allclose(O.dense_attention(q, K, V), ref, rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("grouping", [O.INNER, O.OUTER, O.FP16])
@pytest.mark.parametrize("N", [1, 3, 4, 5, 20])
def test_all_tokens_in_windows_equals_unquantised_attention(grouping, N):
    # N <= w_sink + w_recent: nothing is quantised, the result is plain attention on the fp16 inputs.
    w = synth.tiny(n_tokens=N, grouping=grouping, k_normalize=int(grouping == O.INNER))
    K, V = synth.kv_all(w)
    q = synth.query(w)
    c = O.from_workload(w)
    c.prefill(K, V)
    out = c.decode(q)
    r = w.q_per_kv
    for b in range(w.batch):
        Kr = np.repeat(K[b].astype(np.float64), r, axis=0)
        Vr = np.repeat(V[b].astype(np.float64), r, axis=0)
        ref = sdpa64(q[b].astype(np.float64), Kr, Vr, 1 / math.sqrt(w.head_dim))
        assert np.allclose(out[b], ref, rtol=1e-12, atol=1e-13)
    if grouping != O.FP16:
        e = c.export()
        assert e["n_qk"] == 0 and e["n_qv"] == 0
        assert e["n_sink"] == min(N, w.w_sink) and e["n_k_recent"] == max(0, N - w.w_sink)


@pytest.mark.parametrize("grouping", [O.INNER, O.OUTER])
@pytest.mark.parametrize("bits,G", [(2, 32), (3, 64), (4, 32)])
def test_decode_equals_python_bruteforce(grouping, bits, G):
    # Tiny case: rebuild K~ and V~ element by element with Python loops straight from the
    # exported canonical arrays and the decoding rule, then run textbook attention in Python floats.
    w = synth.tiny(batch=1, n_q_heads=2, n_kv_heads=1, n_tokens=4 + 2 * G + 9 + 6, head_dim=64 if G <= 64 else 128,
                   group=G, k_bits=bits, v_bits=bits, w_sink=4, w_recent=6, grouping=grouping,
                   k_normalize=int(grouping == O.INNER))
    K, V = synth.kv_all(w)
    q = synth.query(w)
    c = O.from_workload(w)
    c.prefill(K, V)
    e = c.export()
    D, N = w.head_dim, w.n_tokens
    half = 2 ** (bits - 1)

    def h(bits16):
        return float(np.array(bits16, dtype=np.uint16).view(np.float16))

    def deq(code, sb, zb):
        s = h(sb & 0x7FFF)
        return s * int(code) + (h(zb) if sb & 0x8000 else -s * half)

    Kt = [[0.0] * D for _ in range(N)]
    Vt = [[0.0] * D for _ in range(N)]
    ws = e["n_sink"]
    for t in range(N):
        for ch in range(D):
            # keys
            if t < ws:
                Kt[t][ch] = float(e["k_sink"][0, t, ch])
            elif t < ws + e["n_qk"]:
                i = t - ws
                sb, zb = ((e["k_scale"][0, i, ch // G], e["k_zero"][0, i, ch // G]) if grouping == O.INNER
                          else (e["k_scale"][0, i // G, ch], e["k_zero"][0, i // G, ch]))
                nrm = float(e["norm"][0, ch]) if grouping == O.INNER else 1.0
                Kt[t][ch] = deq(e["k_code"][0, i, ch], int(sb), int(zb)) * nrm
            else:
                Kt[t][ch] = float(e["k_recent"][0, t - ws - e["n_qk"], ch])
            # values
            if t < ws:
                Vt[t][ch] = float(e["v_sink"][0, t, ch])
            elif t < ws + e["n_qv"]:
                i = t - ws
                sb, zb = ((e["v_scale"][0, i // G, ch], e["v_zero"][0, i // G, ch]) if grouping == O.INNER
                          else (e["v_scale"][0, i, ch // G], e["v_zero"][0, i, ch // G]))
                Vt[t][ch] = deq(e["v_code"][0, i, ch], int(sb), int(zb))
            else:
                Vt[t][ch] = float(e["v_recent"][0, t - ws - e["n_qv"], ch])
    assert e["n_qk"] != e["n_qv"]          # the case has a skew zone (quantised K, fp16 V or vice versa)
    out = c.decode(q)
    for j in range(2):
        qj = [float(x) for x in q[0, j]]
        s = [sum(a * b for a, b in zip(qj, Kt[t])) / math.sqrt(D) for t in range(N)]
        m = max(s)
        p = [math.exp(x - m) for x in s]
        z = math.fsum(p)
        ref = [math.fsum(p[t] * Vt[t][ch] for t in range(N)) / z for ch in range(D)]
        assert np.allclose(out[0, j], ref, rtol=1e-11, atol=1e-12)
    # the oracle's own materialised matrices agree with the element-wise rebuild
    Km, Vm = c.materialize(0)
    assert np.allclose(Km, np.array(Kt), rtol=1e-13, atol=0) and np.allclose(Vm, np.array(Vt), rtol=1e-13, atol=0)


def test_softmax_rows_sum_to_one_and_shift_invariance():
    w = synth.tiny()
    K, V = synth.kv_all(w)
    q = synth.query(w)
    c = O.from_workload(w)
    c.prefill(K, V)
    out, probs = c.decode(q, return_probs=True)
    assert len(probs) == w.batch * w.n_q_heads
    for p in probs.values():
        assert p.shape == (w.n_tokens,) and abs(p.sum() - 1.0) < 1e-12 and p.min() >= 0
    # the output is a convex combination of value rows
    for u in range(w.n_units):
        _, Vm = c.materialize(u)
        b, hh = divmod(u, w.n_kv_heads)
        for j in range(hh * w.q_per_kv, (hh + 1) * w.q_per_kv):
            assert np.all(out[b, j] <= Vm.max(0) + 1e-12) and np.all(out[b, j] >= Vm.min(0) - 1e-12)


def test_lossless_grid_inputs_equal_unquantised_attention():
    # Keys and values that lie exactly on a 2-bit asymmetric grid in every group (after a
    # power-of-two key normalisation) are reproduced exactly, so the quantised path must equal
    # plain attention on the fp16 inputs.
    g = np.random.default_rng(5)
    N, D, G = 4 + 96 + 8, 64, 32
    # every channel's max |K| is 4 -> norm 2 (exact); K/2 lies on 0.25*{-3..0}... grid -> asym exact
    uK = g.integers(0, 4, size=(N, D))
    uK[:, 0::G], uK[:, 1::G] = 0, 3
    K = (0.5 * uK - 1.0) * 2.0
    K[0, :] = 4.0
    uV = g.integers(0, 4, size=(N, D))
    V = 0.25 * uV + 0.5
    for j in range(3):                       # every 32-token value group contains code 0 and code 3
        V[4 + 32 * j, :], V[5 + 32 * j, :] = 0.5, 1.25
    K16, V16 = K.astype(np.float16)[None, None], V.astype(np.float16)[None, None]
    c = O.OracleCache(1, 1, 1, D, N + 8, G, 2, 2, O.ASYM, O.ASYM, w_sink=4, w_recent=8)
    c.prefill(K16, V16)
    assert np.all(c.norm == 2.0) and c.k.n_q == 96 and c.v.n_q == 96
    q = g.standard_normal((1, 1, D)).astype(np.float16)
    ref = O.dense_attention(q[0, 0], K16[0, 0], V16[0, 0])
    assert np.allclose(c.decode(q)[0, 0], ref, rtol=1e-12, atol=1e-13)


def test_norm_definition_and_fold_identity():
    w = synth.tiny(n_tokens=200)
    K, _ = synth.kv_all(w)
    n = O.channel_norm(K.reshape(w.n_units, -1, w.head_dim))
    K32 = K.reshape(w.n_units, -1, w.head_dim).astype(np.float64)
    # max_t |K / norm| = norm (the definition sqrt(max |K|) makes the normalised maximum equal the norm)
    assert np.allclose(np.abs(K32 / n[:, None, :]).max(1), n, rtol=1e-6)
    assert np.allclose(n.astype(np.float64) ** 2, np.abs(K32).max(1), rtol=1e-6)
    # folding: (q * norm) . (k / norm) = q . k
    q = np.random.default_rng(1).standard_normal(w.head_dim)
    for u in range(w.n_units):
        assert np.allclose((K32[u] / n[u]) @ (q * n[u]), K32[u] @ q, rtol=1e-12, atol=1e-12)
    z = np.zeros((1, 5, 8), dtype=np.float16)
    assert np.all(O.channel_norm(z) == 1.0)


@pytest.mark.parametrize("grouping", [O.INNER, O.OUTER])
def test_append_counters_windows_and_cadence(grouping):
    # Section "Latency": inner grouping quantises one key token every step and G value tokens every
    # G steps; outer grouping does the reverse.  Window tokens are bit-identical to the inputs.
    G, ws, wr = 32, 4, 16
    w = synth.tiny(n_tokens=2, group=G, w_sink=ws, w_recent=wr, grouping=grouping,
                   k_normalize=int(grouping == O.INNER))
    K, V = synth.kv_all(w)
    c = O.from_workload(w, max_tokens=400)
    c.prefill(K, V)
    allK, allV = [K.reshape(w.n_units, -1, w.head_dim)], [V.reshape(w.n_units, -1, w.head_dim)]
    prev = c.export()
    for step in range(150):
        k1, v1 = synth.new_token(w, step)
        c.append(k1, v1)
        allK.append(k1.reshape(w.n_units, 1, -1))
        allV.append(v1.reshape(w.n_units, 1, -1))
        e = c.export()
        N = e["n_tokens"]
        assert N == 3 + step
        one_per_step = ("n_qk", "n_k_recent") if grouping == O.INNER else ("n_qv", "n_v_recent")
        g_per_g = ("n_qv", "n_v_recent") if grouping == O.INNER else ("n_qk", "n_k_recent")
        assert e["n_sink"] == min(ws, N)
        assert e[one_per_step[0]] == max(0, N - ws - wr)
        assert e[one_per_step[1]] == min(wr, max(0, N - ws))
        assert e[g_per_g[0]] == (max(0, N - ws - wr) // G) * G
        assert e[g_per_g[0]] % G == 0 and e[g_per_g[0]] - prev[g_per_g[0]] in (0, G)
        if N >= ws + wr:
            assert wr <= e[g_per_g[1]] <= wr + G - 1
        assert 0 <= e[one_per_step[0]] - e[g_per_g[0]] <= G - 1
        assert e["n_sink"] + e["n_qk"] + e["n_k_recent"] == N == e["n_sink"] + e["n_qv"] + e["n_v_recent"]
        prev = e
    Kall, Vall = np.concatenate(allK, 1), np.concatenate(allV, 1)
    e = c.export()
    assert np.array_equal(e["k_sink"], Kall[:, :ws]) and np.array_equal(e["v_sink"], Vall[:, :ws])
    assert np.array_equal(e["k_recent"], Kall[:, ws + e["n_qk"]:])
    assert np.array_equal(e["v_recent"], Vall[:, ws + e["n_qv"]:])


@pytest.mark.parametrize("grouping", [O.INNER, O.OUTER])
@pytest.mark.parametrize("mode", [O.HYBRID, O.SYM])
def test_prefill_then_appends_equals_longer_prefill_under_fixed_norm(grouping, mode):
    w = synth.tiny(n_tokens=300, grouping=grouping, k_mode=mode, v_mode=mode, k_bits=3,
                   k_normalize=int(grouping == O.INNER))
    K, V = synth.kv_all(w)
    norm = O.channel_norm(K.reshape(w.n_units, -1, w.head_dim))
    a = O.from_workload(w)
    a.prefill(K, V, norm=norm)
    b = O.from_workload(w)
    b.prefill(K[:, :, :100], V[:, :, :100], norm=norm)
    for t in range(100, 300):
        b.append(K[:, :, t], V[:, :, t])
    ea, eb = a.export(), b.export()
    for key in ea:
        if key.endswith("err_asym") or key.endswith("err_sym"):
            continue
        assert np.array_equal(ea[key], eb[key]), key
    q = synth.query(w)
    assert np.array_equal(a.decode(q), b.decode(q))


def test_score_error_bound_on_quantised_keys():
    # |q'.(x - x^)| <= sum_g (S_g/2 + fp16 slack) * sum_{c in g} |q'_c|  for every quantised key row.
    w = synth.tiny(batch=1, n_q_heads=1, n_kv_heads=1, n_tokens=260)
    K, V = synth.kv_all(w)
    c = O.from_workload(w)
    c.prefill(K, V)
    e = c.export()
    G, D = w.group, w.head_dim
    q = synth.query(w)[0, 0].astype(np.float64)
    qn = np.abs(q * e["norm"][0])
    x = K[0, 0, w.w_sink:w.w_sink + e["n_qk"]].astype(np.float64) / e["norm"][0].astype(np.float64)
    xh = c.k.dequant(0)
    s = (e["k_scale"][0] & 0x7FFF).view(np.float16).astype(np.float64)           # [n, D/G]
    z = np.abs(e["k_zero"][0].view(np.float16).astype(np.float64))
    bound = ((s / 2 * (1 + 2 ** -7) + z * 2 ** -10 + 1e-6) * qn.reshape(D // G, G).sum(1)[None, :]).sum(1)
    assert np.all(np.abs((x - xh) @ (q * e["norm"][0])) <= bound)


def test_quantised_keys_use_the_normalised_domain():
    # The stored key codes must be those of K / norm (not of K): check via the quantiser itself on
    # an explicitly normalised copy, and that outlier channels no longer dominate group scales.
    w = synth.config1().with_(n_tokens=4 + 64 + 128)
    K, V = synth.kv_all(w)
    c = O.from_workload(w)
    c.prefill(K, V)
    e = c.export()
    n = O.channel_norm(K[0])
    x = (K[0, 0, 4:68].astype(f32) * (f32(1) / n[0])).reshape(64, 4, 32)
    r = O.quantize_groups(x, 2, O.HYBRID)
    assert np.array_equal(e["k_code"][0], r["code"].reshape(64, 128))
    assert np.array_equal(e["k_scale"][0], r["scale_bits"])
    raw = O.quantize_groups(K[0, 0, 4:68].astype(f32).reshape(64, 4, 32), 2, O.HYBRID)
    s_norm = (r["scale_bits"] & 0x7FFF).view(np.float16).astype(np.float64).mean()
    s_raw = (raw["scale_bits"] & 0x7FFF).view(np.float16).astype(np.float64).mean()
    assert s_norm < 0.5 * s_raw


@pytest.mark.parametrize("grouping", [O.INNER, O.OUTER, O.FP16])
@pytest.mark.parametrize("n_q", [1, 2, 5])
def test_multi_query_decode_is_causal_attention(grouping, n_q):
    # n_q query tokens whose own keys / values are the newest n_q cache tokens: query i sees tokens 0 .. N-n_q+i.
    # Pinned to the library's attention with an explicit boolean mask (a) on the raw fp16 tensors when every
    # token is in a window and (b) on the materialised K~, V~ (themselves pinned element by element above)
    # when most tokens are quantised.
    for N, windows_only in ((9, True), (150, False)):
        w = synth.tiny(n_tokens=N, grouping=grouping, k_normalize=int(grouping == O.INNER), w_sink=4,
                       w_recent=8 if windows_only else 12)
        K, V = synth.kv_all(w)
        q = np.stack([synth.query(w, step) for step in range(n_q)], axis=1)          # [B, n_q, Hq, D]
        c = O.from_workload(w)
        c.prefill(K, V)
        out = c.decode_multi(q)
        assert out.shape == (w.batch, n_q, w.n_q_heads, w.head_dim)
        r = w.q_per_kv
        mask = torch.ones(n_q, N, dtype=torch.bool)
        for i in range(n_q):
            mask[i, N - n_q + i + 1:] = False
        for b in range(w.batch):
            for h in range(w.n_kv_heads):
                if windows_only:
                    Km, Vm = K[b, h].astype(np.float64), V[b, h].astype(np.float64)
                else:
                    Km, Vm = c.materialize(b * w.n_kv_heads + h)
                for j in range(h * r, (h + 1) * r):
                    qt = torch.from_numpy(q[b, :, j].astype(np.float64))[None, None]        # [1, 1, n_q, D]
                    ref = torch.nn.functional.scaled_dot_product_attention(
                        qt, torch.from_numpy(Km)[None, None], torch.from_numpy(Vm)[None, None], attn_mask=mask,
                        scale=1 / math.sqrt(w.head_dim))[0, 0].numpy()
                    assert np.allclose(out[b, :, j], ref, rtol=1e-11, atol=1e-12)
        # the newest query sees everything: the same as the single-token decode
        assert np.array_equal(out[:, n_q - 1], c.decode(q[:, n_q - 1]))


def test_key_norm_scopes_per_unit_and_across_heads():
    # Section "Per-channel Normalization of K": norm_k = sqrt(max |K[:, :, k]|).  Read per (batch, KV head) unit by
    # default; the literal scope takes the maximum over all heads as well (oracle-only switch).  Either way the norm
    # cancels between q' = q * norm and k / norm, so with every token inside the windows both give plain attention,
    # and with quantised rows the two differ only through the quantisation grid.
    rng = np.random.default_rng(11)
    K = rng.standard_normal((2, 3, 40, 128)).astype(np.float16)
    K[1, 2, 7, 5] = 50.0                                        # one large key entry in one head
    per_unit = O.channel_norm(K)
    literal = O.channel_norm(K, all_heads=True)
    assert per_unit.shape == literal.shape == (2, 3, 128)
    assert per_unit[1, 2, 5] == np.float32(np.sqrt(np.float32(50.0))) and per_unit[0, 0, 5] < 3
    assert np.all(literal == literal[0, 0]) and literal[0, 0, 5] == np.float32(np.sqrt(np.float32(50.0)))
    assert np.all(literal >= per_unit)
    V = rng.standard_normal((2, 3, 40, 128)).astype(np.float16)
    q = rng.standard_normal((2, 3, 128)).astype(np.float16)
    outs = []
    for flag in (False, True):
        oc = O.OracleCache(2, 3, 3, 128, 64, 32, 2, 2, w_sink=4, w_recent=8, norm_all_heads=flag)
        oc.prefill(K, V)
        assert np.array_equal(oc.norm.reshape(2, 3, 128), literal if flag else per_unit)
        outs.append(oc.decode(q))
    assert np.allclose(outs[0], outs[1], atol=0.5) and not np.array_equal(outs[0], outs[1])
