"""CUDA path vs CPU oracle, element by element, through the C ABI (needs a B200)."""
import numpy as np
import pytest

from oracle import innerq_oracle as O
from paper_2602_23200_b200 import synth
from tests import _parity as P

pytestmark = pytest.mark.gpu


def _torch():
    import torch
    return torch


def gpu_cache(w, max_tokens=None, **opts):
    from paper_2602_23200_b200 import binding as B
    cfg = B.make_config(w, max_tokens=max_tokens or w.n_tokens + 300)
    return B.InnerQCache(cfg)


def dev(x):
    torch = _torch()
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def run_prefill_both(w, max_tokens=None):
    K, V = synth.kv_all(w)
    oc = O.from_workload(w, max_tokens=max_tokens or w.n_tokens + 300)
    oc.prefill(K, V)
    gc = gpu_cache(w, max_tokens)
    gc.innerq_quantize_prefill(dev(K), dev(V))
    return oc, gc, K, V


def check_decode(w, oc, gc, step=0, variants=(0,), splits=(0,)):
    q = synth.query(w, step)
    ref = oc.decode(q)
    worst = 0.0
    for variant in variants:
        for s in splits:
            gc.innerq_set_decode_options(s, variant)
            out = gc.innerq_decode_attention(dev(q)).cpu().numpy()
            worst = max(worst, P.assert_outputs_close(out, ref, f"{w.name} variant={variant} splits={s}"))
    gc.innerq_set_decode_options(0, 0)
    assert gc.innerq_read_device_error() == 0      # no bounded wait inside a kernel ever ran out
    return worst


CASES = [
    # bits, G, mode, sym_variant, N
    (2, 32, O.HYBRID, 0, 333),
    (2, 32, O.HYBRID, 1, 333),
    (2, 64, O.ASYM, 0, 420),
    (2, 128, O.HYBRID, 0, 700),
    (3, 32, O.HYBRID, 0, 333),
    (3, 64, O.SYM, 0, 300),
    (4, 64, O.HYBRID, 0, 420),
    (4, 32, O.SYM, 1, 333),
    (4, 128, O.ASYM, 0, 541),
]


@pytest.mark.parametrize("bits,G,mode,variant,N", CASES)
def test_prefill_and_decode_inner(bits, G, mode, variant, N):
    w = synth.tiny(n_tokens=N, group=G, k_bits=bits, v_bits=bits, k_mode=mode, v_mode=mode, sym_variant=variant)
    oc, gc, _, _ = run_prefill_both(w)
    P.assert_export_equal(gc.innerq_cache_export(), oc.export(), O.INNER, G, mode == O.HYBRID, mode == O.HYBRID)
    check_decode(w, oc, gc, variants=(0, 1, 3, 4), splits=(0, 1, 3, 7))


@pytest.mark.parametrize("bits,G,N", [(2, 32, 333), (3, 64, 420), (4, 128, 541)])
def test_prefill_and_decode_outer(bits, G, N):
    w = synth.tiny(n_tokens=N, group=G, k_bits=bits, v_bits=bits, grouping=O.OUTER, k_normalize=0,
                   k_mode=O.ASYM, v_mode=O.ASYM)
    oc, gc, _, _ = run_prefill_both(w)
    P.assert_export_equal(gc.innerq_cache_export(), oc.export(), O.OUTER, G, False, False)
    check_decode(w, oc, gc, splits=(0, 2))


@pytest.mark.parametrize("bits,G,r,N", [(2, 32, 1, 700), (2, 64, 4, 600), (2, 128, 2, 900), (4, 32, 4, 500),
                                        (4, 64, 8, 555), (4, 128, 1, 1300)])
def test_outer_grouped_fused_kernel(bits, G, r, N):
    # the outer-grouped comparison cache on the fused kernel (variant 3 refuses to fall back), against the generic
    # kernel (variant 1) and the oracle; then appends through the reversed skew zone (packed values, fp16 keys)
    w = synth.tiny(n_tokens=N, group=G, k_bits=bits, v_bits=bits, grouping=O.OUTER, k_normalize=0, k_mode=O.ASYM,
                   v_mode=O.ASYM, n_q_heads=2 * r)
    oc, gc, _, _ = run_prefill_both(w)
    P.assert_export_equal(gc.innerq_cache_export(), oc.export(), O.OUTER, G, False, False)
    check_decode(w, oc, gc, variants=(3, 1), splits=(0, 2, 5))
    for step in range(G + 5):
        k1, v1 = synth.new_token(w, step)
        oc.append(k1, v1)
        gc.innerq_append_token(dev(k1), dev(v1))
        if step in (0, 1, 15, 16, 17, G - 1, G, G + 4):
            check_decode(w, oc, gc, step=step, variants=(3,), splits=(0, 3))
    P.assert_export_equal(gc.innerq_cache_export(), oc.export(), O.OUTER, G, False, False)


@pytest.mark.parametrize("N,mode", [(700, O.HYBRID), (1333, O.ASYM), (164, O.HYBRID), (37, O.HYBRID)])
def test_one_query_head_per_kv_head_kernel_instance(N, mode):
    # 2-bit, G = 32, one query head per KV head: the instance of the fused kernel whose tensor-core columns are
    # (channel group, digit), against the oracle and the generic kernel, for several split counts, one and two chunks
    # per loop iteration, and through appends that cross a value-group eviction
    w = synth.tiny(n_tokens=N, group=32, n_q_heads=2, k_mode=mode, v_mode=mode)
    oc, gc, _, _ = run_prefill_both(w)
    check_decode(w, oc, gc, variants=(2, 3, 4, 1), splits=(0, 1, 3))
    for step in range(40):
        k1, v1 = synth.new_token(w, step)
        oc.append(k1, v1)
        gc.innerq_append_token(dev(k1), dev(v1))
        if step in (0, 7, 31, 32, 39):
            check_decode(w, oc, gc, step=step, variants=(3, 4), splits=(0, 2))



def test_fp16_cache_decode():
    w = synth.tiny(n_tokens=500, grouping=O.FP16, k_normalize=0)
    oc, gc, K, V = run_prefill_both(w)
    e = gc.innerq_cache_export()
    assert e["n_tokens"] == 500 and np.array_equal(e["k_sink"].reshape(K.shape), K)
    check_decode(w, oc, gc, splits=(0, 1, 5))
    for step in range(3):
        k1, v1 = synth.new_token(w, step)
        oc.append(k1, v1)
        gc.innerq_append_token(dev(k1), dev(v1))
    check_decode(w, oc, gc, step=1)


def test_mixed_bits_and_modes():
    w = synth.tiny(n_tokens=400, group=32, k_bits=3, v_bits=2, k_mode=O.SYM, v_mode=O.HYBRID)
    oc, gc, _, _ = run_prefill_both(w)
    P.assert_export_equal(gc.innerq_cache_export(), oc.export(), O.INNER, 32, False, True)
    check_decode(w, oc, gc, variants=(0, 1, 3))


# key bits, value bits, key mode, value mode, G, query heads per KV head, N: packed formats of the fused kernel
# beyond equal-width hybrid ones (3-bit planes, symmetric-only 2-byte metadata, keys and values of different widths
# or metadata forms), with one query head per KV head (group-per-column kernel), several, and two passes of four
FORMATS = [
    (3, 3, O.HYBRID, O.HYBRID, 32, 1, 700),
    (3, 3, O.SYM, O.SYM, 32, 1, 700),
    (3, 2, O.SYM, O.SYM, 32, 1, 600),
    (3, 2, O.SYM, O.HYBRID, 32, 1, 1500),
    (3, 2, O.SYM, O.HYBRID, 64, 4, 600),
    (3, 2, O.SYM, O.SYM, 128, 2, 900),
    (2, 2, O.SYM, O.SYM, 128, 2, 900),
    (4, 4, O.SYM, O.SYM, 32, 1, 500),
    (3, 3, O.ASYM, O.ASYM, 128, 8, 900),
    (3, 3, O.SYM, O.SYM, 64, 8, 555),
    # keys and values of different widths, and 2-bit caches whose two tensors differ in metadata form
    (2, 4, O.HYBRID, O.HYBRID, 32, 1, 700),
    (4, 2, O.HYBRID, O.ASYM, 64, 4, 600),
    (2, 3, O.SYM, O.HYBRID, 32, 2, 500),
    (4, 3, O.HYBRID, O.SYM, 128, 4, 900),
    (3, 4, O.SYM, O.SYM, 64, 1, 450),
    (2, 2, O.SYM, O.HYBRID, 32, 1, 1200),
    (2, 2, O.HYBRID, O.SYM, 64, 4, 640),
]


@pytest.mark.parametrize("kb,vb,km,vm,G,r,N", FORMATS)
def test_fused_kernel_formats(kb, vb, km, vm, G, r, N):
    w = synth.tiny(n_tokens=N, group=G, k_bits=kb, v_bits=vb, k_mode=km, v_mode=vm, n_q_heads=2 * r)
    oc, gc, _, _ = run_prefill_both(w)
    P.assert_export_equal(gc.innerq_cache_export(), oc.export(), O.INNER, G, km == O.HYBRID, vm == O.HYBRID)
    check_decode(w, oc, gc, variants=(3, 1), splits=(0, 2, 5))       # 3: the fused kernel or an error, 1: generic kernel
    for step in range(G + 3):                                          # across a value-group eviction
        k1, v1 = synth.new_token(w, step)
        oc.append(k1, v1)
        gc.innerq_append_token(dev(k1), dev(v1))
    check_decode(w, oc, gc, step=7, variants=(3,), splits=(0, 3))
    # what the appends packed (one row per step, one value group on the way), bit for bit
    P.assert_export_equal(gc.innerq_cache_export(), oc.export(), O.INNER, G, km == O.HYBRID, vm == O.HYBRID)


def test_a_bounded_wait_that_runs_out_is_reported_and_leaves_the_context_usable():
    # The decode kernels wait for their asynchronous copies a bounded number of times and, if a wait runs out, set
    # the cache's device error word and return.  The self-test kernel takes that road on purpose: the kernels' own
    # wait routine, on a barrier nothing ever arrives on.  No fault, no hang: the kernel gives up after 256 polls.
    w = synth.tiny(n_tokens=300)
    oc, gc, _, _ = run_prefill_both(w)
    check_decode(w, oc, gc)                                   # error word still 0 (asserted there)
    gc.innerq_selftest_wait_expiry()
    assert gc.innerq_read_device_error() == 1                 # the expiry is reported ...
    assert gc.innerq_read_device_error() == 1                 # ... for good: the word is sticky
    q = synth.query(w, 3)
    out = gc.innerq_decode_attention(dev(q)).cpu().numpy()    # ... and the context and the cache still work
    P.assert_outputs_close(out, oc.decode(q), "after a wait that ran out")
    # another cache has its own error word
    _, g2, _, _ = run_prefill_both(w)
    assert g2.innerq_read_device_error() == 0


@pytest.mark.parametrize("N", [1, 3, 4, 5, 19, 20, 21, 52, 53])
def test_short_contexts_and_window_edges(N):
    # N <= w_sink, N <= w_sink + w_recent (nothing quantised), first quantised key token, first value group
    w = synth.tiny(n_tokens=N)
    oc, gc, K, V = run_prefill_both(w)
    e, eo = gc.innerq_cache_export(), oc.export()
    P.assert_export_equal(e, eo, O.INNER, w.group)
    check_decode(w, oc, gc, variants=(0, 1))
    if N <= w.w_sink + w.w_recent:
        # every token is in a window: the result is plain attention on the fp16 inputs
        q = synth.query(w)
        out = gc.innerq_decode_attention(dev(q)).cpu().numpy()
        for b in range(w.batch):
            for j in range(w.n_q_heads):
                h = j // w.q_per_kv
                ref = O.dense_attention(q[b, j], K[b, h], V[b, h])
                P.assert_outputs_close(out[b, j][None], ref[None], "all-window")


def test_empty_prefill_then_appends_through_every_phase():
    # start from an empty cache; append through sink fill, recent fill, first key eviction, value evictions
    w = synth.tiny(n_tokens=0, w_sink=4, w_recent=16, group=32)
    oc = O.from_workload(w, max_tokens=200)
    gc = gpu_cache(w, max_tokens=200)
    torch = _torch()
    gc.innerq_quantize_prefill(torch.empty((w.batch, w.n_kv_heads, 0, 128), dtype=torch.float16, device="cuda"),
                               torch.empty((w.batch, w.n_kv_heads, 0, 128), dtype=torch.float16, device="cuda"))
    for step in range(120):
        k1, v1 = synth.new_token(w, step)
        oc.append(k1, v1)
        gc.innerq_append_token(dev(k1), dev(v1))
        if step in (0, 3, 4, 19, 20, 21, 51, 52, 83, 84, 119):
            P.assert_export_equal(gc.innerq_cache_export(), oc.export(), O.INNER, w.group)
            check_decode(w, oc, gc, step=step, variants=(0, 1))


@pytest.mark.parametrize("grouping", [O.INNER, O.OUTER])
def test_prefill_then_appends_matches_oracle(grouping):
    w = synth.tiny(n_tokens=150, grouping=grouping, k_normalize=int(grouping == O.INNER), append_scale=0.5,
                   k_mode=O.HYBRID if grouping == O.INNER else O.ASYM,
                   v_mode=O.HYBRID if grouping == O.INNER else O.ASYM)
    oc, gc, _, _ = run_prefill_both(w)
    for step in range(100):
        k1, v1 = synth.new_token(w, step)
        oc.append(k1, v1)
        gc.innerq_append_token(dev(k1), dev(v1))
        if step % 33 == 32:
            check_decode(w, oc, gc, step=step)
    P.assert_export_equal(gc.innerq_cache_export(), oc.export(), grouping, w.group,
                          grouping == O.INNER, grouping == O.INNER)
    check_decode(w, oc, gc, step=1000, variants=(0, 1) if grouping == O.INNER else (0,))


def test_step_from_host_buffers_matches_separate_calls_and_oracle():
    # innerq_decode_step_host = copies in + append + decode + copy out; across a value-group eviction
    torch = _torch()
    w = synth.tiny(n_tokens=300, k_bits=3, v_bits=2, k_mode=O.SYM, v_mode=O.HYBRID)
    oc, gc, K, V = run_prefill_both(w)
    gc2 = gpu_cache(w)
    gc2.innerq_quantize_prefill(dev(K), dev(V))
    out_h = torch.empty((w.batch, w.n_q_heads, 128), dtype=torch.float16).pin_memory()
    for step in range(40):
        k1, v1 = synth.new_token(w, step)
        q = synth.query(w, step)
        oc.append(k1, v1)
        pin = (lambda t: t.pin_memory()) if step % 2 == 0 else (lambda t: t)    # in-place over the bus / staged copies
        gc.innerq_decode_step_host(pin(torch.from_numpy(k1)), pin(torch.from_numpy(v1)), pin(torch.from_numpy(q)), out_h)
        torch.cuda.synchronize()
        gc2.innerq_append_token(dev(k1), dev(v1))
        ref2 = gc2.innerq_decode_attention(dev(q)).cpu()
        assert torch.equal(out_h, ref2)                       # same kernels, same inputs: identical bits
        if step % 13 == 0 or step == 39:
            P.assert_outputs_close(out_h.numpy(), oc.decode(q), f"host step {step}")
    P.assert_export_equal(gc.innerq_cache_export(), oc.export(), O.INNER, w.group, False, True)
    assert gc.n_tokens == 340


@pytest.mark.parametrize("r,G,bits", [(3, 64, 2), (6, 32, 4), (5, 128, 3), (16, 64, 2)])
def test_query_heads_per_kv_head_not_a_multiple_of_four(r, G, bits):
    # the fused kernel takes up to four query heads of a KV head per pass: partial and multiple passes
    w = synth.tiny(n_tokens=450, group=G, k_bits=bits, v_bits=bits, n_q_heads=2 * r)
    oc, gc, _, _ = run_prefill_both(w)
    check_decode(w, oc, gc, variants=(3, 4, 1), splits=(0, 2))


@pytest.mark.parametrize("w_sink,w_recent", [(0, 0), (0, 7), (5, 0)])
def test_degenerate_windows(w_sink, w_recent):
    # no sink and / or no recent window: every token (w_recent = 0: even the newest) is quantised
    w = synth.tiny(n_tokens=230, w_sink=w_sink, w_recent=w_recent)
    oc, gc, _, _ = run_prefill_both(w)
    P.assert_export_equal(gc.innerq_cache_export(), oc.export(), O.INNER, w.group)
    check_decode(w, oc, gc, variants=(0, 1))
    for step in range(40):
        k1, v1 = synth.new_token(w, step)
        oc.append(k1, v1)
        gc.innerq_append_token(dev(k1), dev(v1))
        if step in (0, 1, 25, 26, 39):
            check_decode(w, oc, gc, step=step, variants=(0, 1))
    P.assert_export_equal(gc.innerq_cache_export(), oc.export(), O.INNER, w.group)


@pytest.mark.parametrize("grouping,r,G,bits,n_q", [(O.INNER, 1, 32, 2, 4), (O.INNER, 1, 32, 2, 7), (O.INNER, 4, 64, 2, 3),
                                                    (O.INNER, 2, 128, 4, 5), (O.INNER, 1, 64, 3, 9), (O.OUTER, 1, 32, 2, 6),
                                                    (O.OUTER, 4, 64, 4, 2)])
def test_multi_query_decode(grouping, r, G, bits, n_q):
    # n_q query tokens per sequence against one cache state, causal among the newest n_q tokens; rows of a KV
    # head share passes over the packed cache four at a time
    inner = grouping == O.INNER
    w = synth.tiny(batch=2, n_q_heads=2 * r, n_kv_heads=2, n_tokens=4 + 20 * 32 + 77, group=G, k_bits=bits, v_bits=bits,
                   w_sink=4, w_recent=24, grouping=grouping, k_normalize=int(inner),
                   **({} if inner else dict(k_mode=O.ASYM, v_mode=O.ASYM)))
    oc, gc, _, _ = run_prefill_both(w)
    for step in range(3):                 # a few appended tokens, so the ring buffers are rotated
        k1, v1 = synth.new_token(w, step)
        oc.append(k1, v1)
        gc.innerq_append_token(dev(k1), dev(v1))
    q = np.stack([synth.query(w, 10 + i) for i in range(n_q)], axis=1)           # [B, n_q, Hq, D]
    ref = oc.decode_multi(q)
    for splits in (0, 1, 3):
        gc.innerq_set_decode_options(splits, 0)
        out = gc.innerq_decode_attention_multi(dev(q)).cpu().numpy()
        P.assert_outputs_close(out, ref, f"multi-query n_q={n_q} splits={splits}")
    gc.innerq_set_decode_options(0, 0)
    # the newest query row is the plain decode of the same cache
    one = gc.innerq_decode_attention(dev(q[:, n_q - 1])).cpu().numpy()
    P.assert_outputs_close(one, ref[:, n_q - 1], "newest query = single-token decode")
    assert gc.innerq_read_device_error() == 0


def test_multi_query_short_contexts_and_limits():
    from paper_2602_23200_b200 import binding as B
    # everything in the windows: even sink tokens are masked by position
    w = synth.tiny(n_tokens=11, w_sink=4, w_recent=16)
    oc, gc, _, _ = run_prefill_both(w)
    for n_q in (1, 2, 6, 11):
        q = np.stack([synth.query(w, i) for i in range(n_q)], axis=1)
        out = gc.innerq_decode_attention_multi(dev(q)).cpu().numpy()
        P.assert_outputs_close(out, oc.decode_multi(q), f"windows only, n_q={n_q}")
    q12 = np.stack([synth.query(w, i) for i in range(12)], axis=1)
    with pytest.raises(B.InnerQError) as ei:              # more query tokens than cached tokens
        gc.innerq_decode_attention_multi(dev(q12))
    assert ei.value.status == -1
    # hidden tokens would reach into the chunks where keys and values are both packed: refused, nothing launched
    w = synth.tiny(n_tokens=4 + 64 + 8, w_sink=4, w_recent=8)
    oc, gc, _, _ = run_prefill_both(w)
    e = oc.export()
    room = w.n_tokens - e["n_sink"] - min(e["n_qk"], e["n_qv"])       # tokens that can be hidden
    q_ok = np.stack([synth.query(w, i) for i in range(room + 1)], axis=1)
    P.assert_outputs_close(gc.innerq_decode_attention_multi(dev(q_ok)).cpu().numpy(), oc.decode_multi(q_ok), "at the limit")
    q_bad = np.stack([synth.query(w, i) for i in range(room + 2)], axis=1)
    with pytest.raises(B.InnerQError) as ei:
        gc.innerq_decode_attention_multi(dev(q_bad))
    assert ei.value.status == -2
    # an unquantised cache has no fused kernel: refused as well
    wf = synth.tiny(n_tokens=40, grouping=O.FP16, k_normalize=0)
    _, gf, _, _ = run_prefill_both(wf)
    with pytest.raises(B.InnerQError) as ei:
        gf.innerq_decode_attention_multi(dev(np.stack([synth.query(wf, i) for i in range(2)], axis=1)))
    assert ei.value.status == -2


@pytest.mark.parametrize("grouping,r,G,bits", [(O.INNER, 1, 32, 2), (O.INNER, 4, 64, 2), (O.INNER, 2, 128, 4), (O.INNER, 1, 32, 3),
                                               (O.OUTER, 2, 32, 2)])
def test_batched_calls_over_sequences_of_different_lengths(grouping, r, G, bits):
    # every sequence has its own cache object and length; one launch appends to / decodes all of them
    from paper_2602_23200_b200 import binding as B
    inner = grouping == O.INNER
    lengths = [1, 37, 164, 700, 333, 4 + 16 + G]
    base = synth.tiny(batch=1, n_q_heads=2 * r, n_kv_heads=2, group=G, k_bits=bits, v_bits=bits, grouping=grouping,
                      k_normalize=int(inner), **({} if inner else dict(k_mode=O.ASYM, v_mode=O.ASYM)))
    ws, ocs, gcs = [], [], []
    for i, n in enumerate(lengths):
        w = base.with_(n_tokens=n, wid=base.wid + 100 + i)
        oc, gc, _, _ = run_prefill_both(w, max_tokens=1000)
        ws.append(w); ocs.append(oc); gcs.append(gc)

    def decode_all(step, who=None):
        who = list(range(len(gcs))) if who is None else who
        q = np.stack([synth.query(ws[i], step) for i in who])                      # [n, 1, Hq, D]
        out = B.innerq_decode_attention_batched([gcs[i] for i in who], dev(q)).cpu().numpy()
        for row, i in enumerate(who):
            P.assert_outputs_close(out[row], ocs[i].decode(q[row]), f"sequence {i} (N={ocs[i].N}) step {step}")

    decode_all(0)
    for step in range(2 * G + 3):                   # every sequence crosses group evictions at its own steps
        who = [i for i in range(len(gcs)) if not (i == 2 and step % 3 == 0)]       # sequence 2 skips some steps
        toks = [synth.new_token(ws[i], step) for i in who]
        for (k1, v1), i in zip(toks, who):
            ocs[i].append(k1, v1)
        B.innerq_append_token_batched([gcs[i] for i in who], dev(np.stack([t[0] for t in toks])),
                                      dev(np.stack([t[1] for t in toks])))
        if step in (0, 1, G - 1, G, 2 * G + 2):
            decode_all(step + 1)
            decode_all(step + 1, who=[3, 0])                                        # any subset, any order
    for i, (oc, gc) in enumerate(zip(ocs, gcs)):
        assert gc.n_tokens == oc.N
        P.assert_export_equal(gc.innerq_cache_export(), oc.export(), grouping, G, k_hybrid=inner, v_hybrid=inner)
        assert gc.innerq_read_device_error() == 0
    # a single-cache call on one of them still agrees
    q = synth.query(ws[4], 99)
    P.assert_outputs_close(gcs[4].innerq_decode_attention(dev(q)).cpu().numpy(), ocs[4].decode(q), "single after batched")


def test_batched_calls_with_caches_that_hold_a_batch_themselves():
    # every cache object may itself hold several sequences of one length: rows of k_new / q are [cache][batch, ...]
    from paper_2602_23200_b200 import binding as B
    base = synth.tiny(batch=3, n_q_heads=4, n_kv_heads=2, group=64)
    ws, ocs, gcs = [], [], []
    for i, n in enumerate([90, 333, 200]):
        w = base.with_(n_tokens=n, wid=base.wid + 700 + i)
        oc, gc, _, _ = run_prefill_both(w, max_tokens=500)
        ws.append(w); ocs.append(oc); gcs.append(gc)
    for step in range(70):
        toks = [synth.new_token(w, step) for w in ws]
        for (k1, v1), oc in zip(toks, ocs):
            oc.append(k1, v1)
        B.innerq_append_token_batched(gcs, dev(np.stack([t[0] for t in toks])), dev(np.stack([t[1] for t in toks])))
        if step in (0, 63, 64, 69):
            q = np.stack([synth.query(w, step) for w in ws])                     # [3, batch, Hq, D]
            out = B.innerq_decode_attention_batched(gcs, dev(q)).cpu().numpy()
            for i in range(3):
                P.assert_outputs_close(out[i], ocs[i].decode(q[i]), f"cache {i} step {step}")
    for w, oc, gc in zip(ws, ocs, gcs):
        P.assert_export_equal(gc.innerq_cache_export(), oc.export(), O.INNER, w.group)


def test_batched_calls_argument_checks():
    from paper_2602_23200_b200 import binding as B
    w = synth.tiny(batch=1, n_q_heads=2, n_kv_heads=2, n_tokens=50)
    _, a, _, _ = run_prefill_both(w, max_tokens=51)
    _, b, _, _ = run_prefill_both(w, max_tokens=51)
    _, other, _, _ = run_prefill_both(w.with_(group=64), max_tokens=51)
    q2 = dev(np.stack([synth.query(w, 0), synth.query(w, 1)]))
    k1, v1 = synth.new_token(w, 0)
    kv2 = dev(np.stack([k1, k1])), dev(np.stack([v1, v1]))
    for bad in ([a, a], [a, other]):                       # the same cache twice; different configurations
        with pytest.raises(B.InnerQError) as ei:
            B.innerq_decode_attention_batched(bad, q2)
        assert ei.value.status == -1
        with pytest.raises(B.InnerQError) as ei:
            B.innerq_append_token_batched(bad, *kv2)
        assert ei.value.status == -1
    B.innerq_append_token_batched([a], dev(k1[None]), dev(v1[None]))           # a is full now (51 of 51)
    with pytest.raises(B.InnerQError) as ei:
        B.innerq_append_token_batched([b, a], *kv2)
    assert ei.value.status == -3 and b.n_tokens == 50 and a.n_tokens == 51      # nothing was appended to b either
    wf = w.with_(grouping=O.FP16, k_normalize=0)
    _, f, _, _ = run_prefill_both(wf, max_tokens=51)
    with pytest.raises(B.InnerQError) as ei:
        B.innerq_decode_attention_batched([f], dev(synth.query(wf, 0)[None]))
    assert ei.value.status == -2
    out = B.innerq_decode_attention_batched([b, a], q2)
    assert _torch().isfinite(out.float()).all()


def test_batched_calls_with_more_caches_than_one_launch_takes():
    from paper_2602_23200_b200 import binding as B
    n = 37                                                  # a launch takes 32: two launches
    base = synth.tiny(batch=1, n_q_heads=2, n_kv_heads=1)
    ws, ocs, gcs = [], [], []
    for i in range(n):
        w = base.with_(n_tokens=20 + 13 * i, wid=base.wid + 300 + i)
        oc, gc, _, _ = run_prefill_both(w, max_tokens=600)
        ws.append(w); ocs.append(oc); gcs.append(gc)
    toks = [synth.new_token(ws[i], 0) for i in range(n)]
    for (k1, v1), oc in zip(toks, ocs):
        oc.append(k1, v1)
    B.innerq_append_token_batched(gcs, dev(np.stack([t[0] for t in toks])), dev(np.stack([t[1] for t in toks])))
    assert gcs[0].innerq_last_launch_count(1) == 2
    q = np.stack([synth.query(ws[i], 1) for i in range(n)])
    out = B.innerq_decode_attention_batched(gcs, dev(q)).cpu().numpy()
    for i in range(n):
        assert gcs[i].n_tokens == ocs[i].N
        P.assert_outputs_close(out[i], ocs[i].decode(q[i]), f"sequence {i} of {n}")


@pytest.mark.parametrize("grouping,r,G", [(O.INNER, 1, 32), (O.INNER, 4, 64), (O.OUTER, 2, 32)])
def test_steps_enqueued_back_to_back_without_host_synchronisation(grouping, r, G):
    # The kernels of consecutive steps overlap on the GPU (each is a programmatic dependent of the one before it and
    # the decode streams the settled part of the cache before it waits): enqueue many steps with no host
    # synchronisation in between, then check every step's output and the final cache against the oracle.
    torch = _torch()
    inner = grouping == O.INNER
    w = synth.tiny(batch=2, n_q_heads=4 * r, n_kv_heads=4, n_tokens=4 + 16 + 40 * 32 + 11, group=G, grouping=grouping,
                   k_normalize=int(inner), **({} if inner else dict(k_mode=O.ASYM, v_mode=O.ASYM)))
    n_steps = 2 * G + 9
    oc, gc, _, _ = run_prefill_both(w, max_tokens=w.n_tokens + n_steps + 4)
    toks = [synth.new_token(w, s) for s in range(n_steps)]
    qs = [synth.query(w, s) for s in range(n_steps)]
    k_all, v_all = dev(np.stack([t[0] for t in toks])), dev(np.stack([t[1] for t in toks]))
    q_all = dev(np.stack(qs))
    outs = torch.empty_like(q_all)
    torch.cuda.synchronize()
    for s in range(n_steps):                       # nothing here waits for the GPU
        gc.innerq_append_token(k_all[s], v_all[s])
        gc.innerq_decode_attention(q_all[s], outs[s])
        if s % 7 == 3:                             # some steps decode twice, some append twice in a row
            gc.innerq_decode_attention(q_all[s], outs[s])
    torch.cuda.synchronize()
    got = outs.cpu().numpy()
    for s in range(n_steps):
        oc.append(*toks[s])
        P.assert_outputs_close(got[s], oc.decode(qs[s]), f"step {s}")
    P.assert_export_equal(gc.innerq_cache_export(), oc.export(), grouping, G, k_hybrid=inner, v_hybrid=inner)
    assert gc.innerq_read_device_error() == 0


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_random_interleaving_of_calls_on_one_stream(seed):
    # Three caches of different formats share one stream; appends, decodes (fused and plain kernels), multi-query
    # decodes and exports are enqueued in random order with no host synchronisation except at exports.  Every output is
    # checked afterwards: the overlap of consecutive kernels must never let a decode miss an append.
    torch = _torch()
    rng = np.random.default_rng(seed)
    specs = [dict(n_q_heads=4, n_kv_heads=4, group=32, k_bits=2, v_bits=2, w_recent=16),
             dict(n_q_heads=8, n_kv_heads=2, group=64, k_bits=4, v_bits=4, w_recent=24),
             dict(n_q_heads=4, n_kv_heads=2, group=32, k_bits=2, v_bits=2, w_recent=16, grouping=O.OUTER, k_normalize=0,
                  k_mode=O.ASYM, v_mode=O.ASYM)]
    ws, ocs, gcs, steps = [], [], [], []
    pool = 160                                     # inputs are put on the device up front: no copy between the calls
    toks, qs, toks_d, qs_d = [], [], [], []
    for i, kw in enumerate(specs):
        w = synth.tiny(batch=1, n_tokens=4 + kw["w_recent"] + 60 * 32 + 5 * i, wid=500 + 10 * seed + i, **kw)
        oc, gc, _, _ = run_prefill_both(w, max_tokens=w.n_tokens + pool + 8)
        ws.append(w); ocs.append(oc); gcs.append(gc); steps.append(0)
        toks.append([synth.new_token(w, s_) for s_ in range(pool)])
        qs.append([synth.query(w, 1000 + s_) for s_ in range(pool)])
        toks_d.append((dev(np.stack([t[0] for t in toks[i]])), dev(np.stack([t[1] for t in toks[i]]))))
        qs_d.append(dev(np.stack(qs[i])))
    torch.cuda.synchronize()
    # 1. the sequence of calls (multi-query is always possible here: the recent window holds at least 16 tokens)
    ops = []
    n_queries = [0] * len(gcs)
    for it in range(300):
        i = int(rng.integers(len(gcs)))
        op = str(rng.choice(["append", "append", "decode", "decode", "plain", "multi"], p=[.3, .2, .25, .1, .05, .1]))
        if op == "append":
            if steps[i] >= pool:
                continue
            ops.append((op, i, steps[i], 0)); steps[i] += 1
        elif op == "multi":
            n_q = int(rng.integers(2, 5))
            ops.append((op, i, n_queries[i] % (pool - 4), n_q)); n_queries[i] += n_q
        else:
            ops.append((op, i, n_queries[i] % pool, 0)); n_queries[i] += 1
    # 2. everything is enqueued without the host ever waiting for the GPU
    outs = []
    for op, i, j, n_q in ops:
        gc = gcs[i]
        if op == "append":
            gc.innerq_append_token(toks_d[i][0][j], toks_d[i][1][j])
            outs.append(None)
        elif op == "multi":
            outs.append(gc.innerq_decode_attention_multi(qs_d[i][j:j + n_q].transpose(0, 1).contiguous()))
        else:
            gc.innerq_set_decode_options(0, 1 if op == "plain" else 0)
            outs.append(gc.innerq_decode_attention(qs_d[i][j]))
            gc.innerq_set_decode_options(0, 0)
    torch.cuda.synchronize()
    # 3. the oracle goes through the same sequence
    for (op, i, j, n_q), out in zip(ops, outs):
        oc = ocs[i]
        if op == "append":
            oc.append(*toks[i][j])
        elif op == "multi":
            P.assert_outputs_close(out.cpu().numpy(), oc.decode_multi(np.stack(qs[i][j:j + n_q], axis=1)), f"multi, cache {i}")
        else:
            P.assert_outputs_close(out.cpu().numpy(), oc.decode(qs[i][j]), f"{op}, cache {i}")
    for i, gc in enumerate(gcs):
        w = ws[i]
        assert gc.n_tokens == ocs[i].N and gc.innerq_read_device_error() == 0
        P.assert_export_equal(gc.innerq_cache_export(), ocs[i].export(), w.grouping, w.group,
                              k_hybrid=w.k_mode == O.HYBRID, v_hybrid=w.v_mode == O.HYBRID)


def test_capacity_and_argument_errors():
    from paper_2602_23200_b200 import binding as B
    torch = _torch()
    w = synth.tiny(n_tokens=40)
    gc = gpu_cache(w, max_tokens=41)
    K, V = synth.kv_all(w)
    gc.innerq_quantize_prefill(dev(K), dev(V))
    k1, v1 = synth.new_token(w, 0)
    gc.innerq_append_token(dev(k1), dev(v1))
    with pytest.raises(B.InnerQError) as ei:
        gc.innerq_append_token(dev(k1), dev(v1))
    assert ei.value.status == -3 and gc.n_tokens == 41
    K2, V2 = synth.kv_all(w.with_(n_tokens=42))
    with pytest.raises(B.InnerQError) as ei:
        gc.innerq_quantize_prefill(dev(K2), dev(V2))
    assert ei.value.status == -3 and gc.n_tokens == 41
    empty = gpu_cache(w, max_tokens=41)
    q = dev(synth.query(w))
    with pytest.raises(B.InnerQError) as ei:
        empty.innerq_decode_attention(q)
    assert ei.value.status == -1
    # the context is still healthy
    out = gc.innerq_decode_attention(q)
    assert torch.isfinite(out.float()).all()


def test_config1_full_parity():
    w = synth.config1()
    oc, gc, _, _ = run_prefill_both(w)
    flips = P.assert_export_equal(gc.innerq_cache_export(), oc.export(), O.INNER, w.group)
    worst = check_decode(w, oc, gc, variants=(0, 1, 3, 4), splits=(0, 1, 4, 13))
    print(f"config1: contested flips {flips}, worst err/tol {worst:.3f}")


@pytest.mark.parametrize("kw", [dict(), dict(group=64, k_bits=3, v_bits=3, n_q_heads=8), dict(k_bits=4, v_bits=2, k_mode=O.SYM),
                                dict(grouping=O.OUTER, k_normalize=0, k_mode=O.ASYM, v_mode=O.ASYM, group=64),
                                dict(grouping=O.FP16, k_normalize=0)],
                         ids=["2bit", "3bit_g64", "k4sym_v2", "outer", "fp16"])
def test_import_restores_an_exported_cache(kw):
    # checkpoint / resume: export a cache that has been prefilled and stepped, import the arrays into a fresh cache of
    # the same configuration: identical export, identical decode output (same bits), and both caches continue alike
    import torch
    w = synth.tiny(n_tokens=500, **kw)
    oc, gc, _, _ = run_prefill_both(w)
    for step in range(w.group + 5):
        k1, v1 = synth.new_token(w, step)
        oc.append(k1, v1)
        gc.innerq_append_token(dev(k1), dev(v1))
    saved = gc.innerq_cache_export()
    g2 = gpu_cache(w)
    g2.innerq_cache_import(saved)
    assert g2.n_tokens == gc.n_tokens
    again = g2.innerq_cache_export()
    for key, val in saved.items():
        assert np.array_equal(np.asarray(val), np.asarray(again[key])), key
    q = dev(synth.query(w, 3))
    assert torch.equal(gc.innerq_decode_attention(q), g2.innerq_decode_attention(q))
    check_decode(w, oc, g2, step=3)
    for step in range(100, 100 + w.group + 2):                 # both continue through another group eviction
        k1, v1 = synth.new_token(w, step)
        oc.append(k1, v1)
        for c in (gc, g2):
            c.innerq_append_token(dev(k1), dev(v1))
    a, b = gc.innerq_cache_export(), g2.innerq_cache_export()
    for key, val in a.items():
        assert np.array_equal(np.asarray(val), np.asarray(b[key])), key
    check_decode(w, oc, g2, step=9)
