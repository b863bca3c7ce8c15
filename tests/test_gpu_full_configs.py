"""Parity at the benchmark configurations' full sizes (needs a B200).

The CUDA path runs the whole workload in the launch configuration `bench.py` uses; the oracle, which
would need minutes for all (batch, KV head) units, is run on a sample of units and compared on those:
packed codes / scales / zero-points / masks / norms / windows bit-exact, attention outputs within
|err| <= 2e-3 * max|out| + 1e-3.
"""
import numpy as np
import pytest

from oracle import innerq_oracle as O
from paper_2602_23200_b200 import synth
from tests import _parity as P

pytestmark = pytest.mark.gpu


def dev(x):
    import torch
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def make_gpu(w, K, V, extra=64):
    from paper_2602_23200_b200 import binding as B
    gc = B.InnerQCache(B.make_config(w, max_tokens=w.n_tokens + extra))
    gc.innerq_quantize_prefill(dev(K), dev(V))
    return gc


def sub_oracle(w, K, V, units, extra=64):
    """Oracle over the sampled units only, laid out as batch 1 with len(units) KV heads."""
    Ku = K.reshape(w.n_units, w.n_tokens, w.head_dim)[units]
    Vu = V.reshape(w.n_units, w.n_tokens, w.head_dim)[units]
    ws = w.with_(batch=1, n_kv_heads=len(units), n_q_heads=len(units) * w.q_per_kv)
    oc = O.from_workload(ws, max_tokens=w.n_tokens + extra)
    oc.prefill(Ku[None], Vu[None])
    return oc


def q_rows(w, q, units):
    """Query heads of the sampled units, as the sub-oracle's [1, len(units) * r, D]."""
    r = w.q_per_kv
    rows = [q[u // w.n_kv_heads, (u % w.n_kv_heads) * r + i] for u in units for i in range(r)]
    return np.stack(rows)[None]


def slice_export(e, units):
    out = {}
    for k, v in e.items():
        out[k] = v[units] if isinstance(v, np.ndarray) and v.ndim >= 2 else v
    return out


def compare(w, gc, oc, units, step=0, check_export=True):
    if check_export:
        flips = P.assert_export_equal(slice_export(gc.innerq_cache_export(), units), oc.export(), w.grouping, w.group,
                                      w.k_mode == O.HYBRID, w.v_mode == O.HYBRID)
    else:
        flips = 0
    q = synth.query(w, step)
    out = gc.innerq_decode_attention(dev(q)).cpu().numpy()
    ref = oc.decode(q_rows(w, q, units))
    worst = P.assert_outputs_close(q_rows(w, out, units), ref, f"{w.name} step {step}")
    assert gc.innerq_read_device_error() == 0
    return flips, worst


def kv_tiled_over_batch(w):
    """K, V with batch entry 0 generated and repeated over the batch (generation time of the large configs)."""
    K1, V1 = synth.kv_all(w.with_(batch=1))
    return np.repeat(K1, w.batch, axis=0), np.repeat(V1, w.batch, axis=0)


def test_config2_prefill_then_steps():
    # 32 heads x 32768 tokens, 2-bit, G = 32; each step appends one token, then decodes.
    w = synth.config2()
    K, V = synth.kv_all(w)
    units = [0, 13, 31]
    gc, oc = make_gpu(w, K, V, extra=128), sub_oracle(w, K, V, units, extra=128)
    compare(w, gc, oc, units, step=1000)
    worst = 0.0
    for step in range(40):                      # crosses value-group evictions (every 32 steps) and 40 key evictions
        k1, v1 = synth.new_token(w, step)
        gc.innerq_append_token(dev(k1), dev(v1))
        oc.append(k1.reshape(w.n_units, -1)[units][None], v1.reshape(w.n_units, -1)[units][None])
        if step in (0, 3, 4, 5, 35, 36, 39):
            _, e = compare(w, gc, oc, units, step=step, check_export=step in (4, 39))
            worst = max(worst, e)
    print(f"config2: worst err/tol over steps {worst:.3f}")
    # 40 more steps enqueued back to back, no host synchronisation in between (the way bench.py's timed loop runs:
    # the kernels of consecutive steps overlap), every step's output checked afterwards
    import torch
    n_more = 40
    toks = [synth.new_token(w, 100 + s) for s in range(n_more)]
    qs = [synth.query(w, 100 + s) for s in range(n_more)]
    k_all, v_all, q_all = dev(np.stack([t[0] for t in toks])), dev(np.stack([t[1] for t in toks])), dev(np.stack(qs))
    outs = torch.empty_like(q_all)
    torch.cuda.synchronize()
    for s in range(n_more):
        gc.innerq_append_token(k_all[s], v_all[s])
        gc.innerq_decode_attention(q_all[s], outs[s])
    torch.cuda.synchronize()
    got = outs.cpu().numpy()
    worst_b2b = 0.0
    for s in range(n_more):
        k1, v1 = toks[s]
        oc.append(k1.reshape(w.n_units, -1)[units][None], v1.reshape(w.n_units, -1)[units][None])
        ref = oc.decode(q_rows(w, qs[s], units))
        worst_b2b = max(worst_b2b, P.assert_outputs_close(q_rows(w, got[s], units), ref, f"back-to-back step {s}"))
    P.assert_export_equal(slice_export(gc.innerq_cache_export(), units), oc.export(), w.grouping, w.group, True, True)
    assert gc.innerq_read_device_error() == 0
    print(f"config2, 40 steps back to back: worst err/tol {worst_b2b:.3f}")
    # the generic kernel on the same cache (full size): an on-device cross-check of the packed layout
    gc.innerq_set_decode_options(0, 1)
    _, e1 = compare(w, gc, oc, units, step=77, check_export=False)
    gc.innerq_set_decode_options(0, 0)
    print(f"config2, generic kernel: err/tol {e1:.3f}")


@pytest.mark.parametrize("splits", [0, 4])
def test_config2_inputs_written_by_the_kernel_right_before_each_call(splits):
    # splits = 4: one CTA per SM and launch, so that two or three consecutive decodes are resident at the same time
    # (the operating point bench.py reports as one_cta_per_sm_launches); 0: the default, one wave per launch.
    # The way a model uses the library: q, k_new and v_new of every step are produced on the same stream by an
    # ordinary kernel (here an elementwise op into three buffers that are REUSED by every step) immediately before
    # innerq_append_token / innerq_decode_attention, which are launched as programmatic dependents and read their
    # inputs before they wait for their predecessors.  120 steps enqueued without host synchronisation; every
    # output and the final cache contents against the oracle.
    import torch
    w = synth.config2()
    K, V = synth.kv_all(w)
    units = [7, 24]
    n_steps = 120
    gc, oc = make_gpu(w, K, V, extra=n_steps + 8), sub_oracle(w, K, V, units, extra=n_steps + 8)
    gc.innerq_set_decode_options(splits, 0)
    del K, V
    toks = [synth.new_token(w, 500 + s) for s in range(n_steps)]
    qs = [synth.query(w, 500 + s) for s in range(n_steps)]
    k_src, v_src, q_src = dev(np.stack([t[0] for t in toks])), dev(np.stack([t[1] for t in toks])), dev(np.stack(qs))
    k_buf, v_buf, q_buf = torch.zeros_like(k_src[0]), torch.zeros_like(v_src[0]), torch.zeros_like(q_src[0])
    one = torch.ones((), dtype=torch.float16, device="cuda")
    outs = torch.empty_like(q_src)
    torch.cuda.synchronize()
    for s in range(n_steps):
        torch.mul(k_src[s], one, out=k_buf)              # three ordinary kernels: the step's inputs come into being
        torch.mul(v_src[s], one, out=v_buf)
        if s % 2 == 0:
            torch.mul(q_src[s], one, out=q_buf)          # q before the append on even steps ...
        gc.innerq_append_token(k_buf, v_buf)
        if s % 2 == 1:
            torch.mul(q_src[s], one, out=q_buf)          # ... and between append and decode on odd ones
        gc.innerq_decode_attention(q_buf, outs[s])
    torch.cuda.synchronize()
    got = outs.cpu().numpy()
    worst = 0.0
    for s in range(n_steps):
        k1, v1 = toks[s]
        oc.append(k1.reshape(w.n_units, -1)[units][None], v1.reshape(w.n_units, -1)[units][None])
        ref = oc.decode(q_rows(w, qs[s], units))
        worst = max(worst, P.assert_outputs_close(q_rows(w, got[s], units), ref, f"produced inputs, step {s}"))
    P.assert_export_equal(slice_export(gc.innerq_cache_export(), units), oc.export(), w.grouping, w.group, True, True)
    assert gc.innerq_read_device_error() == 0
    print(f"config2, inputs produced on the stream, {n_steps} steps back to back: worst err/tol {worst:.3f}")


def test_config2_paged_cache():
    # the same workload with the packed records in 512-token pages of a pool, handed out in a shuffled order; the
    # steps are enqueued back to back and cross a page boundary (the 32636 packed key rows of the prefill fill 63.7 pages)
    import torch
    from paper_2602_23200_b200 import binding as B
    w = synth.config2()
    K, V = synth.kv_all(w)
    units = [5, 30]
    n_steps, page = 140, 512
    cfg = B.make_config(w, max_tokens=w.n_tokens + n_steps + 8)
    n_pages = (w.n_tokens + n_steps) // page + 3
    pool = B.PagePool(cfg, page, n_pages, order=np.random.default_rng(17).permutation(n_pages))
    pool.buf.fill_(0x5A)
    gc = B.InnerQCache(cfg, pool=pool)
    gc.ensure_pages(w.n_tokens)
    gc.innerq_quantize_prefill(dev(K), dev(V))
    oc = sub_oracle(w, K, V, units, extra=n_steps + 8)
    compare(w, gc, oc, units, step=500)
    toks = [synth.new_token(w, 300 + s) for s in range(n_steps)]
    qs = [synth.query(w, 300 + s) for s in range(n_steps)]
    k_all, v_all, q_all = dev(np.stack([t[0] for t in toks])), dev(np.stack([t[1] for t in toks])), dev(np.stack(qs))
    outs = torch.empty_like(q_all)
    pages_before = gc.pages_assigned
    torch.cuda.synchronize()
    for s in range(n_steps):
        gc.ensure_pages(gc.n_tokens + 1)
        gc.innerq_append_token(k_all[s], v_all[s])
        gc.innerq_decode_attention(q_all[s], outs[s])
    torch.cuda.synchronize()
    assert gc.pages_assigned == pages_before + 1
    got = outs.cpu().numpy()
    worst = 0.0
    for s in range(n_steps):
        k1, v1 = toks[s]
        oc.append(k1.reshape(w.n_units, -1)[units][None], v1.reshape(w.n_units, -1)[units][None])
        if s < 2 or 124 <= s < 134 or s == n_steps - 1:
            ref = oc.decode(q_rows(w, qs[s], units))
            worst = max(worst, P.assert_outputs_close(q_rows(w, got[s], units), ref, f"paged, step {s}"))
    P.assert_export_equal(slice_export(gc.innerq_cache_export(), units), oc.export(), w.grouping, w.group, True, True)
    assert gc.innerq_read_device_error() == 0
    print(f"config2, paged cache, {n_steps} steps back to back: worst err/tol {worst:.3f}")


@pytest.mark.parametrize("bits", [4, 2])
def test_config3_gqa_batch16(bits):
    w = synth.config3(bits)
    K, V = synth.kv_all(w)
    units = [0, 77, 127]
    gc, oc = make_gpu(w, K, V), sub_oracle(w, K, V, units)
    flips, worst = compare(w, gc, oc, units)
    k1, v1 = synth.new_token(w, 0)
    gc.innerq_append_token(dev(k1), dev(v1))
    oc.append(k1.reshape(w.n_units, -1)[units][None], v1.reshape(w.n_units, -1)[units][None])
    _, worst2 = compare(w, gc, oc, units, step=1)
    print(f"config3 {bits}-bit: contested flips {flips}, worst err/tol {max(worst, worst2):.3f}")


@pytest.mark.parametrize("kb,vb,sym", [(3, 3, False), (3, 2, True), (4, 4, False)])
def test_config2_shape_with_other_code_widths(kb, vb, sym):
    # the 32-head, 32768-token shape with 3- and 4-bit codes (one query head per KV head and G = 32: the kernel
    # instance whose MMA columns are groups, not heads); sym: the paper's presets keep the keys symmetric
    w = synth.config2().with_(k_bits=kb, v_bits=vb)
    if sym:
        w = w.with_(k_mode=O.SYM)
    K, V = synth.kv_all(w)
    units = [3, 18]
    gc, oc = make_gpu(w, K, V), sub_oracle(w, K, V, units)
    del K, V
    flips, worst = compare(w, gc, oc, units)
    for step in range(3):
        k1, v1 = synth.new_token(w, step)
        gc.innerq_append_token(dev(k1), dev(v1))
        oc.append(k1.reshape(w.n_units, -1)[units][None], v1.reshape(w.n_units, -1)[units][None])
    _, worst2 = compare(w, gc, oc, units, step=3)
    print(f"config-2 shape k{kb}v{vb}: contested flips {flips}, worst err/tol {max(worst, worst2):.3f}")


def test_config4_long_context_prefill_and_decode():
    # batch 4 x 8 KV heads x 131072 tokens, 2-bit, G = 128: full prefill quantisation, then decode.
    w = synth.config4()
    K, V = kv_tiled_over_batch(w)
    units = [3, 20]
    gc, oc = make_gpu(w, K, V), sub_oracle(w, K, V, units)
    del K, V
    flips, worst = compare(w, gc, oc, units)
    print(f"config4: contested flips {flips}, worst err/tol {worst:.3f}")


SWEEP = [(b, g, m, O.INNER, 0) for b in (2, 3, 4) for g in (32, 64, 128) for m in (O.HYBRID, O.ASYM)] + \
        [(2, 64, O.HYBRID, O.INNER, 1), (2, 64, O.ASYM, O.OUTER, 0), (4, 64, O.ASYM, O.OUTER, 0), (2, 64, O.ASYM, O.FP16, 0)]


@pytest.mark.parametrize("bits,G,mode,grouping,variant", SWEEP)
def test_config5_sweep_point(bits, G, mode, grouping, variant):
    # The sweep of bits x group size x mode on the config-3 shape and data; batch reduced from 16 to 2 to keep
    # the run short (units are independent), full context length.
    w = synth.config5(bits, G, mode, grouping, variant).with_(batch=2)
    K, V = synth.kv_all(w)
    units = [5]
    gc = make_gpu(w, K, V)
    oc = sub_oracle(w, K, V, units)
    if grouping == O.FP16:
        q = synth.query(w)
        out = gc.innerq_decode_attention(dev(q)).cpu().numpy()
        P.assert_outputs_close(q_rows(w, out, units), oc.decode(q_rows(w, q, units)), "fp16 cache")
        return
    compare(w, gc, oc, units)


def test_config2_multi_query_call():
    # four query tokens per call on the 32-head / 32768-token cache (the configuration bench.py's multi-query leg
    # times): sampled heads against the oracle's causal decode of the same cache state
    w = synth.config2()
    K, V = synth.kv_all(w)
    units = [2, 30]
    gc, oc = make_gpu(w, K, V), sub_oracle(w, K, V, units)
    n_q = 4
    q = np.stack([synth.query(w, 200 + i) for i in range(n_q)], axis=1)                  # [B, n_q, Hq, D]
    out = gc.innerq_decode_attention_multi(dev(q)).cpu().numpy()
    q_sub = np.stack([q_rows(w, q[:, i], units)[0] for i in range(n_q)], axis=0)[None]   # [1, n_q, len(units)*r, D]
    ref = oc.decode_multi(q_sub)
    got = np.stack([q_rows(w, out[:, i], units)[0] for i in range(n_q)], axis=0)[None]
    worst = P.assert_outputs_close(got, ref, "config2 multi-query")
    assert gc.innerq_read_device_error() == 0
    print(f"config2, 4 query tokens per call: worst err/tol {worst:.3f}")


def test_config3_shape_sequences_of_different_lengths():
    # the batched call of bench.py's ragged leg: 16 sequences (8 KV heads, r = 4, 2-bit, G = 64) of 1024 .. 8192
    # tokens, one cache object each; two of the sequences are checked against their own oracle caches
    from paper_2602_23200_b200 import binding as B
    w = synth.config3(2)
    fracs = [1.0, 0.125, 0.5, 0.25, 0.75, 1.0, 0.375, 0.625]
    lengths = [int(w.n_tokens * fracs[i % len(fracs)]) for i in range(w.batch)]
    w1 = w.with_(batch=1)
    K, V = synth.kv_all(w1)                       # one sequence's data, cut to each length
    cfg = B.make_config(w1, max_tokens=w.n_tokens + 8)
    caches = []
    for n in lengths:
        c = B.InnerQCache(cfg)
        c.innerq_quantize_prefill(dev(K[:, :, :n]), dev(V[:, :, :n]))
        caches.append(c)
    q = np.stack([synth.query(w1, i) for i in range(w.batch)])                           # [16, 1, Hq, D]
    out = B.innerq_decode_attention_batched(caches, dev(q)).cpu().numpy()
    worst = 0.0
    for i in (1, 4):                              # 1024 and 6144 tokens
        wi = w1.with_(n_tokens=lengths[i])
        Ki, Vi = K[:, :, :lengths[i]], V[:, :, :lengths[i]]
        units = [0, 5]
        oc = sub_oracle(wi, np.ascontiguousarray(Ki), np.ascontiguousarray(Vi), units)
        ref = oc.decode(q_rows(wi, q[i], units))
        worst = max(worst, P.assert_outputs_close(q_rows(wi, out[i], units), ref, f"sequence {i}"))
    for c in caches:
        assert c.innerq_read_device_error() == 0
    print(f"config-3 shape, 16 sequences of mixed lengths: worst err/tol {worst:.3f}")
