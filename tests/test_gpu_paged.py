"""Paged caches (packed records in pages of a shared pool) against the CPU oracle, through the C ABI (needs a B200).

The oracle knows nothing of pages: a paged cache must give, element by element, what a contiguous one gives.  Pools
hand their pages out in a seeded random order, so consecutive page slots are never neighbours in memory."""
import numpy as np
import pytest

from oracle import innerq_oracle as O
from paper_2602_23200_b200 import synth
from tests import _parity as P

pytestmark = pytest.mark.gpu

ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CAPACITY = -1, -2, -3      # include/innerq.h


def _torch():
    import torch
    return torch


def dev(x):
    return _torch().from_numpy(np.ascontiguousarray(x)).cuda()


def make_pool(cfg, page_tokens, n_pages, seed=0):
    from paper_2602_23200_b200 import binding as B
    order = np.random.default_rng(seed).permutation(n_pages)
    pool = B.PagePool(cfg, page_tokens, n_pages, order=order)
    pool.buf.fill_(0xA5)          # stale bytes in every page
    return pool


def paged_pair(w, page_tokens, max_tokens, n_pages=None, seed=0, pool=None):
    """(oracle cache, paged CUDA cache) prefilled with the workload's tokens."""
    from paper_2602_23200_b200 import binding as B
    cfg = B.make_config(w, max_tokens=max_tokens)
    if pool is None:
        pool = make_pool(cfg, page_tokens, n_pages or (max_tokens // page_tokens + 3), seed)
    gc = B.InnerQCache(cfg, pool=pool)
    K, V = synth.kv_all(w)
    oc = O.from_workload(w, max_tokens=max_tokens)
    oc.prefill(K, V)
    gc.ensure_pages(w.n_tokens)
    gc.innerq_quantize_prefill(dev(K), dev(V))
    return oc, gc


def check_decode(w, oc, gc, step=0, variants=(0,), splits=(0,)):
    q = synth.query(w, step)
    ref = oc.decode(q)
    for variant in variants:
        for s in splits:
            gc.innerq_set_decode_options(s, variant)
            out = gc.innerq_decode_attention(dev(q)).cpu().numpy()
            P.assert_outputs_close(out, ref, f"{w.name} paged variant={variant} splits={s}")
    gc.innerq_set_decode_options(0, 0)
    assert gc.innerq_read_device_error() == 0


def steps(w, oc, gc, first, n, check_every=0, **kw):
    for s in range(first, first + n):
        k1, v1 = synth.new_token(w, s)
        oc.append(k1, v1)
        gc.ensure_pages(gc.n_tokens + 1)
        gc.innerq_append_token(dev(k1), dev(v1))
        if check_every and (s - first) % check_every == check_every - 1:
            check_decode(w, oc, gc, step=s, **kw)


# key bits, value bits, key mode, value mode, G, query heads per KV head, grouping, tokens at prefill, page size
PAGED_CASES = [
    (2, 2, O.HYBRID, O.HYBRID, 32, 1, O.INNER, 700, 128),      # one chunk per group, two chunks per copy
    (2, 2, O.HYBRID, O.HYBRID, 32, 1, O.INNER, 733, 256),
    (2, 2, O.HYBRID, O.HYBRID, 64, 4, O.INNER, 600, 128),
    (2, 2, O.ASYM, O.ASYM, 128, 2, O.INNER, 900, 128),         # a page is one group
    (3, 2, O.SYM, O.HYBRID, 32, 1, O.INNER, 650, 128),
    (3, 3, O.HYBRID, O.HYBRID, 64, 8, O.INNER, 555, 256),
    (4, 4, O.HYBRID, O.HYBRID, 32, 4, O.INNER, 500, 128),
    (4, 4, O.SYM, O.SYM, 128, 1, O.INNER, 1100, 512),
    (2, 2, O.ASYM, O.ASYM, 32, 2, O.OUTER, 700, 128),
    (4, 4, O.ASYM, O.ASYM, 64, 4, O.OUTER, 600, 256),
    (3, 3, O.ASYM, O.ASYM, 64, 1, O.OUTER, 420, 128),          # generic kernel only
]


@pytest.mark.parametrize("kb,vb,km,vm,G,r,grouping,N,page", PAGED_CASES)
def test_paged_prefill_appends_and_decode(kb, vb, km, vm, G, r, grouping, N, page):
    inner = grouping == O.INNER
    w = synth.tiny(n_tokens=N, group=G, k_bits=kb, v_bits=vb, k_mode=km, v_mode=vm, n_q_heads=2 * r, grouping=grouping,
                   k_normalize=int(inner))
    n_steps = 2 * page + G + 5                      # the appends cross two page boundaries
    oc, gc = paged_pair(w, page, max_tokens=N + n_steps + 8, seed=kb * 7 + G)
    hyb = (km == O.HYBRID, vm == O.HYBRID)
    P.assert_export_equal(gc.innerq_cache_export(), oc.export(), grouping, G, *hyb)
    check_decode(w, oc, gc, variants=(0, 1), splits=(0, 1, 3, 7))
    steps(w, oc, gc, 0, n_steps, check_every=37, variants=(0,), splits=(0, 5))
    P.assert_export_equal(gc.innerq_cache_export(), oc.export(), grouping, G, *hyb)
    check_decode(w, oc, gc, step=3, variants=(0, 1), splits=(0, 2))
    assert gc.pages_assigned == gc.innerq_cache_pages_for(gc.n_tokens)


def test_paged_cache_grows_from_empty():
    from paper_2602_23200_b200 import binding as B
    torch = _torch()
    w = synth.tiny(n_tokens=0, w_sink=4, w_recent=16, group=32)
    cfg = B.make_config(w, max_tokens=400)
    gc = B.InnerQCache(cfg, pool=make_pool(cfg, 128, 5, seed=3))
    oc = O.from_workload(w, max_tokens=400)
    empty = torch.empty((w.batch, w.n_kv_heads, 0, 128), dtype=torch.float16, device="cuda")
    gc.innerq_quantize_prefill(empty, empty)
    assert gc.pages_assigned == 0 and gc.innerq_cache_pages_for(20) == 0 and gc.innerq_cache_pages_for(21) == 1
    steps(w, oc, gc, 0, 300, check_every=29, variants=(0, 1))
    P.assert_export_equal(gc.innerq_cache_export(), oc.export(), O.INNER, 32)
    assert gc.pages_assigned == 3


def test_two_caches_share_a_pool_and_a_third_reuses_released_pages():
    from paper_2602_23200_b200 import binding as B
    wa = synth.tiny(n_tokens=500, group=64, n_q_heads=8).with_(wid=21)
    wb = synth.tiny(n_tokens=333, group=64, n_q_heads=8).with_(wid=22)
    cfg = B.make_config(wa, max_tokens=900)
    pool = make_pool(cfg, 128, 12, seed=5)
    oa, ga = paged_pair(wa, 128, 900, pool=pool)
    ob, gb = paged_pair(wb, 128, 900, pool=pool)
    for s in range(0, 200, 2):                      # the caches grow in turns: their pages interleave in the pool
        steps(wa, oa, ga, s, 2)
        steps(wb, ob, gb, s, 2)
    check_decode(wa, oa, ga, step=1, splits=(0, 3))
    check_decode(wb, ob, gb, step=2, splits=(0, 3))
    P.assert_export_equal(ga.innerq_cache_export(), oa.export(), O.INNER, 64)
    P.assert_export_equal(gb.innerq_cache_export(), ob.export(), O.INNER, 64)
    # cache A ends: its pages go back to the pool, dirty, and a new sequence takes them
    held = ga.pages_assigned
    free_before = len(pool.free)
    ga.release_to_pool()
    assert ga.n_tokens == 0 and ga.pages_assigned == 0 and len(pool.free) == free_before + held
    pool.free = pool.free[-held:] + pool.free[:-held]            # hand the released pages out first
    wc = synth.tiny(n_tokens=640, group=64, n_q_heads=8).with_(wid=23)
    oc, gc = paged_pair(wc, 128, 900, pool=pool)
    steps(wc, oc, gc, 0, 70)
    check_decode(wc, oc, gc, step=4, variants=(0, 1), splits=(0, 2))
    P.assert_export_equal(gc.innerq_cache_export(), oc.export(), O.INNER, 64)
    # ... and cache B never noticed
    steps(wb, ob, gb, 200, 3)
    check_decode(wb, ob, gb, step=5)
    P.assert_export_equal(gb.innerq_cache_export(), ob.export(), O.INNER, 64)


@pytest.mark.parametrize("grouping,r,G", [(O.INNER, 1, 32), (O.INNER, 4, 128), (O.OUTER, 2, 32)])
def test_paged_batched_calls_over_sequences_of_different_lengths(grouping, r, G):
    from paper_2602_23200_b200 import binding as B
    inner = grouping == O.INNER
    lengths = [900, 37, 411, 5, 1290, 260]
    n_steps = 140
    base = synth.tiny(batch=1, n_kv_heads=2, n_q_heads=2 * r, group=G, grouping=grouping, k_normalize=int(inner),
                      **({} if inner else dict(k_mode=O.ASYM, v_mode=O.ASYM)))
    ws = [base.with_(n_tokens=n, wid=40 + i) for i, n in enumerate(lengths)]
    cap = max(lengths) + n_steps + 8
    cfg = B.make_config(ws[0], max_tokens=cap)
    pool = make_pool(cfg, 128, sum((n + n_steps) // 128 + 2 for n in lengths), seed=11)
    pairs = [paged_pair(w, 128, cap, pool=pool) for w in ws]
    caches = [g for _, g in pairs]
    for s in range(n_steps):
        toks = [synth.new_token(w, s) for w in ws]
        for (oc, gc), (k1, v1) in zip(pairs, toks):
            oc.append(k1, v1)
            gc.ensure_pages(gc.n_tokens + 1)
        B.innerq_append_token_batched(caches, dev(np.stack([t[0] for t in toks])), dev(np.stack([t[1] for t in toks])))
        if s % 23 == 22 or s == n_steps - 1:
            qs = [synth.query(w, s) for w in ws]
            out = B.innerq_decode_attention_batched(caches, dev(np.stack(qs))).cpu().numpy()
            for i, (oc, _) in enumerate(pairs):
                P.assert_outputs_close(out[i], oc.decode(qs[i]), f"sequence {i} step {s}")
    for oc, gc in pairs:
        P.assert_export_equal(gc.innerq_cache_export(), oc.export(), grouping, G, inner, inner)
        assert gc.innerq_read_device_error() == 0


def test_paged_multi_query_call():
    w = synth.tiny(n_tokens=800, group=32, n_q_heads=2)
    oc, gc = paged_pair(w, 128, 900, seed=2)
    steps(w, oc, gc, 0, 40)
    n_q = 5
    rng = np.random.default_rng(8)
    q = rng.standard_normal((w.batch, n_q, w.n_q_heads, 128)).astype(np.float16)
    out = gc.innerq_decode_attention_multi(dev(q)).cpu().numpy()
    ref = oc.decode_multi(q)
    for i in range(n_q):
        P.assert_outputs_close(out[:, i], ref[:, i], f"query {i}")


@pytest.mark.parametrize("early", [True, False])
def test_paged_steps_enqueued_back_to_back(early):
    # No host synchronisation between steps: kernels of consecutive steps overlap.  Pages are assigned either well
    # before the step that first writes them or right before it (the table update is then a copy between two kernels).
    torch = _torch()
    w = synth.tiny(batch=2, n_q_heads=4, n_kv_heads=4, n_tokens=4 + 16 + 20 * 32 + 11, group=32)
    n_steps = 300
    oc, gc = paged_pair(w, 128, w.n_tokens + n_steps + 4, seed=9)
    if early:
        gc.ensure_pages(w.n_tokens + n_steps)
    toks = [synth.new_token(w, s) for s in range(n_steps)]
    qs = [synth.query(w, s) for s in range(n_steps)]
    k_all, v_all = dev(np.stack([t[0] for t in toks])), dev(np.stack([t[1] for t in toks]))
    q_all = dev(np.stack(qs))
    outs = torch.empty_like(q_all)
    torch.cuda.synchronize()
    for s in range(n_steps):
        gc.ensure_pages(gc.n_tokens + 1)
        gc.innerq_append_token(k_all[s], v_all[s])
        gc.innerq_decode_attention(q_all[s], outs[s])
    torch.cuda.synchronize()
    got = outs.cpu().numpy()
    for s in range(n_steps):
        oc.append(*toks[s])
        if s % 3 == 0 or s > n_steps - 5:
            P.assert_outputs_close(got[s], oc.decode(qs[s]), f"step {s}")
    P.assert_export_equal(gc.innerq_cache_export(), oc.export(), O.INNER, 32)
    assert gc.innerq_read_device_error() == 0


def test_paged_argument_and_capacity_errors():
    from paper_2602_23200_b200 import binding as B
    w = synth.tiny(n_tokens=300, group=32)
    cfg = B.make_config(w, max_tokens=600)
    for bad in (0, 64, 192, -128):
        with pytest.raises(B.InnerQError) as e:
            B.innerq_paged_cache_bytes(cfg, bad)
        assert e.value.status == ERR_INVALID_ARG
    with pytest.raises(B.InnerQError) as e:
        B.innerq_paged_cache_bytes(B.make_config(w, max_tokens=600, grouping=B.GROUPING_FP16), 128)
    assert e.value.status == ERR_UNSUPPORTED
    cb, wb, pb, mp = B.innerq_paged_cache_bytes(cfg, 128)
    assert mp == -(-(600 - 4 - 16 + 32) // 128) and pb % 256 == 0
    assert cb < B.innerq_cache_bytes(cfg)[0]            # the packed records are not in the cache buffer
    pool = make_pool(cfg, 128, 6)
    gc = B.InnerQCache(cfg, pool=pool)
    K, V = synth.kv_all(w)
    with pytest.raises(B.InnerQError) as e:             # no pages yet
        gc.innerq_quantize_prefill(dev(K), dev(V))
    assert e.value.status == ERR_CAPACITY and gc.n_tokens == 0
    need = gc.innerq_cache_pages_for(300)
    assert need == 3
    for bad in ([6], [-1], [0, 0]):
        with pytest.raises(B.InnerQError) as e:
            gc.innerq_cache_assign_pages(bad)
        assert e.value.status == ERR_INVALID_ARG and gc.pages_assigned == 0
    gc.innerq_cache_assign_pages([4, 1])
    with pytest.raises(B.InnerQError) as e:             # page 1 is already in this cache
        gc.innerq_cache_assign_pages([2, 1])
    assert e.value.status == ERR_INVALID_ARG and gc.pages_assigned == 2
    with pytest.raises(B.InnerQError) as e:             # still one page short
        gc.innerq_quantize_prefill(dev(K), dev(V))
    assert e.value.status == ERR_CAPACITY
    gc.innerq_cache_assign_pages([5])
    gc.innerq_quantize_prefill(dev(K), dev(V))
    oc = O.from_workload(w, max_tokens=600)
    oc.prefill(K, V)
    # tokens until the next page is needed: appends work up to there, then report CAPACITY and change nothing
    n = 300
    while gc.innerq_cache_pages_for(n + 1) == 3:
        n += 1
    for s in range(n - 300):
        k1, v1 = synth.new_token(w, s)
        oc.append(k1, v1)
        gc.innerq_append_token(dev(k1), dev(v1))
    k1, v1 = synth.new_token(w, 999)
    with pytest.raises(B.InnerQError) as e:
        gc.innerq_append_token(dev(k1), dev(v1))
    assert e.value.status == ERR_CAPACITY and gc.n_tokens == n
    check_decode(w, oc, gc, variants=(0, 1))
    with pytest.raises(B.InnerQError) as e:             # at most max_pages
        gc.innerq_cache_assign_pages([0, 2, 3])
    assert e.value.status == ERR_CAPACITY
    # a contiguous cache has no pages
    cc = B.InnerQCache(cfg)
    assert cc.innerq_cache_pages_for(500) == 0 and cc.pages_assigned == 0
    with pytest.raises(B.InnerQError) as e:
        cc.innerq_cache_assign_pages([0])
    assert e.value.status == ERR_INVALID_ARG


@pytest.mark.parametrize("seed", [1, 2])
def test_random_interleaving_of_calls_on_paged_caches(seed):
    # Two pools (two formats), two caches on each; appends (pages taken just in time), decodes with both kernels,
    # multi-query decodes and restarts (a cache hands its pages back and is prefilled with a new sequence out of the
    # same pool) are enqueued in random order on one stream with no host synchronisation; every output is checked
    # against the oracle afterwards.
    from paper_2602_23200_b200 import binding as B
    torch = _torch()
    rng = np.random.default_rng(100 + seed)
    specs = [dict(n_q_heads=4, n_kv_heads=4, group=32, k_bits=2, v_bits=2, w_recent=16),
             dict(n_q_heads=8, n_kv_heads=2, group=64, k_bits=3, v_bits=2, k_mode=O.SYM, w_recent=24)]
    n_in, cap = 200, 1400
    slots = []                                     # one per cache: dict(w, oc, gc, step, spec index, pool)
    inputs = {}                                    # wid -> host and device copies of the tokens and queries

    def sequence(si, wid, n_tokens):
        w = synth.tiny(batch=1, n_tokens=n_tokens, wid=wid, **specs[si])
        toks = [synth.new_token(w, s) for s in range(n_in)]
        qs = [synth.query(w, 1000 + s) for s in range(n_in)]
        K, V = synth.kv_all(w)
        inputs[wid] = dict(w=w, toks=toks, qs=qs, K=K, V=V, Kd=dev(K), Vd=dev(V),
                           kd=dev(np.stack([t[0] for t in toks])), vd=dev(np.stack([t[1] for t in toks])),
                           qd=dev(np.stack(qs)))
        return w

    wid = 700 + 50 * seed
    for si in range(len(specs)):
        w0 = sequence(si, wid, 500); wid += 1
        cfg = B.make_config(w0, max_tokens=cap)
        pool = make_pool(cfg, 128, 2 * (cap // 128 + 2), seed=seed + si)
        for k in range(2):
            w = w0
            if k == 1:
                w = sequence(si, wid, 300 + 64 * seed); wid += 1
            gc = B.InnerQCache(cfg, pool=pool)
            gc.ensure_pages(w.n_tokens)
            gc.innerq_quantize_prefill(inputs[w.wid]["Kd"], inputs[w.wid]["Vd"])
            slots.append(dict(wid=w.wid, gc=gc, step=0, nq=0, si=si))
    # sequences that restarts will switch to, made (and copied to the device) up front
    spare = []
    for k in range(6):
        si = k % len(specs)
        w = sequence(si, wid, 200 + 90 * k); wid += 1
        spare.append(w.wid)
    torch.cuda.synchronize()
    ops = []
    for it in range(320):
        i = int(rng.integers(len(slots)))
        s = slots[i]
        op = str(rng.choice(["append", "decode", "plain", "multi", "restart"], p=[.5, .3, .05, .1, .05]))
        if op == "append":
            if s["step"] >= n_in:
                continue
            ops.append((op, i, s["wid"], s["step"], 0)); s["step"] += 1
        elif op == "restart":
            cand = [x for x in spare if inputs[x]["w"].group == specs[s["si"]]["group"]]
            if not cand:
                continue
            spare.remove(cand[0])
            s.update(wid=cand[0], step=0, nq=0)
            ops.append((op, i, cand[0], 0, 0))
        elif op == "multi":
            n_q = int(rng.integers(2, 5))
            ops.append((op, i, s["wid"], s["nq"] % (n_in - 4), n_q)); s["nq"] += n_q
        else:
            ops.append((op, i, s["wid"], s["nq"] % n_in, 0)); s["nq"] += 1
    outs = []
    for op, i, w_id, j, n_q in ops:                # nothing here waits for the GPU
        gc, x = slots[i]["gc"], inputs[w_id]
        if op == "append":
            gc.ensure_pages(gc.n_tokens + 1)
            gc.innerq_append_token(x["kd"][j], x["vd"][j])
            outs.append(None)
        elif op == "restart":
            gc.release_to_pool()
            gc.ensure_pages(x["w"].n_tokens)
            gc.innerq_quantize_prefill(x["Kd"], x["Vd"])
            outs.append(None)
        elif op == "multi":
            outs.append(gc.innerq_decode_attention_multi(x["qd"][j:j + n_q].transpose(0, 1).contiguous()))
        else:
            gc.innerq_set_decode_options(0, 1 if op == "plain" else 0)
            outs.append(gc.innerq_decode_attention(x["qd"][j]))
            gc.innerq_set_decode_options(0, 0)
    torch.cuda.synchronize()
    ocs = {}

    def oracle_for(i, w_id):
        x = inputs[w_id]
        oc = O.from_workload(x["w"], max_tokens=cap)
        oc.prefill(x["K"], x["V"])
        ocs[i] = oc

    started = set()
    for (op, i, w_id, j, n_q), out in zip(ops, outs):
        if i not in started:                        # the sequence the cache was created with
            started.add(i)
            if op != "restart":
                oracle_for(i, w_id)
        x = inputs[w_id]
        if op == "restart":
            oracle_for(i, w_id)
        elif op == "append":
            ocs[i].append(*x["toks"][j])
        elif op == "multi":
            P.assert_outputs_close(out.cpu().numpy(), ocs[i].decode_multi(np.stack(x["qs"][j:j + n_q], axis=1)), f"multi, cache {i}")
        else:
            P.assert_outputs_close(out.cpu().numpy(), ocs[i].decode(x["qs"][j]), f"{op}, cache {i}")
    for i, oc in ocs.items():
        gc, w = slots[i]["gc"], inputs[slots[i]["wid"]]["w"]
        assert gc.n_tokens == oc.N and gc.innerq_read_device_error() == 0
        assert gc.pages_assigned == gc.innerq_cache_pages_for(gc.n_tokens)
        P.assert_export_equal(gc.innerq_cache_export(), oc.export(), w.grouping, w.group,
                              k_hybrid=w.k_mode == O.HYBRID, v_hybrid=w.v_mode == O.HYBRID)


def test_paged_table_longer_than_the_kernel_parameter_takes():
    # a single-cache launch passes up to 512 page indices in its parameter space; a cache with more pages makes the
    # same kernel read the table from the cache buffer (as batched launches always do)
    w = synth.tiny(batch=1, n_kv_heads=1, n_q_heads=2, n_tokens=66100, group=32)
    oc, gc = paged_pair(w, 128, 66100 + 140, seed=4)
    assert gc.pages_assigned > 512
    check_decode(w, oc, gc, variants=(0,), splits=(0, 5))
    steps(w, oc, gc, 0, 130, check_every=43, variants=(0,))
    P.assert_export_equal(gc.innerq_cache_export(), oc.export(), O.INNER, 32)
