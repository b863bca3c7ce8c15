#!/usr/bin/env python
"""Benchmark of the InnerQ decode path on B200.

A "step" is one pass of the whole hot path over one batch of synthetic input: innerq_append_token
(one new fp16 token per KV head, quantise-on-evict) followed by innerq_decode_attention over the
whole packed cache.  The default workload is the 7B-class MHA configuration (32 heads, head_dim
128, batch 1, 32768 tokens of context, 2-bit, group 32, sink 4, recent 128).

The packed cache of that workload (about 100 MB) would fit in the 126 MB L2, so the bench rotates
over several independent cache instances (same contents, different memory; total several times
the L2 size) and step i uses instance i mod R: every decode streams its cache from HBM.

Prints ONE JSON line on rank 0.  `--impl reference` times the CPU oracle instead (host cores).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2602_23200_b200 import synth  # noqa: E402

D = 128


def workload_by_name(name: str):
    """c1 .. c4 (c3_4bit / c3_2bit); a suffix "+fp16" or "+outer" selects the comparison cache of the same shape."""
    if "+" in name:
        base, variant = name.split("+", 1)
        w = workload_by_name(base)
        if variant == "fp16":
            return w.with_(name=w.name + "+fp16", grouping=synth.FP16, k_normalize=0)
        if variant == "outer":
            return w.with_(name=w.name + "+outer", grouping=synth.OUTER, k_normalize=0, k_mode=synth.ASYM, v_mode=synth.ASYM)
        raise SystemExit(f"unknown variant {variant}")
    if name == "c1":
        return synth.config1()
    if name == "c2":
        return synth.config2()
    if name == "c3_4bit":
        return synth.config3(4)
    if name == "c3_2bit":
        return synth.config3(2)
    if name == "c4":
        return synth.config4()
    raise SystemExit(f"unknown workload {name}")


def payload_bytes(w):
    """(bytes per quantised K token, bytes per quantised V token) of one unit, dense zero-points."""
    def row(bits, mode):
        return 16 * bits + (D // w.group) * (2 if mode == synth.SYM else 4)

    def blk(bits, mode):
        return 16 * bits + D * (2 if mode == synth.SYM else 4) / w.group
    if w.grouping == synth.FP16:
        return 2 * D, 2 * D
    if w.grouping == synth.INNER:
        return row(w.k_bits, w.k_mode), blk(w.v_bits, w.v_mode)
    return blk(w.k_bits, synth.ASYM), row(w.v_bits, synth.ASYM)


def decode_algorithmic_bytes(w, N, sym_frac_k=0.0, sym_frac_v=0.0):
    """Bytes one decode call must move: packed codes, scale/zero pairs, fp16 windows, q, out, norm.

    Returns (dense, minimal): `dense` counts the zero-point of every group (they are stored dense);
    `minimal` leaves out the zero-points of symmetric groups, which the result does not depend on."""
    U = w.n_units
    ws, wr, G = w.w_sink, w.w_recent, w.group
    if w.grouping == synth.FP16:
        b = U * N * 2 * D * 2 + 2 * w.batch * w.n_q_heads * D * 2
        return b, b
    mid = max(0, N - ws - wr)
    row_q, blk_q = mid, (mid // G) * G
    n_qk, n_qv = (row_q, blk_q) if w.grouping == synth.INNER else (blk_q, row_q)
    kb, vb = payload_bytes(w)
    n_sink = min(N, ws)
    per_unit = n_qk * kb + n_qv * vb + (N - n_qk) * 2 * D + (N - n_qv) * 2 * D
    extra = 2 * w.batch * w.n_q_heads * D * 2 + (U * D * 4 if w.k_normalize else 0)
    dense = U * per_unit + extra
    k_groups = n_qk * (D // G) if w.grouping == synth.INNER else (n_qk // G) * D
    v_groups = (n_qv // G) * D if w.grouping == synth.INNER else n_qv * (D // G)
    k_has_z = (w.k_mode != synth.SYM) or w.grouping == synth.OUTER
    v_has_z = (w.v_mode != synth.SYM) or w.grouping == synth.OUTER
    minimal = dense - U * 2 * (k_groups * sym_frac_k * k_has_z + v_groups * sym_frac_v * v_has_z)
    del n_sink
    return float(dense), float(minimal)


def stored_counters(workload: str):
    """Counters of one decode launch of `workload` from the committed ncu summary (profiles/decode_counters.json)."""
    try:
        with open(os.path.join(ROOT, "profiles", "decode_counters.json")) as f:
            return json.load(f).get(workload)
    except Exception:
        return None


def pipe_roofs_gbs(counters, bytes_per_decode, sm_mhz):
    """Second roofs of the packed decode kernel from its measured instruction counts.

    A sub-partition issues at most one warp instruction per cycle, its 16-lane ALU pipe takes one warp instruction
    per 2 cycles and its tensor pipe one m16n8k16 MMA per 8 cycles (measured with a stand-alone loop on this GPU).
    The time each of the three needs for the launch's instructions, spread evenly over 148 SMs x 4 sub-partitions at
    the sampled SM clock, turns the launch's algorithmic bytes into a roof in GB/s; the lowest is returned first."""
    if not counters:
        return None
    per_s = 148 * 4 * (sm_mhz or 1965.0) * 1e6
    t = {"issue": counters["warp_instructions"] / per_s, "alu_pipe": 2.0 * counters["alu_pipe"] / per_s,
         "tensor_pipe": 8.0 * counters["tensor_pipe"] / per_s}
    roofs = {k: bytes_per_decode / v / 1e9 for k, v in t.items()}
    low = min(roofs, key=roofs.get)
    return {"lowest": low, "gbs": roofs[low], "all_gbs": roofs}


class ClockSampler(threading.Thread):
    """Samples SM clocks and clock-event (throttle) reasons through NVML while the timed region runs.

    Read-only queries; nothing about the GPU is changed."""
    REASONS = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40, "sw_power_cap": 0x4}

    def __init__(self, index: int, period_s: float = 0.002):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.sm, self.mem, self.mask, self.sm_max = [], [], 0, None
        self._stop_evt = threading.Event()
        self._h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def run(self):
        if self._h is None:
            return
        nv = self._nv
        while not self._stop_evt.is_set():
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                self.mem.append(float(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_MEM)))
                self.mask |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
            except Exception:
                try:
                    self.mask |= int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                except Exception:
                    pass
            self._stop_evt.wait(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        reasons = [n for n, bit in self.REASONS.items() if self.mask & bit]
        return {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_max_mhz": self.sm_max,
                "mem_mhz": float(np.median(self.mem)) if self.mem else None, "reasons": reasons, "samples": len(self.sm)}


def measured_peak_gbs():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def stored_traffic(workload: str):
    """DRAM bytes (read + written) per decode launch from the committed ncu summary, if any."""
    c = stored_counters(workload)
    return c["dram_read_bytes"] + c["dram_write_bytes"] if c else None


# ------------------------------------------------------------------------------------- oracle legs
def oracle_steps(w, n_steps, units=None):
    """Times the CPU oracle on `n_steps` steps (append + decode).  Returns (seconds per step, bytes per step, cores)."""
    from oracle import innerq_oracle as O
    sub = w if units is None else w.with_(batch=1, n_q_heads=units * w.q_per_kv, n_kv_heads=units)
    K, V = synth.kv_all(sub)
    oc = O.from_workload(sub, max_tokens=sub.n_tokens + n_steps + 8)
    oc.prefill(K, V)
    del K, V
    times, nbytes = [], []
    for step in range(n_steps):
        k1, v1 = synth.new_token(sub, step)
        q = synth.query(sub, step)
        t0 = time.perf_counter()
        oc.append(k1, v1)
        oc.decode(q)
        times.append(time.perf_counter() - t0)
        nbytes.append(decode_algorithmic_bytes(sub, oc.N)[0])
    extra = {}
    try:
        from threadpoolctl import threadpool_info, threadpool_limits
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        with threadpool_limits(limits=1):          # one more step on a single thread
            k1, v1 = synth.new_token(sub, n_steps)
            q = synth.query(sub, n_steps)
            t0 = time.perf_counter()
            oc.append(k1, v1)
            oc.decode(q)
            extra["single_thread_s_per_step"] = time.perf_counter() - t0
    except Exception:
        cores = 1
    if sub.grouping != synth.FP16:
        # hybrid groups whose two candidates' L1 errors differ by less than 1e-4 relative: either mask is right there
        e = oc.export()
        n_cont = n_all = 0
        for name, mode in (("k", sub.k_mode), ("v", sub.v_mode)):
            if mode == synth.HYBRID:
                ea, es = e[f"{name}_err_asym"], e[f"{name}_err_sym"]
                n_cont += int((np.abs(ea - es) <= 1e-4 * np.maximum(ea, es)).sum())
                n_all += int(ea.size)
        extra["contested_hybrid_groups"] = n_cont
        extra["hybrid_groups"] = n_all
    return float(np.mean(times)), float(np.mean(nbytes)), cores, extra


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    units = min(w.n_units, 4)
    for _ in range(args.warmup and 1):
        pass
    t, b, cores, _ = oracle_steps(w, max(1, min(args.steps, 8)), units=units)
    gbs = b / t / 1e9
    line = {"impl": "reference", "metric": "decode_step_algorithmic_hbm_gbs", "value": gbs, "unit": "GB/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3,
            "us_per_step": t * 1e6 * (w.n_units / units), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(w, args),
            "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": cores, "kind": "oracle",
                             "sample": f"{units} of {w.n_units} KV heads, {max(1, min(args.steps, 8))} steps of append+decode"},
            "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def config_dict(w, args):
    return {"workload": w.name, "batch": w.batch, "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads,
            "head_dim": w.head_dim, "context": w.n_tokens, "k_bits": w.k_bits, "v_bits": w.v_bits, "group": w.group,
            "w_sink": w.w_sink, "w_recent": w.w_recent, "grouping": ["inner", "outer", "fp16"][w.grouping],
            "step": "innerq_append_token + innerq_decode_attention",
            "l2": f"rotating {args.instances} cache instances (> L2) so every decode streams from HBM"}


def max_over_ranks(value: float, device="cpu") -> float:
    """Maximum of a per-rank time over all ranks (each rank times its own replica on the device)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbs(bytes_per_step_per_rank: float, seconds_per_step: float, world: int) -> float:
    """Weak scaling: every rank runs its own batch of sequences; no data-path collective exists on this path."""
    return world * bytes_per_step_per_rank / seconds_per_step / 1e9


# ------------------------------------------------------------------------------------- CUDA arm
def run_ours(args, w):
    import torch
    import torch.distributed as dist
    from paper_2602_23200_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    R, Kst, W = args.instances, args.steps, max(args.warmup, 3)
    total_steps = W + Kst
    e2e_steps = max(4, min(Kst, 32))
    split_steps = 2 * R * w.group if w.grouping != synth.FP16 else 0     # extra steps timed one by one (below)
    cfg = B.make_config(w, max_tokens=w.n_tokens + (total_steps + e2e_steps + split_steps) // R + 16)
    Kh, Vh = synth.kv_all(w)
    Kd, Vd = torch.from_numpy(Kh).cuda(), torch.from_numpy(Vh).cuda()
    caches = []
    for _ in range(R):
        c = B.InnerQCache(cfg)
        c.innerq_quantize_prefill(Kd, Vd)
        if args.splits or args.variant:
            c.innerq_set_decode_options(args.splits, args.variant)
        caches.append(c)
    # fraction of symmetric groups (their zero-points are not needed by the result)
    ex = caches[0].innerq_cache_export(codes=False)
    sym_k = float(1.0 - ((ex["k_scale"] & 0x8000) != 0).mean()) if "k_scale" in ex and ex["k_scale"].size else 0.0
    sym_v = float(1.0 - ((ex["v_scale"] & 0x8000) != 0).mean()) if "v_scale" in ex and ex["v_scale"].size else 0.0
    # information only: how far the quantised cache moves the attention output away from the unquantised one
    # (relative L2 over all heads, same q), measured against the library's fp16 cache of the same inputs
    rel_l2 = None
    if w.grouping != synth.FP16:
        wf = w.with_(grouping=synth.FP16, k_normalize=0)
        ref_cache = B.InnerQCache(B.make_config(wf, max_tokens=w.n_tokens + 8))
        ref_cache.innerq_quantize_prefill(Kd, Vd)
        q0 = torch.from_numpy(synth.query(w, 0)).cuda()
        o_ref = ref_cache.innerq_decode_attention(q0).float()
        o_q = caches[0].innerq_decode_attention(q0).float()
        rel_l2 = float(((o_q - o_ref).norm() / o_ref.norm()).item())
        ref_cache.close()
        del ref_cache, o_ref, o_q
    # sequences of different lengths, one cache object each, decoded by one batched call (information; needs a batch)
    ragged_sets, ragged_lengths = [], []
    if w.batch > 1 and w.grouping != synth.FP16 and args.ragged:
        fracs = [1.0, 0.125, 0.5, 0.25, 0.75, 1.0, 0.375, 0.625]
        ragged_lengths = [max(w.w_sink + w.w_recent + w.group, int(w.n_tokens * fracs[i % len(fracs)])) for i in range(w.batch)]
        w1 = w.with_(batch=1)
        cfg1 = B.make_config(w1, max_tokens=w.n_tokens + 8)
        per_set = sum(ragged_lengths) * w.n_kv_heads * sum(payload_bytes(w))
        for _ in range(max(2, min(6, int(400e6 // max(per_set, 1)) + 1))):
            cs = []
            for i, n_i in enumerate(ragged_lengths):
                c = B.InnerQCache(cfg1)
                c.innerq_quantize_prefill(Kd[i:i + 1, :, :n_i].contiguous(), Vd[i:i + 1, :, :n_i].contiguous())
                cs.append(c)
            ragged_sets.append(cs)
    # the same caches with their packed records in pages of a shared pool, pages handed out in a shuffled order
    # (information: what the page table costs the decode kernel)
    paged_caches = []
    if args.paged and w.grouping != synth.FP16:
        per_cache = -(-cfg.max_tokens // args.paged) + 1
        order = np.random.default_rng(5).permutation(R * per_cache)
        pool = B.PagePool(cfg, args.paged, R * per_cache, order=order)
        for _ in range(R):
            c = B.InnerQCache(cfg, pool=pool)
            c.ensure_pages(w.n_tokens)
            c.innerq_quantize_prefill(Kd, Vd)
            paged_caches.append(c)
    del Kd, Vd, Kh, Vh, ex
    torch.cuda.empty_cache()

    n_in = total_steps + e2e_steps + split_steps
    toks = [synth.new_token(w, s) for s in range(n_in)]
    qs = [synth.query(w, s) for s in range(n_in)]
    k_new = torch.from_numpy(np.stack([t[0] for t in toks])).cuda()
    v_new = torch.from_numpy(np.stack([t[1] for t in toks])).cuda()
    q_all = torch.from_numpy(np.stack(qs)).cuda()
    out = torch.empty_like(q_all[0])
    stream = torch.cuda.current_stream()

    def step(i):
        c = caches[i % R]
        c.innerq_append_token(k_new[i], v_new[i])
        c.innerq_decode_attention(q_all[i], out)
        return c

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(W):
        step(i)
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.15)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # The decode kernel is bracketed by its own events on every 8th step only: an event between append and decode
    # keeps the decode from being launched as a programmatic dependent of the append, so the other steps run the
    # way a serving loop would.  The bracketed decodes are the ones the roofline figure is computed from.
    ev_every = 8
    dec_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range((Kst + ev_every - 1) // ev_every)]
    barrier()
    ev0.record(stream)
    for j in range(Kst):
        i = W + j
        c = caches[i % R]
        c.innerq_append_token(k_new[i], v_new[i])
        if j % ev_every == 0:
            dec_ev[j // ev_every][0].record(stream)
            c.innerq_decode_attention(q_all[i], out)
            dec_ev[j // ev_every][1].record(stream)
        else:
            c.innerq_decode_attention(q_all[i], out)
    ev1.record(stream)
    barrier()
    clocks = sampler.stop()
    # bookkeeping outside the timed region: launches and bytes per step follow from N alone
    launches = Kst * (caches[0].innerq_last_launch_count(1) + caches[0].innerq_last_launch_count(2))
    bytes_dense = bytes_min = 0.0
    n_now = [w.n_tokens + (W + Kst - 1 - r) // R + 1 for r in range(R)]       # tokens per cache after the loop
    for j in range(Kst):
        i = W + j
        n_step = w.n_tokens + i // R + 1
        bd, bm = decode_algorithmic_bytes(w, n_step, sym_k, sym_v)
        bytes_dense += bd
        bytes_min += bm
    assert all(caches[r].n_tokens == n_now[r] for r in range(R))
    ms_total = ev0.elapsed_time(ev1)
    dec_ms = [a.elapsed_time(b) for a, b in dec_ev]
    ms_total = max_over_ranks(ms_total, "cuda")
    ms_step = ms_total / Kst
    value_gbs = whole_job_gbs(bytes_min / Kst, ms_step * 1e-3, world)

    # end to end: host buffers in, host buffer out, copies inside the timed region
    kh = torch.from_numpy(np.stack([t[0] for t in toks])).pin_memory()
    vh = torch.from_numpy(np.stack([t[1] for t in toks])).pin_memory()
    qh = torch.from_numpy(np.stack(qs)).pin_memory()
    oh = torch.empty_like(qh[0]).pin_memory()

    def e2e_step(i):
        # the C-ABI call with host buffers: three host -> device copies, append, decode, device -> host copy
        c = caches[i % R]
        c.innerq_decode_step_host(kh[i], vh[i], qh[i], oh)
        torch.cuda.synchronize()
        return c

    base = total_steps
    e2e_step(base)
    barrier()
    t0 = time.perf_counter()
    e2e_bytes = 0.0
    for j in range(1, e2e_steps):
        c = e2e_step(base + j)
        e2e_bytes += decode_algorithmic_bytes(w, c.n_tokens, sym_k, sym_v)[1]
    torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / (e2e_steps - 1)
    e2e_s = max_over_ranks(e2e_s, "cuda")
    e2e_gbs = whole_job_gbs(e2e_bytes / (e2e_steps - 1), e2e_s, world)
    # decode kernel alone, launches back to back (no host work between them), same rotation over instances
    b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    nb = max(16, min(Kst, 64))
    barrier()
    b0.record(stream)
    for i in range(nb):
        caches[i % R].innerq_decode_attention(q_all[i % len(qs)], out)
    b1.record(stream)
    torch.cuda.synchronize()
    b2b_us = b0.elapsed_time(b1) / nb * 1e3
    paged = None
    if paged_caches:
        for c in paged_caches:
            c.innerq_decode_attention(q_all[0], out)
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        p0.record(stream)
        for i in range(nb):
            paged_caches[i % R].innerq_decode_attention(q_all[i % len(qs)], out)
        p1.record(stream)
        torch.cuda.synchronize()
        paged = {"page_tokens": args.paged, "pages_per_cache": paged_caches[0].pages_assigned,
                 "page_bytes": pool.page_bytes, "us_per_decode_back_to_back": p0.elapsed_time(p1) / nb * 1e3,
                 "contiguous_us_per_decode_back_to_back": b2b_us}
    # the append kernel alone, each call between its own events (extra tokens beyond the timed steps)
    app_n = 16
    app_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(app_n)]
    for j in range(app_n):
        i = total_steps + e2e_steps + split_steps + j
        app_ev[j][0].record(stream)
        caches[j % R].innerq_append_token(k_new[i % n_in], v_new[i % n_in])
        app_ev[j][1].record(stream)
    torch.cuda.synchronize()
    append_us = float(np.median([a.elapsed_time(b) for a, b in app_ev])) * 1e3
    # several query tokens per sequence in one call (causal among the newest n_q tokens), back to back like the above
    multi = None
    if args.n_q > 1 and w.grouping != synth.FP16:
        qm = torch.stack([q_all[i % len(qs)] for i in range(args.n_q)], dim=1).contiguous()     # [B, n_q, Hq, D]
        om = torch.empty_like(qm)
        for i in range(R):
            caches[i].innerq_decode_attention_multi(qm, om)
        m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        m0.record(stream)
        for i in range(nb):
            caches[i % R].innerq_decode_attention_multi(qm, om)
        m1.record(stream)
        torch.cuda.synchronize()
        multi_us = m0.elapsed_time(m1) / nb * 1e3
        multi = {"n_q": args.n_q, "us_per_call_back_to_back": multi_us, "us_per_query_token": multi_us / args.n_q,
                 "launches_per_call": caches[0].innerq_last_launch_count(2),
                 "single_query_us_back_to_back": b2b_us}
    ragged = None
    if ragged_sets:
        qr = q_all[0].reshape(w.batch, 1, w.n_q_heads, w.head_dim).contiguous()
        outr = torch.empty_like(qr)
        for cs in ragged_sets:
            B.innerq_decode_attention_batched(cs, qr, outr)
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        r0.record(stream)
        for i in range(nb):
            B.innerq_decode_attention_batched(ragged_sets[i % len(ragged_sets)], qr, outr)
        r1.record(stream)
        torch.cuda.synchronize()
        ragged_us = r0.elapsed_time(r1) / nb * 1e3
        tok = sum(ragged_lengths)
        ragged = {"lengths": ragged_lengths, "us_per_call_back_to_back": ragged_us,
                  "tokens_per_call": tok * w.n_kv_heads,
                  "us_if_time_scaled_with_tokens": b2b_us * tok / (w.batch * w.n_tokens),
                  "cache_sets_rotated": len(ragged_sets)}
        for cs in ragged_sets:
            for c in cs:
                c.close()
    # steps timed one by one (events around append + decode): those on which a value group (inner grouping) or a key
    # group (outer grouping) of G tokens is quantised, against the others
    step_split = None
    if split_steps:
        base2 = total_steps + e2e_steps
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(split_steps)]
        evict = []
        for j in range(split_steps):
            i = base2 + j
            c = caches[i % R]
            n_before = c.n_tokens
            evs[j][0].record(stream)
            c.innerq_append_token(k_new[i], v_new[i])
            c.innerq_decode_attention(q_all[i], out)
            evs[j][1].record(stream)
            mid0, mid1 = n_before - w.w_sink - w.w_recent, n_before + 1 - w.w_sink - w.w_recent
            evict.append(mid1 > 0 and mid1 // w.group > max(mid0, 0) // w.group)
        torch.cuda.synchronize()
        t_us = np.array([a_.elapsed_time(b_) * 1e3 for a_, b_ in evs])
        ev_mask = np.array(evict)
        step_split = {"steps": split_steps, "group_eviction_steps": int(ev_mask.sum()),
                      "us_median_group_eviction": float(np.median(t_us[ev_mask])) if ev_mask.any() else None,
                      "us_median_other": float(np.median(t_us[~ev_mask])) if (~ev_mask).any() else None}
    h2d = (kh[0].numel() + vh[0].numel() + qh[0].numel()) * 2
    d2h = oh.numel() * 2

    if rank == 0:
        peak, which = measured_peak_gbs()
        dec_us = float(np.mean(dec_ms)) * 1e3
        achieved = (bytes_min / Kst) / (dec_us * 1e-6) / 1e9      # bytes per decode vary by < 0.1 % over the steps
        line = {
            "metric": "decode_step_algorithmic_hbm_gbs", "value": value_gbs, "unit": "GB/s", "n_gpus": world,
            "steps": Kst, "warmup": W, "ms_per_step": ms_step, "us_per_step": ms_step * 1e3,
            "us_per_decode": dec_us, "us_per_decode_median": float(np.median(dec_ms)) * 1e3,
            "us_per_decode_min": float(np.min(dec_ms)) * 1e3, "us_per_decode_back_to_back": b2b_us,
            "us_per_append_median": append_us,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": config_dict(w, args),
            "bytes_per_decode": {"dense_zero_points": bytes_dense / Kst, "minimal": bytes_min / Kst,
                                 "sym_group_fraction": {"k": sym_k, "v": sym_v}},
            "info": {"rel_l2_vs_fp16_cache_attention": rel_l2},
            "second_roof": pipe_roofs_gbs(stored_counters(w.name), bytes_min / Kst, clocks.get("sm_mhz")),
            "step_us_by_kind": step_split, "multi_query": multi, "ragged_batch": ragged, "paged_cache": paged,
            "pct_of_nominal_8TBs": 100.0 * achieved / 8000.0,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_source": which, "traffic": stored_traffic(w.name),
                         "note": "achieved is from decodes bracketed by their own events (every 8th step), which "
                                 "cannot overlap their neighbours; in the timed loop consecutive kernels overlap "
                                 "(a whole step, append included, takes us_per_step: frac_of_step); back to back "
                                 "the decode kernel averages us_per_decode_back_to_back (time per decode of a chain "
                                 "of launches over rotating cache instances, in which the next launch's CTAs fill "
                                 "the slots the current one leaves idle: a rate, not one launch's duration)",
                         "frac_of_step": value_gbs / world / peak,
                         "achieved_back_to_back": (bytes_min / Kst) / (b2b_us * 1e-6) / 1e9,
                         "frac_back_to_back": (bytes_min / Kst) / (b2b_us * 1e-6) / 1e9 / peak,
                         "kernel": "innerq_decode_attention (split + merge)"},
            "e2e": {"value": e2e_gbs, "unit": "GB/s", "us_per_step": e2e_s * 1e6, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h},
            "gpu_launches": launches, "clocks": clocks,
        }
        if not args.no_cpu_baseline and world == 1:
            units = min(w.n_units, 4)
            t, b, cores, extra = oracle_steps(w, 3, units=units)
            line["cpu_baseline"] = {"value": b / t / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
                                    "us_per_step_full_workload": t * 1e6 * (w.n_units / units),
                                    "sample": f"{units} of {w.n_units} KV heads, 3 steps of append+decode"}
            if "single_thread_s_per_step" in extra:
                line["cpu_baseline"]["single_thread_value"] = b / extra["single_thread_s_per_step"] / 1e9
            if "hybrid_groups" in extra:
                line["info"]["contested_hybrid_groups_in_sample"] = [extra["contested_hybrid_groups"], extra["hybrid_groups"]]
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1024)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--instances", type=int, default=4, help="cache instances rotated to defeat L2 residency")
    ap.add_argument("--splits", type=int, default=0)
    ap.add_argument("--variant", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--paged", type=int, default=1024, help="page size in tokens of the paged-cache leg (0: skip it)")
    ap.add_argument("--ragged", type=int, default=1, help="1: also time a batched decode over sequences of mixed lengths")
    ap.add_argument("--n-q", type=int, default=4, help="query tokens per call of the multi-query leg (0/1: skip it)")
    args = ap.parse_args()
    w = workload_by_name(args.workload)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
