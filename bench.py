#!/usr/bin/env python
"""Benchmark of the InnerQ decode path on B200.

A "step" is one pass of the whole hot path over one batch of synthetic input: innerq_append_token
(one new fp16 token per KV head, quantise-on-evict) followed by innerq_decode_attention over the
whole packed cache.  The default workload is the 7B-class MHA configuration (32 heads, head_dim
128, batch 1, 32768 tokens of context, 2-bit, group 32, sink 4, recent 128).

The packed cache of that workload (about 100 MB) would fit in the 126 MB L2, so the bench rotates
over several independent cache instances (same contents, different memory; total several times
the L2 size) and step i uses instance i mod R: every decode streams its cache from HBM.

What is timed (all with CUDA events on the launching stream, after untimed warm steps that run
straight into the timed ones):
  * `value`, `ms_per_step`: EXACTLY --steps steps of append + decode between two events;
  * `us_per_step_fixed_leg`: the same loop over a fixed number of steps, whatever --steps says;
  * `roofline`: the decode kernel alone, 48 launches each between its own events, MEDIAN;
  * `us_per_decode_back_to_back`: a chain of decode launches;
  * `e2e`: the host-buffer entry point, one step at a time with a synchronisation per step;
  * `per_config`: the long-context GQA workload (decode alone / chained / step and the full prefill
    quantisation) and the batch-16 GQA workload at 4 and 2 bits, same legs.

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
    """c1 .. c4 (c3_4bit / c3_2bit), c5_b<bits>_g<group>_<hybrid|asym|sym|literal> (sweep on the config-3 shape);
    a suffix "+fp16" or "+outer" selects the comparison cache of the same shape, "+k<K>v<V>" (e.g. c2+k3v3) other
    code widths and "+k<K>v<V>sym" those widths in all-symmetric mode (the paper's Base preset is +k3v3sym)."""
    if "+" in name:
        base, variant = name.split("+", 1)
        w = workload_by_name(base)
        if len(variant) in (4, 7) and variant[0] == "k" and variant[2] == "v" and variant[1] in "234" and variant[3] in "234" \
                and variant[4:] in ("", "sym"):
            kw = dict(name=w.name + "+" + variant, k_bits=int(variant[1]), v_bits=int(variant[3]))
            if variant[4:] == "sym":
                kw.update(k_mode=synth.SYM, v_mode=synth.SYM)
            return w.with_(**kw)
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
    if name.startswith("c5_"):      # sweep point on the config-3 shape: c5_b<bits>_g<group>_<hybrid|asym|sym|literal>
        try:
            _, b, g, mode = name.split("_")
            bits, group = int(b[1:]), int(g[1:])
            m = {"hybrid": synth.HYBRID, "asym": synth.ASYM, "sym": synth.SYM, "literal": synth.HYBRID}[mode]
            return synth.config5(bits, group, m, synth.INNER, 1 if mode == "literal" else 0).with_(name=name)
        except (ValueError, KeyError):
            pass
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
    per_unit = n_qk * kb + n_qv * vb + (N - n_qk) * 2 * D + (N - n_qv) * 2 * D
    extra = 2 * w.batch * w.n_q_heads * D * 2 + (U * D * 4 if w.k_normalize else 0)
    dense = U * per_unit + extra
    k_groups = n_qk * (D // G) if w.grouping == synth.INNER else (n_qk // G) * D
    v_groups = (n_qv // G) * D if w.grouping == synth.INNER else n_qv * (D // G)
    k_has_z = (w.k_mode != synth.SYM) or w.grouping == synth.OUTER
    v_has_z = (w.v_mode != synth.SYM) or w.grouping == synth.OUTER
    minimal = dense - U * 2 * (k_groups * sym_frac_k * k_has_z + v_groups * sym_frac_v * v_has_z)
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
class Legs:
    """Timed legs over a set of cache instances of one workload (rotated so that every decode streams from HBM).

    Every leg starts behind a short device-side delay (`torch.cuda._sleep`), recorded BEFORE the leg's first event,
    so that the host has its launches queued when the GPU reaches them: what the events then bracket is device time,
    the way a serving loop that runs ahead of the GPU sees it, not the host's launch latency from an idle stream."""

    def __init__(self, w, caches, k_new, v_new, q_all, out, first_step=0):
        import torch
        self.torch, self.w, self.caches, self.R = torch, w, caches, len(caches)
        self.k_new, self.v_new, self.q_all, self.out = k_new, v_new, q_all, out
        self.stream = torch.cuda.current_stream()
        self.i = first_step                 # index of the next unused (k_new, v_new, q) triple
        # the step loop passes addresses (buffers validated here once), so that the host stays ahead of the GPU
        from paper_2602_23200_b200.binding import _dev_ptr
        c = caches[0].cfg
        n = k_new.shape[0]
        self.kp = _dev_ptr(k_new, "k_new", (n, c.batch, c.n_kv_heads, c.head_dim), caches[0].device)
        self.vp = _dev_ptr(v_new, "v_new", (n, c.batch, c.n_kv_heads, c.head_dim), caches[0].device)
        self.qp = _dev_ptr(q_all, "q", (n, c.batch, c.n_q_heads, c.head_dim), caches[0].device)
        self.op = _dev_ptr(out, "out", (c.batch, c.n_q_heads, c.head_dim), caches[0].device)
        self.kv_stride, self.q_stride = k_new[0].numel() * 2, q_all[0].numel() * 2
        self.sp = int(self.stream.cuda_stream)

    def _ev(self):
        return self.torch.cuda.Event(enable_timing=True)

    def delay(self, cycles=300_000):
        self.torch.cuda._sleep(cycles)      # ~0.15 ms at 1.9 GHz; outside every timed region

    def step(self):
        i = self.i
        c = self.caches[i % self.R]
        c.innerq_append_token_ptr(self.kp + i * self.kv_stride, self.vp + i * self.kv_stride, self.sp)
        c.innerq_decode_attention_ptr(self.qp + i * self.q_stride, self.op, self.sp)
        self.i += 1
        return c

    def steps(self, n, warm=0):
        """n steps (append + decode) between two events, after `warm` untimed steps that run straight into them.
        Returns (us per step on the device, us per step the host needed to enqueue them)."""
        self.delay()
        for _ in range(warm):
            self.step()
        e0, e1 = self._ev(), self._ev()
        e0.record(self.stream)
        t0 = time.perf_counter()
        for _ in range(n):
            self.step()
        host_us = (time.perf_counter() - t0) * 1e6 / n
        e1.record(self.stream)
        self.torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / n, host_us

    def decodes_bracketed(self, n):
        """n decodes, each between its own pair of events (no overlap with its neighbours).  Returns a list of us."""
        evs = [(self._ev(), self._ev()) for _ in range(n)]
        self.delay()
        nq = len(self.q_all)
        for j in range(4):                                      # untimed, so that the first bracket is not the coldest
            self.caches[j % self.R].innerq_decode_attention_ptr(self.qp + (j % nq) * self.q_stride, self.op, self.sp)
        # Event timestamps advance in steps of about 2 us on this GPU: a spacer of random length in front of every
        # bracket keeps the brackets from all falling on the same side of a step (median and mean then tell more).
        spacer = np.random.default_rng(7).integers(0, 8000, size=n)
        for j, (a, b) in enumerate(evs):                        # calls by address: the host stays ahead of the GPU
            self.torch.cuda._sleep(int(spacer[j]))
            a.record(self.stream)
            self.caches[j % self.R].innerq_decode_attention_ptr(self.qp + (j % nq) * self.q_stride, self.op, self.sp)
            b.record(self.stream)
        self.torch.cuda.synchronize()
        return [a.elapsed_time(b) * 1e3 for a, b in evs]

    def bracket_floor(self, n=32):
        """Median us between the two events of a bracket that holds one trivial kernel (a 32-byte torch fill): what the
        bracketing itself and a kernel launch cost on this machine, for reading `us_per_decode_alone`."""
        x = self.torch.zeros(8, device=self.out.device)
        evs = [(self._ev(), self._ev()) for _ in range(n)]
        self.delay()
        for _ in range(4):
            x.fill_(1.0)
        for a, b in evs:
            a.record(self.stream)
            x.fill_(1.0)
            b.record(self.stream)
        self.torch.cuda.synchronize()
        return float(np.median([a.elapsed_time(b) * 1e3 for a, b in evs]))

    def decodes_chained(self, n, caches=None, call=None):
        """n decodes launched back to back over the rotating instances: us per decode of the chain."""
        caches = caches or self.caches
        nq = len(self.q_all)
        call = call or (lambda c, j: c.innerq_decode_attention_ptr(self.qp + (j % nq) * self.q_stride, self.op, self.sp))
        self.delay()
        for j in range(4):
            call(caches[j % len(caches)], j)
        e0, e1 = self._ev(), self._ev()
        e0.record(self.stream)
        for j in range(n):
            call(caches[j % len(caches)], j)
        e1.record(self.stream)
        self.torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / n

    def small_launches(self, nbytes, peak, n_steps=96):
        """The same legs with one CTA per SM and launch (148 / units splits per unit instead of one wave of two CTAs
        per SM): consecutive launches then share the GPU, which hides each launch's start and end behind its
        neighbours' streaming (higher step rate) and makes a launch that runs alone slower (half the warps per SM).
        The library's default stays the latency-optimal split; `innerq_set_decode_options` selects this one."""
        sp = max(1, 148 // self.w.n_units)
        for c in self.caches:
            c.innerq_set_decode_options(sp, 0)
        try:
            step, _ = self.steps(n_steps, warm=16)
            chain = self.decodes_chained(64)
            alone = float(np.median(self.decodes_bracketed(16)))
        finally:
            for c in self.caches:
                c.innerq_set_decode_options(0, 0)
        gbs = lambda us: nbytes / us / 1e3
        return {"n_splits": sp, "us_per_step": step, "us_per_decode_back_to_back": chain, "us_per_decode_alone_median": alone,
                "frac_of_measured_peak": {"step": gbs(step) / peak, "chained": gbs(chain) / peak, "alone_median": gbs(alone) / peak}}

    def sides(self, n=64):
        """us per decode in a chain for the full fused kernel, without its key-side arithmetic and without its
        value-side arithmetic (decode options 6 / 7: timing only, all bytes still streamed); None if the cache's format
        has no fused kernel."""
        from paper_2602_23200_b200.binding import InnerQError
        res = {}
        try:
            for name, variant in (("full", 2), ("without_key_side", 6), ("without_value_side", 7)):
                for c in self.caches:
                    c.innerq_set_decode_options(0, variant)
                res[name] = self.decodes_chained(n)
        except InnerQError:
            res = None
        for c in self.caches:
            c.innerq_set_decode_options(0, 0)
        return res

    def appends_bracketed(self, n):
        evs = [(self._ev(), self._ev()) for _ in range(n)]
        self.delay()
        for j, (a, b) in enumerate(evs):
            i = self.i
            a.record(self.stream)
            self.caches[i % self.R].innerq_append_token(self.k_new[i], self.v_new[i])
            b.record(self.stream)
            self.i += 1
        self.torch.cuda.synchronize()
        return [a.elapsed_time(b) * 1e3 for a, b in evs]

    def steps_one_by_one(self, n):
        """n steps, each between its own events; returns (us list, mask of the steps that evict a group of G tokens)."""
        w = self.w
        evs = [(self._ev(), self._ev()) for _ in range(n)]
        evict = []
        self.delay()
        for a, b in evs:
            n_before = self.caches[self.i % self.R].n_tokens
            a.record(self.stream)
            self.step()
            b.record(self.stream)
            mid0, mid1 = n_before - w.w_sink - w.w_recent, n_before + 1 - w.w_sink - w.w_recent
            evict.append(mid1 > 0 and mid1 // w.group > max(mid0, 0) // w.group)
        self.torch.cuda.synchronize()
        return np.array([a.elapsed_time(b) * 1e3 for a, b in evs]), np.array(evict)


def stats(us):
    us = np.asarray(us, dtype=np.float64)
    return {"median": float(np.median(us)), "min": float(us.min()), "mean": float(us.mean()), "n": int(us.size)}


def make_inputs(w, n):
    import torch
    toks = [synth.new_token(w, s) for s in range(n)]
    qs = [synth.query(w, s) for s in range(n)]
    kh, vh, qh = np.stack([t[0] for t in toks]), np.stack([t[1] for t in toks]), np.stack(qs)
    return (kh, vh, qh), (torch.from_numpy(kh).cuda(), torch.from_numpy(vh).cuda(), torch.from_numpy(qh).cuda())


def kv_device(w, tiled):
    """fp16 K, V of the workload on the device.  tiled: batch entry 0 is generated and repeated over the batch
    (host generation time of the large shapes; units are independent, so timings do not depend on it)."""
    import torch
    if tiled and w.batch > 1:
        K1, V1 = synth.kv_all(w.with_(batch=1))
        Kd, Vd = torch.from_numpy(K1).cuda(), torch.from_numpy(V1).cuda()
        return Kd.expand(w.batch, -1, -1, -1).contiguous(), Vd.expand(w.batch, -1, -1, -1).contiguous()
    Kh, Vh = synth.kv_all(w)
    return torch.from_numpy(Kh).cuda(), torch.from_numpy(Vh).cuda()


def sym_fractions(cache):
    ex = cache.innerq_cache_export(codes=False)
    f = lambda a: float(1.0 - ((a & 0x8000) != 0).mean()) if a is not None and a.size else 0.0
    return f(ex.get("k_scale")), f(ex.get("v_scale"))


def prefill_algorithmic_bytes(w):
    """Bytes a prefill quantisation must move: fp16 K and V read once, the packed cache and the windows written."""
    U, N = w.n_units, w.n_tokens
    dense, _ = decode_algorithmic_bytes(w, N)
    return float(U * N * D * 2 * 2 + dense)


def measure_config(name, peak, R=2, n_steps=128):
    """One more workload for the line's `per_config` block: decode alone / chained, the step, and (c4) the prefill."""
    import torch
    from paper_2602_23200_b200 import binding as B
    w = workload_by_name(name)
    n_in = 32 + n_steps + 8 + 16 + 96
    cfg = B.make_config(w, max_tokens=w.n_tokens + n_in // R + 16)
    Kd, Vd = kv_device(w, tiled=True)
    caches = []
    pre_us = []
    for _ in range(R):
        c = B.InnerQCache(cfg)
        c.innerq_quantize_prefill(Kd, Vd)
        caches.append(c)
    res = {"config": {"batch": w.batch, "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads, "context": w.n_tokens,
                      "bits": w.k_bits, "group": w.group, "instances_rotated": R}}
    if name == "c4":
        # the full prefill quantisation of the 131072-token cache, each call between its own events
        for rep in range(4):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            caches[rep % R].innerq_quantize_prefill(Kd, Vd)
            e1.record()
            torch.cuda.synchronize()
            pre_us.append(e0.elapsed_time(e1) * 1e3)
        pb = prefill_algorithmic_bytes(w)
        med = float(np.median(pre_us[1:]))
        res["prefill"] = {"us": stats(pre_us[1:]), "algorithmic_bytes": pb, "gbs": pb / med / 1e3,
                          "frac_of_measured_peak": pb / med / 1e3 / peak, "pct_of_nominal_8TBs": pb / med / 1e3 / 80.0,
                          "launches": caches[0].innerq_last_launch_count(0)}
    sym_k, sym_v = sym_fractions(caches[0])
    del Kd, Vd
    torch.cuda.empty_cache()
    _, (k_new, v_new, q_all) = make_inputs(w, n_in)
    legs = Legs(w, caches, k_new, v_new, q_all, torch.empty_like(q_all[0]))
    nbytes = decode_algorithmic_bytes(w, w.n_tokens + 1, sym_k, sym_v)[1]
    alone = stats(legs.decodes_bracketed(32))
    chain = legs.decodes_chained(64)
    step, step_host = legs.steps(n_steps, warm=32)
    sides = legs.sides()
    small = legs.small_launches(nbytes, peak)
    gbs = lambda us: nbytes / us / 1e3
    res.update({
        "one_cta_per_sm_launches": small,
        "bytes_per_decode_minimal": nbytes, "sym_group_fraction": {"k": sym_k, "v": sym_v},
        "us_per_decode_alone": alone, "us_per_decode_chained": chain, "us_per_step": step,
        "host_us_per_step_enqueue": step_host, "us_per_decode_chained_by_side": sides,
        "frac_of_measured_peak": {"alone_median": gbs(alone["median"]) / peak, "chained": gbs(chain) / peak,
                                  "step": gbs(step) / peak},
        "pct_of_nominal_8TBs": {"alone_median": gbs(alone["median"]) / 80.0, "chained": gbs(chain) / 80.0,
                                "step": gbs(step) / 80.0},
    })
    for c in caches:
        assert c.innerq_read_device_error() == 0
        c.close()
    return res


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
    packed = w.grouping != synth.FP16
    WARM = 64                       # untimed steps that run straight into the timed region (besides the W warm-up steps)
    LEG = args.leg_steps            # the step-rate leg that does not depend on --steps
    e2e_steps = max(4, min(Kst, 32))
    split_steps = 2 * R * w.group if packed else 0           # steps timed one by one (below)
    n_in = W + WARM + Kst + 32 + LEG + e2e_steps + split_steps + 16 + 16 + 96
    cfg = B.make_config(w, max_tokens=w.n_tokens + n_in // R + 16)
    Kd, Vd = kv_device(w, tiled=False)
    caches = []
    for _ in range(R):
        c = B.InnerQCache(cfg)
        c.innerq_quantize_prefill(Kd, Vd)
        if args.splits or args.variant:
            c.innerq_set_decode_options(args.splits, args.variant)
        caches.append(c)
    sym_k, sym_v = sym_fractions(caches[0]) if packed else (0.0, 0.0)
    # information only: how far the quantised cache moves the attention output away from the unquantised one
    # (relative L2 over all heads, same q), measured against the library's fp16 cache of the same inputs
    rel_l2 = None
    if packed:
        wf = w.with_(grouping=synth.FP16, k_normalize=0)
        ref_cache = B.InnerQCache(B.make_config(wf, max_tokens=w.n_tokens + 8))
        ref_cache.innerq_quantize_prefill(Kd, Vd)
        q0 = torch.from_numpy(synth.query(w, 0)).cuda()
        o_ref = ref_cache.innerq_decode_attention(q0).float()
        o_q = caches[0].innerq_decode_attention(q0).float()
        rel_l2 = float(((o_q - o_ref).norm() / o_ref.norm()).item())
        ref_cache.close()
        del ref_cache, o_ref, o_q
    # the paper-literal symmetric variant (clipped signed range): the regime in which most groups stay symmetric
    literal_caches = []
    if packed and args.literal and w.sym_variant == 0 and (w.k_mode == synth.HYBRID or w.v_mode == synth.HYBRID):
        cfg_l = B.make_config(w.with_(sym_variant=1), max_tokens=w.n_tokens + 16)
        for _ in range(R):
            c = B.InnerQCache(cfg_l)
            c.innerq_quantize_prefill(Kd, Vd)
            literal_caches.append(c)
    # sequences of different lengths, one cache object each, decoded by one batched call (information; needs a batch)
    ragged_sets, ragged_lengths = [], []
    if w.batch > 1 and packed and args.ragged:
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
    if args.paged and packed:
        per_cache = -(-cfg.max_tokens // args.paged) + 1
        order = np.random.default_rng(5).permutation(R * per_cache)
        pool = B.PagePool(cfg, args.paged, R * per_cache, order=order)
        for _ in range(R):
            c = B.InnerQCache(cfg, pool=pool)
            c.ensure_pages(w.n_tokens)
            c.innerq_quantize_prefill(Kd, Vd)
            paged_caches.append(c)
    del Kd, Vd
    torch.cuda.empty_cache()

    (kh_np, vh_np, qh_np), (k_new, v_new, q_all) = make_inputs(w, n_in)
    out = torch.empty_like(q_all[0])
    legs = Legs(w, caches, k_new, v_new, q_all, out)
    stream = legs.stream

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- the timed region of the contract: W warm-up steps, then EXACTLY Kst steps between two events --------
    for _ in range(W):
        legs.step()
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.05)
    barrier()
    legs.delay()
    for _ in range(WARM):           # untimed; they run straight into the timed steps, so those start on a busy GPU
        legs.step()
    i_first = legs.i
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(Kst):
        legs.step()
    ev1.record(stream)
    barrier()
    ms_total = max_over_ranks(ev0.elapsed_time(ev1), "cuda")
    ms_step = ms_total / Kst
    launches = Kst * (caches[0].innerq_last_launch_count(1) + caches[0].innerq_last_launch_count(2))
    bytes_dense = bytes_min = 0.0
    for i in range(i_first, i_first + Kst):
        bd, bm = decode_algorithmic_bytes(w, w.n_tokens + i // R + 1, sym_k, sym_v)
        bytes_dense += bd
        bytes_min += bm
    bytes_dense /= Kst
    bytes_min /= Kst                 # bytes per decode vary by < 0.1 % over the whole run
    value_gbs = whole_job_gbs(bytes_min, ms_step * 1e-3, world)
    # ---- the same step loop over a fixed number of steps (does not depend on --steps) ------------------------
    leg_us, leg_host_us = legs.steps(LEG, warm=32)
    # ---- the decode kernel alone: every launch between its own events (the roofline figure), and chained -------
    alone = stats(legs.decodes_bracketed(48))
    alone["trivial_kernel_in_the_same_bracket_us"] = legs.bracket_floor()
    b2b_us = legs.decodes_chained(64)
    clocks = sampler.stop()
    assert all(c.n_tokens == w.n_tokens + (legs.i - 1 - r) // R + 1 for r, c in enumerate(caches))

    # ---- end to end: host buffers in, host buffer out, through the C-ABI call that takes host pointers --------
    kh = torch.from_numpy(kh_np).pin_memory()
    vh = torch.from_numpy(vh_np).pin_memory()
    qh = torch.from_numpy(qh_np).pin_memory()
    oh = torch.empty_like(qh[0]).pin_memory()

    def e2e_step():
        i = legs.i
        c = caches[i % R]
        c.innerq_decode_step_host(kh[i], vh[i], qh[i], oh)
        torch.cuda.synchronize()
        legs.i += 1
        return c

    e2e_step()
    barrier()
    t0 = time.perf_counter()
    e2e_bytes = 0.0
    for _ in range(1, e2e_steps):
        c = e2e_step()
        e2e_bytes += decode_algorithmic_bytes(w, c.n_tokens, sym_k, sym_v)[1]
    torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / (e2e_steps - 1)
    e2e_s = max_over_ranks(e2e_s, "cuda")
    e2e_gbs = whole_job_gbs(e2e_bytes / (e2e_steps - 1), e2e_s, world)
    h2d = (kh[0].numel() + vh[0].numel() + qh[0].numel()) * 2
    d2h = oh.numel() * 2

    # ---- information legs ----------------------------------------------------------------------------------
    paged = None
    if paged_caches:
        paged = {"page_tokens": args.paged, "pages_per_cache": paged_caches[0].pages_assigned,
                 "page_bytes": pool.page_bytes, "us_per_decode_back_to_back": legs.decodes_chained(64, caches=paged_caches),
                 "contiguous_us_per_decode_back_to_back": b2b_us}
    literal = None
    if literal_caches:
        lk, lv = sym_fractions(literal_caches[0])
        literal = {"sym_group_fraction": {"k": lk, "v": lv},
                   "bytes_per_decode_minimal": decode_algorithmic_bytes(w.with_(sym_variant=1), w.n_tokens, lk, lv)[1],
                   "us_per_decode_back_to_back": legs.decodes_chained(64, caches=literal_caches)}
        for c in literal_caches:
            c.close()
    sides = legs.sides() if packed and not (args.splits or args.variant) else None
    small = legs.small_launches(bytes_min, measured_peak_gbs()[0]) if packed and not (args.splits or args.variant) else None
    append_us = float(np.median(legs.appends_bracketed(16)))
    multi = None
    if args.n_q > 1 and packed:
        qm = torch.stack([q_all[i] for i in range(args.n_q)], dim=1).contiguous()     # [B, n_q, Hq, D]
        om = torch.empty_like(qm)
        multi_us = legs.decodes_chained(64, call=lambda c, j: c.innerq_decode_attention_multi(qm, om))
        multi = {"n_q": args.n_q, "us_per_call_back_to_back": multi_us, "us_per_query_token": multi_us / args.n_q,
                 "launches_per_call": caches[0].innerq_last_launch_count(2),
                 "single_query_us_back_to_back": b2b_us}
    ragged = None
    if ragged_sets:
        qr = q_all[0].reshape(w.batch, 1, w.n_q_heads, w.head_dim).contiguous()
        outr = torch.empty_like(qr)
        ragged_us = legs.decodes_chained(64, caches=ragged_sets,
                                         call=lambda cs, j: B.innerq_decode_attention_batched(cs, qr, outr))
        tok = sum(ragged_lengths)
        ragged = {"lengths": ragged_lengths, "us_per_call_back_to_back": ragged_us,
                  "tokens_per_call": tok * w.n_kv_heads,
                  "us_if_time_scaled_with_tokens": b2b_us * tok / (w.batch * w.n_tokens),
                  "cache_sets_rotated": len(ragged_sets)}
        for cs in ragged_sets:
            for c in cs:
                c.close()
    # steps timed one by one: those on which a value group (inner grouping) or a key group (outer grouping) of G
    # tokens is quantised, against the others
    step_split = None
    if split_steps:
        t_us, ev_mask = legs.steps_one_by_one(split_steps)
        step_split = {"steps": split_steps, "group_eviction_steps": int(ev_mask.sum()),
                      "us_median_group_eviction": float(np.median(t_us[ev_mask])) if ev_mask.any() else None,
                      "us_median_other": float(np.median(t_us[~ev_mask])) if (~ev_mask).any() else None}
    dev_err = max(c.innerq_read_device_error() for c in caches)
    for c in caches + paged_caches:
        c.close()
    del caches, paged_caches, legs
    torch.cuda.empty_cache()

    if rank == 0:
        peak, which = measured_peak_gbs()
        gbs = lambda us: bytes_min / us / 1e3
        achieved = gbs(alone["median"])
        counters = stored_counters(w.name)
        line = {
            "metric": "decode_step_algorithmic_hbm_gbs", "value": value_gbs, "unit": "GB/s", "n_gpus": world,
            "steps": Kst, "warmup": W, "ms_per_step": ms_step, "us_per_step": ms_step * 1e3,
            "us_per_step_fixed_leg": {"steps": LEG, "us": leg_us, "frac_of_measured_peak": gbs(leg_us) / peak,
                                      "host_us_per_step_enqueue": leg_host_us},
            "us_per_decode": alone["median"], "us_per_decode_alone": alone, "us_per_decode_back_to_back": b2b_us,
            "us_per_append_median": append_us, "us_per_decode_back_to_back_by_side": sides,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": config_dict(w, args),
            "bytes_per_decode": {"dense_zero_points": bytes_dense, "minimal": bytes_min,
                                 "sym_group_fraction": {"k": sym_k, "v": sym_v}},
            "info": {"rel_l2_vs_fp16_cache_attention": rel_l2, "device_error_word": dev_err,
                     "untimed_steps_before_the_timed_region": W + WARM},
            "paper_literal_sym_variant": literal,
            "second_roof": pipe_roofs_gbs(counters, bytes_min, clocks.get("sm_mhz")),
            "step_us_by_kind": step_split, "one_cta_per_sm_launches": small, "multi_query": multi, "ragged_batch": ragged, "paged_cache": paged,
            "pct_of_nominal_8TBs": {"decode_alone_median": achieved / 80.0, "decode_back_to_back": gbs(b2b_us) / 80.0,
                                    "step": value_gbs / world / 80.0},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_source": which, "traffic": stored_traffic(w.name),
                         "traffic_source": ("stored in profiles/decode_counters.json: "
                                            + str((counters or {}).get("captured_at", "ncu capture of one launch")))
                         if counters else None,
                         "note": "achieved = algorithmic bytes of one decode / MEDIAN duration of 48 decode launches "
                                 "that are each bracketed by their own events (us_per_decode_alone), so none "
                                 "overlaps its neighbours; in the step loop consecutive kernels overlap (a whole "
                                 "step, append included, takes us_per_step: frac_of_step); launched back to back "
                                 "the decode kernel averages us_per_decode_back_to_back (a rate: the next "
                                 "launch's CTAs fill the slots the current one leaves idle)",
                         "frac_of_step": value_gbs / world / peak,
                         "achieved_back_to_back": gbs(b2b_us), "frac_back_to_back": gbs(b2b_us) / peak,
                         "kernel": "innerq_decode_attention (split + merge)"},
            "e2e": {"value": e2e_gbs, "unit": "GB/s", "us_per_step": e2e_s * 1e6, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h},
            "gpu_launches": launches, "clocks": clocks,
        }
        if args.per_config and world == 1:
            line["per_config"] = {}
            for name in args.per_config.split(","):
                if name and workload_by_name(name).name != w.name:
                    line["per_config"][name] = measure_config(name, peak)
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
    ap.add_argument("--steps", type=int, default=256)
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
    ap.add_argument("--leg-steps", type=int, default=512, help="steps of the step-rate leg that does not depend on --steps")
    ap.add_argument("--literal", type=int, default=1, help="1: also report the paper-literal symmetric variant")
    ap.add_argument("--per-config", default="c4,c3_4bit,c3_2bit",
                    help="further workloads measured into the line's per_config block ('' to skip)")
    ap.add_argument("--tokens", type=int, default=0, help="context length instead of the workload's own (experiments)")
    args = ap.parse_args()
    w = workload_by_name(args.workload)
    if args.tokens > 0:
        w = w.with_(n_tokens=args.tokens, name=f"{w.name}@{args.tokens}")
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
