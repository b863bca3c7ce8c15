"""Decode latency over context length for the paper's presets (Section "Latency", Tables of dequantisation
latencies and the hybrid ablation), on the shape of one decoder layer of an 8B-class GQA model:
batch 1, 32 query heads, 8 KV heads, head_dim 128, group 32, sink 32, recent 96.

Presets: Base (3-bit symmetric K and V), Hybrid (3-bit symmetric K, 2-bit hybrid V), Small (3-bit symmetric K,
2-bit symmetric V), the 2-bit and 4-bit hybrid caches of the benchmark configurations, an outer-grouped
(per-channel K, per-token V) 2-bit cache and the unquantised fp16 cache.  The hybrid mask is decided by the data:
besides the presets on the workload's own values (whose measured asymmetric fraction is printed), the mask
ablation rows rebuild the values group by group so that 1, 10, 50 and 99 % of the value groups prefer the
asymmetric candidate (values_with_mask_density).  Key side and value side are one fused kernel here; what each side
costs is measured as the difference between the full kernel and the same kernel with that side's unpack + MMA work
left out of its streaming loop (decode variants 6 and 7 of innerq_set_decode_options, timing only), all bytes still
streamed: the second table.

    python -m paper_2602_23200_b200.latency_study [--out table.md] [--lengths 512,4096,32768]

Each cell is the time of one innerq_decode_attention call: "cold" with L2 flushed before the call (CUDA events
around the single launch, median of `--reps`), "warm" as the mean of back-to-back calls on the same cache.
"""
from __future__ import annotations

import argparse
import json
import statistics
import sys

import numpy as np

from . import synth

PRESETS = [
    # name, overrides
    ("Base K3s/V3s", dict(k_bits=3, v_bits=3, k_mode=synth.SYM, v_mode=synth.SYM)),
    ("Hybrid K3s/V2h", dict(k_bits=3, v_bits=2, k_mode=synth.SYM, v_mode=synth.HYBRID)),
    ("Small K3s/V2s", dict(k_bits=3, v_bits=2, k_mode=synth.SYM, v_mode=synth.SYM)),
    ("2-bit hybrid", dict(k_bits=2, v_bits=2)),
    ("2-bit hybrid, literal sym", dict(k_bits=2, v_bits=2, sym_variant=1)),
    ("2-bit all-asym", dict(k_bits=2, v_bits=2, k_mode=synth.ASYM, v_mode=synth.ASYM)),
    ("2-bit all-sym", dict(k_bits=2, v_bits=2, k_mode=synth.SYM, v_mode=synth.SYM)),
    ("4-bit hybrid", dict(k_bits=4, v_bits=4)),
    ("outer-grouped 2-bit", dict(k_bits=2, v_bits=2, grouping=synth.OUTER, k_normalize=0, k_mode=synth.ASYM,
                                 v_mode=synth.ASYM)),
    ("fp16", dict(grouping=synth.FP16, k_normalize=0)),
]

# The hybrid-mask ablation (Table "hybrid_ablation": the value kernel against the fraction of asymmetric groups),
# on the "Hybrid" preset.  The mask is decided by the data, so the values are built group by group to land on
# the wanted fraction: see values_with_mask_density.
MASK_DENSITIES = [0.01, 0.10, 0.50, 0.99]
MASK_PRESET = dict(k_bits=3, v_bits=2, k_mode=synth.SYM, v_mode=synth.HYBRID)


def values_with_mask_density(V, w_sink: int, G: int, density: float, seed: int = 5):
    """Copy of the fp16 values V [B, Hkv, N, D] in which a fraction `density` of the (G tokens x 1 channel) groups
    behind the sink prefers the asymmetric candidate and the rest the symmetric one.  Asymmetric groups: the
    original values shifted by +3 (far from zero-centred).  Symmetric groups: values from {-1, 0, 1} with at least
    one -1, which the 2-bit symmetric quantiser (codes -1, 0, 1 times the scale max|x|) reproduces exactly, while
    the asymmetric one (four levels between min and max) cannot hit 0 when both signs occur, and ties go to the
    symmetric candidate."""
    V = np.array(V, dtype=np.float16, copy=True)
    Bn, H, N, D = V.shape
    n_groups = max(0, (N - w_sink) // G)
    if n_groups == 0:
        return V
    body = V[:, :, w_sink:w_sink + n_groups * G].astype(np.float32).reshape(Bn, H, n_groups, G, D)
    rng = np.random.default_rng(seed)
    asym = rng.random((Bn, H, n_groups, 1, D)) < density
    sym_vals = np.where(np.abs(body) > 0.67, np.sign(body), 0.0).astype(np.float32)
    sym_vals[:, :, :, 0, :] = -1.0
    body = np.where(asym, body + 3.0, sym_vals)
    V[:, :, w_sink:w_sink + n_groups * G] = body.reshape(Bn, H, n_groups * G, D).astype(np.float16)
    return V


def layer_workload(n_tokens: int, **kw) -> synth.Workload:
    base = synth.Workload("layer8b", 21, batch=1, n_q_heads=32, n_kv_heads=8, n_tokens=n_tokens, group=32,
                          w_sink=32, w_recent=96, v_dist="student_t4", n_hashed_outliers=3, outlier_lo=10.0,
                          outlier_hi=30.0)
    return base.with_(**kw)


def _chain(cache, q, out, n: int) -> float:
    """us per call of n calls launched back to back.  The calls go by address (buffers validated by the warm-up call
    above them) and start behind a short device-side delay, so that the host's launch rate is not what is timed."""
    import torch
    qp, op, sp = q.data_ptr(), out.data_ptr(), int(torch.cuda.current_stream().cuda_stream)
    torch.cuda._sleep(400_000)
    for _ in range(4):
        cache.innerq_decode_attention_ptr(qp, op, sp)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n):
        cache.innerq_decode_attention_ptr(qp, op, sp)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / n


def time_decode(cache, q, out, flush, reps: int):
    import torch
    for _ in range(3):
        cache.innerq_decode_attention(q, out)
    torch.cuda.synchronize()
    cold = []
    for _ in range(reps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        cache.innerq_decode_attention(q, out)
        e1.record()
        torch.cuda.synchronize()
        cold.append(e0.elapsed_time(e1) * 1e3)
    return statistics.median(cold), _chain(cache, q, out, 4 * reps)


def time_sides(cache, q, out, reps: int):
    """(full, without the key side, without the value side) in us per call, back to back; None where the cache's
    format has no fused kernel."""
    from . import binding as B
    res = []
    for variant in (2, 6, 7):
        try:
            cache.innerq_set_decode_options(0, variant)
            for _ in range(3):
                cache.innerq_decode_attention(q, out)
        except B.InnerQError:
            cache.innerq_set_decode_options(0, 0)
            return None
        res.append(_chain(cache, q, out, 4 * reps))
    cache.innerq_set_decode_options(0, 0)
    return tuple(res)


def asym_fraction(cache, which: str) -> float:
    e = cache.innerq_cache_export(codes=False)
    s = e.get(which)
    if s is None or s.size == 0:
        return float("nan")
    return float(((s & 0x8000) != 0).mean())


def main(argv=None) -> int:
    ap = argparse.ArgumentParser(description=__doc__.split("\n\n")[0])
    ap.add_argument("--lengths", default="512,1024,2048,4096,8192,16384,32768")
    ap.add_argument("--reps", type=int, default=15)
    ap.add_argument("--out", default="")
    args = ap.parse_args(argv)
    import torch
    from . import binding as B

    lengths = [int(x) for x in args.lengths.split(",")]
    n_max = max(lengths)
    K, V = synth.kv_all(layer_workload(n_max))
    Kd, Vd = torch.from_numpy(K).cuda(), torch.from_numpy(V).cuda()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")      # larger than L2
    rows, records, side_rows = [], [], []
    for name, kw in PRESETS:
        cells = []
        sides = []
        frac_v = float("nan")
        for n in lengths:
            w = layer_workload(n, **kw)
            cache = B.InnerQCache(B.make_config(w, max_tokens=n + 64))
            cache.innerq_quantize_prefill(Kd[:, :, :n].contiguous(), Vd[:, :, :n].contiguous())
            q = torch.from_numpy(synth.query(w)).cuda()
            out = torch.empty_like(q)
            cold, warm = time_decode(cache, q, out, flush, args.reps)
            if cache.innerq_read_device_error() != 0:
                raise RuntimeError("a bounded wait inside the decode kernel ran out")
            if n == n_max and w.grouping == synth.INNER:
                frac_v = asym_fraction(cache, "v_scale")
            cells.append((cold, warm))
            rec = {"preset": name, "n_tokens": n, "cold_us": round(cold, 2), "warm_us": round(warm, 2)}
            if w.grouping != synth.FP16:
                sd = time_sides(cache, q, out, args.reps)
                sides.append(sd)
                if sd:
                    rec.update({"full_us": round(sd[0], 2), "without_key_side_us": round(sd[1], 2),
                                "without_value_side_us": round(sd[2], 2)})
            records.append(rec)
            cache.close()
        rows.append((name, frac_v, cells))
        if sides and all(sides):
            side_rows.append((name, sides))
        print(f"{name:28s} " + " ".join(f"{c:7.1f}/{wm:<7.1f}" for c, wm in cells), flush=True)
    base_w = layer_workload(n_max)
    for density in MASK_DENSITIES:
        name = f"Hybrid K3s/V2h, mask {100 * density:g} % wanted"
        Vm = torch.from_numpy(values_with_mask_density(V, base_w.w_sink, base_w.group, density)).cuda()
        cells = []
        frac_v = float("nan")
        for n in lengths:
            w = layer_workload(n, **MASK_PRESET)
            cache = B.InnerQCache(B.make_config(w, max_tokens=n + 64))
            cache.innerq_quantize_prefill(Kd[:, :, :n].contiguous(), Vm[:, :, :n].contiguous())
            q = torch.from_numpy(synth.query(w)).cuda()
            out = torch.empty_like(q)
            cold, warm = time_decode(cache, q, out, flush, args.reps)
            if n == n_max:
                frac_v = asym_fraction(cache, "v_scale")
            cells.append((cold, warm))
            records.append({"preset": name, "n_tokens": n, "cold_us": round(cold, 2), "warm_us": round(warm, 2)})
            cache.close()
        rows.append((name, frac_v, cells))
        print(f"{name:28s} " + " ".join(f"{c:7.1f}/{wm:<7.1f}" for c, wm in cells), flush=True)
        del Vm
    lines = ["| preset (asym fraction of V groups) | " + " | ".join(str(n) for n in lengths) + " |",
             "|---|" + "---|" * len(lengths)]
    for name, fv, cells in rows:
        tag = name if np.isnan(fv) else f"{name} ({100 * fv:.0f} %)"
        lines.append(f"| {tag} | " + " | ".join(f"{c:.1f} / {wm:.1f}" for c, wm in cells) + " |")
    table = "\n".join(lines)
    print("\nµs per decode call, cold (L2 flushed) / warm (back to back):\n" + table)
    lines = ["| preset | " + " | ".join(str(n) for n in lengths) + " |", "|---|" + "---|" * len(lengths)]
    for name, sides in side_rows:
        lines.append(f"| {name} | " + " | ".join(f"{f - nk:.1f} + {f - nv:.1f} of {f:.1f}" for f, nk, nv in sides) + " |")
    side_table = "\n".join(lines)
    print("\nµs per call, back to back: key side + value side (full minus the kernel without that side) of the full "
          "kernel's time; the rest is streaming, soft-max, metadata and fixed cost, which both sides share:\n" + side_table)
    table = table + "\n\n" + side_table
    if args.out:
        with open(args.out, "w") as f:
            f.write(table + "\n\n" + "\n".join(json.dumps(r) for r in records) + "\n")
    return 0


if __name__ == "__main__":
    sys.exit(main())
