"""The benchmark's cross-rank logic on CPU: two gloo ranks, each a replica with its own timing.
The path has no data-path collective (units are independent); ranks only agree on the slowest time."""
import os
import sys

import pytest

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 10.0 + 5.0 * rank                     # rank 1 is slower
    slowest = bench.max_over_ranks(mine, "cpu")
    out[rank] = (slowest, bench.whole_job_gbs(1e9, slowest * 1e-3, world))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_weak_scaling_value():
    world, port = 2, 29731
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 15.0                      # both ranks see the slowest replica's time
    assert abs(res[0][1] - 2 * 1e9 / 15e-3 / 1e9) < 1e-9       # whole-job throughput = ranks x per-rank bytes / time


def test_single_process_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_gbs(2e9, 1e-3, 1) == 2000.0


def test_algorithmic_bytes_follow_the_library_payload():
    # the roofline numerator: bytes per quantised token as bench.py counts them = what the C ABI says the packed
    # cache holds per token, for every mode (zero-points stored or not) and both groupings
    sys.path.insert(0, ROOT)
    import bench
    from paper_2602_23200_b200 import binding as B, synth
    for kw in (dict(), dict(k_bits=3, v_bits=2, k_mode=synth.SYM, v_mode=synth.HYBRID), dict(group=128, k_bits=4, v_bits=4),
               dict(k_mode=synth.SYM, v_mode=synth.SYM, group=64),
               dict(grouping=synth.OUTER, k_normalize=0, k_mode=synth.ASYM, v_mode=synth.ASYM, group=64)):
        w = synth.tiny(**kw)
        kb, vb = B.innerq_token_payload_bytes(B.make_config(w))
        assert bench.payload_bytes(w) == (kb, vb), kw
    # and the whole-call count on a case small enough to add up by hand: everything in windows -> fp16 rows only
    w = synth.tiny(n_tokens=12, w_sink=4, w_recent=16)
    dense, minimal = bench.decode_algorithmic_bytes(w, 12)
    rows = w.n_units * 12 * 2 * 256
    extras = w.batch * w.n_q_heads * 128 * 2 * 2 + w.n_units * 128 * 4
    assert dense == minimal == rows + extras
    # second roofs from the stored instruction counts: one sub-partition issues 1 instruction, 1/2 ALU-pipe instruction
    # and 1/8 MMA per cycle; the lowest of the three is reported
    assert bench.pipe_roofs_gbs(None, 1e6, 1965.0) is None
    c = {"warp_instructions": 592 * 1965, "alu_pipe": 592 * 1965, "tensor_pipe": 592 * 100}
    r = bench.pipe_roofs_gbs(c, 1e6, 1965.0)      # 1 us of issue, 2 us of ALU pipe, 0.41 us of tensor pipe
    assert r["lowest"] == "alu_pipe" and r["gbs"] == pytest.approx(500.0)
    assert r["all_gbs"]["issue"] == pytest.approx(1000.0)
    # every bench workload with a packed cache has its counters and DRAM traffic on file
    for name in ("c1", "c2", "c3_4bit", "c3_2bit", "c4"):
        w = bench.workload_by_name(name)
        c = bench.stored_counters(w.name)
        assert c is not None and c["alu_pipe"] < c["warp_instructions"], name
        assert bench.stored_traffic(w.name) == c["dram_read_bytes"] + c["dram_write_bytes"]


def test_sweep_workload_names_and_prefill_bytes():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2602_23200_b200 import synth
    w = bench.workload_by_name("c5_b4_g128_asym")
    assert (w.k_bits, w.v_bits, w.group, w.k_mode, w.v_mode, w.sym_variant) == (4, 4, 128, synth.ASYM, synth.ASYM, 0)
    assert (w.batch, w.n_kv_heads, w.n_tokens) == (16, 8, 8192)
    w = bench.workload_by_name("c5_b2_g64_literal")
    assert (w.k_mode, w.sym_variant) == (synth.HYBRID, 1)
    w = bench.workload_by_name("c5_b2_g32_hybrid+outer")
    assert w.grouping == synth.OUTER and w.k_normalize == 0 and w.group == 32
    with pytest.raises(SystemExit):
        bench.workload_by_name("c5_b2_g64_nonsense")
    # other code widths on a named shape: the paper's presets on the 32-head shape
    w = bench.workload_by_name("c2+k3v2")
    assert (w.k_bits, w.v_bits, w.n_kv_heads, w.n_tokens, w.k_mode) == (3, 2, 32, 32768, synth.HYBRID)
    w = bench.workload_by_name("c2+k3v3sym")
    assert (w.k_bits, w.v_bits, w.k_mode, w.v_mode) == (3, 3, synth.SYM, synth.SYM)
    with pytest.raises(SystemExit):
        bench.workload_by_name("c2+k5v3")
    # a prefill quantisation reads K and V once (fp16) and writes what a decode then reads
    w = synth.tiny(n_tokens=400)
    assert bench.prefill_algorithmic_bytes(w) == w.n_units * 400 * 128 * 2 * 2 + bench.decode_algorithmic_bytes(w, 400)[0]
    st = bench.stats([3.0, 1.0, 2.0, 10.0])
    assert (st["median"], st["min"], st["mean"], st["n"]) == (2.5, 1.0, 4.0, 4)
