"""Host logic of bench.py that needs no GPU: the replica aggregation over ranks (gloo,
world size 2), the clock-sample parser and the workload bookkeeping."""
import json
import os
import subprocess
import sys
import textwrap

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2508_09035_b200 import workloads as wl  # noqa: E402


def test_aggregate_single_rank_is_identity():
    assert bench.aggregate_over_ranks(12.5, 4160.0, 1) == (12.5, 4160.0)


def test_aggregate_over_two_gloo_ranks(tmp_path):
    """Replicas: time is the max over ranks, units are summed."""
    script = tmp_path / "agg.py"
    script.write_text(textwrap.dedent("""
        import os, sys, json
        sys.path.insert(0, %r)
        import torch.distributed as dist
        import bench
        rank = int(os.environ["RANK"])
        dist.init_process_group("gloo", rank=rank, world_size=2)
        ms, units = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 100.0 * (rank + 1), 2)
        if rank == 0:
            print(json.dumps({"ms": ms, "units": units}))
        dist.destroy_process_group()
    """ % ROOT))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29631", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r)),
                              stdout=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=120)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs)
    res = json.loads(outs[0].strip().splitlines()[-1])
    assert res == {"ms": 15.0, "units": 300.0}


def test_clock_sampler_summary():
    s = bench.ClockSampler(0)
    s.rows = [["1350", "1965", "900.1", "0x4", "Not Active", "Not Active", "Not Active", "Active"],
              ["1365", "1965", "950.0", "0x0", "Not Active", "Not Active", "Not Active", "Not Active"],
              ["1950", "1965", "300.0", "0x0", "Not Active", "Not Active", "Not Active", "Not Active"]]
    out = s.stop()
    assert out["sm_mhz"] == 1365.0 and out["sm_max_mhz"] == 1965.0
    assert out["reasons"] == ["sw_power_cap"] and out["samples"] == 3


def test_workload_flops_and_shapes():
    w = wl.config_c2()
    assert w.n_tokens == 4160 and w.pairs_per_head() == 8654880
    assert abs(w.attention_flops() - 141.8e9) < 0.1e9
    assert [c.length for c in w.seqs[0].calls] == [512] * 8 + [64]
    assert [c.window for c in w.seqs[0].calls] == [False] * 7 + [True, False]
    w5 = wl.config_c5(n_seqs=4, len_lo=64, len_hi=512, chunk=128, max_received=8)
    assert len(w5.seqs) == 4 and all(64 <= s.n_prompt <= 512 for s in w5.seqs)
    st = wl.config_c3(n_layers=2, n_prompt=256, chunk=128, received_per_chunk=16)
    assert len(st.token_ids) == 288 and int((st.kind == wl.RECEIVED).sum()) == 32
    assert st.weight(0, "q").shape == (1536, 1536) and st.weight(1, "k").shape == (1536, 256)
    e = st.embedding_rows(st.token_ids[:3])
    assert e.shape == (3, 1536) and abs(float(e.std()) - 0.02) < 0.003


def test_grouped_calls_cover_every_call_once():
    """bench.py drives several sequences with batched calls: every call of every sequence
    appears exactly once, per sequence in its original order, and the grouping equals the one
    the parity tests use."""
    from tests import helpers as H
    w5 = wl.config_c5(n_seqs=5, len_lo=64, len_hi=700, chunk=128, max_received=8)
    groups = bench.grouped_calls(w5)
    assert [(k, win, [(si, c.pos0, c.length) for si, c in g]) for k, win, g in groups] == \
           [(k, win, [(si, c.pos0, c.length) for si, c in g]) for k, win, g in H.batched_steps(w5)]
    seen = {si: [] for si in range(5)}
    for kind, win, g in groups:
        assert len({si for si, _ in g}) == len(g)             # a sequence at most once per call
        for si, c in g:
            assert c.kind == kind and c.window == win
            seen[si].append(c.pos0)
    for si, s in enumerate(w5.seqs):
        assert seen[si] == [c.pos0 for c in s.calls]
    w2 = wl.config_c2()
    assert [g[0][1].pos0 for _, _, g in bench.grouped_calls(w2)] == [c.pos0 for c in w2.seqs[0].calls]


def test_attention_bytes_per_launch_and_traffic_scaling():
    """Algorithmic bytes of the mean attention launch: q + out of the call's rows and one read of
    the sequence's K and V up to its new length; the ncu capture is scaled by that figure and is
    dropped when the kernel source no longer matches the capture."""
    w = wl.small_like("bytes", 3, 8, 2, 128, 512, 256, 0, window="last")
    # two calls of 256 rows: lengths 256 and 512 after them
    per_row_q = 8 * 128 * 2
    per_pos_kv = 2 * 2 * 128 * 2
    want = (2 * 256 * per_row_q + 256 * per_pos_kv + 2 * 256 * per_row_q + 512 * per_pos_kv) / 2
    assert bench.attention_bytes_per_launch(w) == want
    cap = dict(bench.FWD_ATTN_TRAFFIC_CAPTURE)
    try:
        bench.FWD_ATTN_TRAFFIC_CAPTURE.update(dram_bytes=2.0e6, algorithmic_bytes=1.0e6,
                                              source_sha256=bench.attention_source_tag())
        assert bench.scaled_traffic(w) == 2.0 * want
        bench.FWD_ATTN_TRAFFIC_CAPTURE.update(source_sha256="not the kernel's hash")
        assert bench.scaled_traffic(w) is None
    finally:
        bench.FWD_ATTN_TRAFFIC_CAPTURE.update(cap)


def test_traffic_capture_belongs_to_the_kernel_source_in_the_tree():
    """The committed capture must have been taken on the committed attention kernel."""
    assert bench.FWD_ATTN_TRAFFIC_CAPTURE["source_sha256"] == bench.attention_source_tag()
