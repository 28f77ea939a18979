"""Host-side logic of bench.py and of the workload generators (no GPU)."""
import json
import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
from paper_1810_08313_b200 import workloads as wl  # noqa: E402


def test_clock_csv_parsing():
    text = "1965, 1965, 612.1, Not Active, Not Active, Not Active, Active\n" \
           "1800, 1965, 980.0, Not Active, Not Active, Not Active, Active\n" \
           "1342, 1965, 1001.2, Not Active, Not Active, Not Active, Not Active\n"
    c = bench.parse_clock_csv(text)
    assert c["sm_mhz"] == 1800.0 and c["sm_max_mhz"] == 1965.0 and c["reasons"] == ["sw_power_cap"] and c["samples"] == 3
    assert bench.parse_clock_csv("")["samples"] == 0
    bad = bench.parse_clock_csv("1965, 1965, 600, Active, Not Active, Not Active, Not Active\n")
    assert bad["reasons"] == ["hw_slowdown"]


def test_clock_csv_with_timestamps_is_cut_to_the_timed_region():
    import datetime
    t0 = datetime.datetime(2026, 1, 2, 3, 4, 5).timestamp()
    def stamp(dt):
        return datetime.datetime.fromtimestamp(t0 + dt).strftime("%Y/%m/%d %H:%M:%S.%f")[:-3]
    text = "".join(f"{stamp(0.02 * i)}, {1000 + i}, 1965, 500.0, Not Active, Not Active, Not Active, "
                   f"{'Active' if i == 7 else 'Not Active'}\n" for i in range(10))
    c = bench.parse_clock_csv(text, t0 + 0.05, t0 + 0.11)            # samples 3, 4, 5
    assert c["samples"] == 3 and c["sm_mhz"] == 1004.0 and c["reasons"] == []
    c = bench.parse_clock_csv(text)                                  # no window: everything
    assert c["samples"] == 10 and c["reasons"] == ["sw_power_cap"]
    assert bench.parse_clock_csv(text, t0 + 5.0, t0 + 6.0)["samples"] == 0


def test_both_arms_print_the_same_workload_keys():
    w = wl.WORKLOADS["c3_mlp_bf16"]
    c = bench.workload_config(w, 20)
    assert c["workload"] == "c3_mlp_bf16" and c["momentum"] == 0.9 and c["lr"] == 0.05 and c["tau"] == 20
    assert set(c) == {"workload", "dims", "m", "batch", "tau", "momentum", "lr", "dataset_rows"}


def test_work_models():
    w2, w3 = wl.WORKLOADS["c2_mlp_fp32"], wl.WORKLOADS["c3_mlp_bf16"]
    assert abs(bench.flops_per_replica_step(w2) / 1e9 - 1.010) < 0.01      # 1.01 GFLOP per replica-step
    assert abs(bench.flops_per_replica_step(w3) / 1e9 - 19.36) < 0.05      # 19.36 GFLOP per replica-step
    # update kernel, bf16 workload: layers 0-2 share one launch; 18 bytes per parameter per replica plus the
    # two operand tiles of every layer
    assert bench.streamed_update_layers(w3) == [0, 1, 2] and bench.streamed_update_layers(w2) == [0, 1]
    assert bench.update_state_bytes_per_launch(w3, 0) == 16 * 18 * (2048 * 3072 + 2 * 2048 * 2048)     # 18 B per parameter
    by = bench.update_bytes_per_launch(w3, 0)
    assert by == 16 * (18 * 2048 * 3072 + 2 * 256 * (2048 + 3072)) + 2 * 16 * (18 * 2048 * 2048 + 2 * 256 * 4096)
    # fp32 workload: 16 bytes per parameter, fp32 operands
    assert bench.update_bytes_per_launch(w2, 1) == 8 * (16 * 512 * 3072 + 4 * 128 * 3584) + 8 * (16 * 512 * 512 + 4 * 128 * 1024)
    assert bench.uses_tensor_cores(w3, "dw", 0) and bench.uses_tensor_cores(w2, "fwd", 0)
    assert not bench.uses_tensor_cores(w2, "fwd", 2) and not bench.uses_tensor_cores(w2, "dw", 2)
    assert not bench.uses_tensor_cores(wl.WORKLOADS["c1_softmax"], "dw", 0)
    peaks = {"hbm_gbs": 6547.2, "bf16_tflops": 1682.0, "bf16_tflops_sustained": 1398.0, "source": "measured"}
    r = bench.roofline_for(("dw", 0), 0.4e-3, w3, peaks, {"sm_mhz": 1900.0})
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / 6547.2) < 1e-12
    assert abs(r["achieved"] - 16 * 18 * 14_680_064 / 0.4e-3 / 1e9) < 1e-6 and r["operand_bytes_per_launch"] > 0
    r = bench.roofline_for(("fwd", 0), 60e-6, w2, peaks, {"sm_mhz": 1900.0})
    assert r["bound"] == "tensor" and abs(r["peak"] - 1398.0 * 1.1 / 2.25 / 3) < 1e-9
    r = bench.roofline_for(("fwd", 2), 10e-6, w2, peaks, {"sm_mhz": 1900.0})
    assert r["bound"] == "alu"
    r = bench.roofline_for(("avg", 0), 40e-6, w2, peaks, {})
    assert r["bound"] == "hbm" and abs(r["achieved"] - 8 * 8 * 1_841_162 * 2 / 40e-6 / 1e9) < 1e-6
    assert bench.probe_rows_for(w2) == 4096 and bench.probe_rows_for(wl.WORKLOADS["c4_lsq"]) == 4096


def test_peaks_loader_has_a_fallback(tmp_path, monkeypatch):
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    p = bench.load_peaks()
    assert p["source"] == "fallback" and p["hbm_gbs"] == 6650.0
    (tmp_path / "MEASURED_PEAKS.json").write_text(json.dumps({"hbm_gbs": 6000.0, "bf16_tflops": 1500.0,
                                                              "bf16_tflops_sustained": 1300.0}))
    p = bench.load_peaks()
    assert p["source"] == "measured" and p["hbm_gbs"] == 6000.0


def _rank_main(rank, world, port, out):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, units = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 100.0 * (rank + 1))
    out.put((rank, ms, units))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation_over_gloo():
    """--gpus N > 1 runs N independent jobs; the reported time is the max over ranks and the units add up."""
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, 15.0, 300.0), (1, 15.0, 300.0)]


def test_single_process_aggregation_is_identity():
    assert bench.aggregate_over_ranks(12.5, 640.0) == (12.5, 640.0)


# ---- workload generators ------------------------------------------------------------------------

def test_generators_are_deterministic_and_shaped():
    a = wl.gaussian_rows(7, 100, 12); b = wl.gaussian_rows(7, 100, 12)
    assert a.dtype == np.float32 and a.shape == (100, 12) and np.array_equal(a, b)
    assert not np.array_equal(a, wl.gaussian_rows(8, 100, 12))
    offs = wl.batch_row_offsets(3, 50, 4, 1000, 32)
    assert offs.shape == (50, 4) and offs.dtype == np.int64
    assert offs.min() >= 0 and offs.max() + 32 <= 1000 and np.all(offs % 32 == 0)
    u = wl.uniform_flat(1, 3, 1001)
    assert u.shape == (3, 1001) and u.min() >= -1.0 and u.max() < 1.0
    assert wl.n_params((3072, 512, 512, 10)) == 1_841_162 and wl.n_params((4096, 1), False) == 4096
    x1 = wl.random_mlp_point(5, (20, 10, 4))
    assert x1.size == wl.n_params((20, 10, 4)) and np.all(x1[200:210] == 0)        # biases start at zero
    y = wl.teacher_labels(5, a, (12, 9, 5))
    assert y.dtype == np.int32 and y.min() >= 0 and y.max() < 5 and len(np.unique(y)) > 1


def test_bf16_rounding_is_nearest_even_and_idempotent():
    x = np.array([1.0, 1.00390625, 1.005859375, 1.01171875, -3.14159, 1e-30, 65504.0], dtype=np.float32)
    r = wl.round_to_bf16(x)
    assert np.array_equal(wl.round_to_bf16(r), r)
    assert np.all((r.view(np.uint32) & 0xFFFF) == 0)
    assert r[0] == 1.0 and r[1] == 1.0            # 1 + 2^-8 is a tie: rounds to even (1.0)
    assert r[2] == np.float32(1.0078125)          # 1 + 1.5 * 2^-8 rounds up
    assert r[3] == np.float32(1.015625)           # 1 + 3 * 2^-8 is a tie: rounds to even (1 + 2^-6)
    import torch
    t = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(t, r)


def test_workload_table_matches_the_configurations():
    w = wl.WORKLOADS
    assert w["c1_softmax"].dims == (784, 10) and w["c1_softmax"].m == 4 and w["c1_softmax"].batch == 32
    assert w["c2_mlp_fp32"].dims == (3072, 512, 512, 10) and w["c2_mlp_fp32"].m == 8 and w["c2_mlp_fp32"].momentum == 0.9
    assert w["c3_mlp_bf16"].m == 16 and w["c3_mlp_bf16"].batch == 256 and w["c3_mlp_bf16"].adacomm_tau0 == 20
    assert w["c4_lsq"].m == 32 and w["c4_lsq"].batch == 64 and w["c4_lsq"].lr == 1e-4
    assert wl.AVERAGING_SWEEP_P[0] == wl.n_params(w["c3_mlp_bf16"].dims)
    X, y = wl.make_dataset(w["c1_softmax"], n_rows=256)
    assert X.shape == (256, 784) and y.dtype == np.int32
    A, t = wl.make_dataset(w["c4_lsq"], n_rows=128)
    assert A.shape == (128, 4096) and t.dtype == np.float32
    assert np.all(wl.initial_point(w["c1_softmax"]) == 0)
