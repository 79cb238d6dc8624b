"""The benchmark's accounting (no GPU): the algorithmic bytes and flops that the roofline fractions are computed from,
checked against figures worked out by hand for the pi0-scale expert, and the classification of the bound."""
import os

import bench
from paper_2609_12075_b200 import workloads as W


def test_algorithmic_work_of_the_batch_one_workload_by_hand():
    wl = W.config_c2()
    cfg = wl.cfg
    assert (cfg.n_layers, cfg.d_model, cfg.d_ff, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim) == (18, 1024, 4096, 8, 1, 256)
    assert len(wl.prefix_len) == 1 and int(wl.prefix_len[0]) == 816 and cfg.horizon == 50
    w = bench.algorithmic_work(cfg, wl.prefix_len, wl.n_steps)
    # one layer's weights, bf16: QKV 1024 x (2048 + 2 x 256), O 2048 x 1024, gate and up 2 x 1024 x 4096, down 4096 x 1024
    layer = 2 * (1024 * 2560 + 2048 * 1024 + 2 * 1024 * 4096 + 4096 * 1024)
    assert layer == 34603008
    assert w["per_class"]["gemm_gateup"]["bytes"] == 16 * 2 ** 20 and w["per_class"]["gemm_qkv"]["bytes"] == 5 * 2 ** 20
    # embedding side: the two time-MLP matrices, the action projection and the read-out
    embed = 2 * (2 * 1024 * 1024 + 32 * 1024 + 1024 * 32)
    # the prefix cache of one layer: 816 rows x (K and V) x 256 channels x 2 bytes
    kv_layer = 816 * 2 * 256 * 2
    assert w["step_bytes"] == 18 * (layer + kv_layer) + embed == 642220032
    # flops: 51 tokens through the four projections, attention of 51 x 8 query rows over 816 + 51 keys (QK and PV)
    proj = 2 * 51 * (layer // 2)
    att = 4 * 51 * 8 * 256 * (816 + 51)
    assert w["per_class"]["attention"]["flops"] == att
    assert w["step_flops"] == 18 * (proj + att) + 2 * 50 * (embed // 2)


def test_bound_is_memory_at_batch_one_and_tensor_at_batch_thirty_two():
    peaks = {"hbm_gbs": 6456.0, "bf16_tflops_sustained": 1431.0}
    c2, c4 = W.config_c2(), W.config_c4()
    _, r2 = bench.step_roofline(c2.cfg, c2.prefix_len, c2.n_steps, 6.7, peaks)
    _, r4 = bench.step_roofline(c4.cfg, c4.prefix_len, c4.n_steps, 18.0, peaks)
    assert r2["bound"] == "hbm" and r4["bound"] == "tensor"
    # 642 MB per step at 6456 GB/s, ten steps: 0.995 ms
    assert abs(r2["floor_ms_per_call"] - 10 * 642220032 / 6456e9 * 1e3) < 1e-9
    assert abs(r2["frac"] - r2["floor_ms_per_call"] / 6.7) < 1e-12 and 0.14 < r2["frac"] < 0.16
    assert abs(r4["achieved_tflops"] - r4["flops_per_euler_step"] * c4.n_steps / 18.0e-3 / 1e12) < 1e-6
    assert 0 < r4["frac"] < 1


def test_traffic_is_read_from_the_committed_profile_summaries():
    t = bench.traffic_from_profile("gemm_tc_kernel", "c2")
    assert t is not None and 8.0e6 < t < 1.0e7         # measured DRAM bytes of one projection launch (8.65 MB algorithmic)
    assert bench.traffic_from_profile("no_such_kernel", "c2") is None
    assert os.path.exists(os.path.join(bench.ROOT, "profiles", "gemm_tc_kernel_c2.md"))


def test_layer_timeline_on_a_synthetic_trace():
    import numpy as np
    rows, t = [], 1000
    for i in range(6):  # two kernel classes in turn, 5 us apart; only class 0 stamps its accumulators
        c = i % 2
        rows.append([c, 64, t - 500, t - 400, t + 3000, t + 3500, t, t + 10, t + 2000 if c == 0 else 0, t + 2500 if c == 0 else 0])
        t += 5000
    tl = bench.layer_timeline(np.array(rows, dtype=np.int64), ["a", "b"])
    a, b = tl["a"], tl["b"]
    assert a["launches"] == 3 and a["blocks"] == 64 and a["interval"] == 5.0
    assert abs(a["main"] - 2.49) < 1e-9 and abs(a["epilogue"] - 1.0) < 1e-9 and abs(a["handover"] - 1.51) < 1e-9
    assert b["launches"] == 2 and abs(b["release_to_end"] - 3.49) < 1e-9 and "main" not in b   # (the last launch has no successor)
