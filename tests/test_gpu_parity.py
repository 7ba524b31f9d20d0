"""Element-by-element parity of the CUDA path against the CPU oracle on small and ragged cases."""
import numpy as np
import pytest
import torch

import paper_2507_07114_b200 as L
import workload
from parity_util import (GpuRun, assert_rel, assert_same, compare_outputs, compare_state, make_oracle,
                         run_parity, to_np)

pytestmark = pytest.mark.gpu
CFG = workload.baseline_workloads()
LOSSLESS, SKIP, REG = L.LOSSY_SELF_LOSSLESS, L.LOSSY_ZERO_SKIP, L.LOSSY_REGISTER_PATH
# the fused call has two kernels: the bulk-copy pipeline (default) and the register path
PATHS = pytest.mark.parametrize("path_flag", [0, REG], ids=["bulk", "reg"])


@PATHS
def test_config1_w4_sgd_fp32_all_steps(path_flag):
    w = CFG["cfg1_w4_sgd_f32"]
    run_parity(w, w.steps, flags=path_flag)


@pytest.mark.parametrize("mode", ["bulk", "reg", "unfused", "unfused_reg"])
def test_config2_shape_scaled_ragged(mode):
    # W=8, bf16 grads, Adam, P=2048: 37 packets + a short one whose length is not a multiple of 8
    w = workload.scaled(CFG["cfg2_w8_layer_adam"], 2048 * 37 + 1003)
    run_parity(w, 12, fused=not mode.startswith("unfused"), flags=REG if mode.endswith("reg") else 0)


@PATHS
@pytest.mark.parametrize("name", ["cfg3_w64_layer_p01", "cfg3_w64_layer_p10"])
def test_config3_shape_scaled(name, path_flag):
    w = workload.scaled(CFG[name], 4096 * 130 + 40)
    run_parity(w, 6, flags=path_flag)


@pytest.mark.parametrize("P", [256, 1024, 2048, 4096])
@pytest.mark.parametrize("p", [0.0, 0.01, 0.05, 0.1, 0.3])
def test_config5_sweep_scaled(P, p):
    w = workload.scaled(CFG["cfg5_w16_layer_sweep"], 4096 * 40 + 256 * 3, packet_elems=P, p=p)
    gpu, orc = run_parity(w, 4)
    if p == 0.0:
        assert float(gpu.norms.abs().max()) == 0.0
        assert int(gpu.count.min()) == 16


def test_config4_buckets_streamed_with_packet_base():
    """Bucket-by-bucket streaming: every bucket has its own context, shard map and global packet ids."""
    base = CFG["cfg4_w8_full_model"]
    sizes = [2048 * 21, 2048 * 21, 2048 * 13 + 512]
    pb = 0
    tot_g, tot_o = np.zeros(8), np.zeros(8)
    for b, n in enumerate(sizes):
        w = workload.scaled(base, n, packet_base=pb, seed=100 + b, name=f"cfg4_bucket{b}")
        gpu, orc = run_parity(w, 3)
        tot_g += to_np(gpu.sumsq)
        tot_o += orc.drift_sumsq()
        pb += w.K
    assert_rel(np.sqrt(tot_g), np.sqrt(tot_o), "model-level drift norms")
    # masks depend on the global packet id: the same bucket at another base gives other masks
    w0 = workload.scaled(base, sizes[0], packet_base=0, seed=100)
    w1 = workload.scaled(base, sizes[0], packet_base=5, seed=100)
    g0, _ = run_parity(w0, 1)
    g1, _ = run_parity(w1, 1)
    assert not torch.equal(g0.recv, g1.recv)


EDGE = [
    # name, W, n, P, p, opt, gd, rd, flags
    ("one_worker", 1, 5000, 256, 0.3, "adam", "bf16", "bf16", 0),
    ("w63", 63, 8 * 700 + 3, 8, 0.2, "sgd", "f32", "f32", 0),
    ("w33", 33, 264 * 50, 264, 0.1, "adam", "bf16", "f32", 0),
    ("fewer_packets_than_workers", 8, 3 * 512 - 100, 512, 0.2, "adam", "f32", "bf16", 0),
    ("single_short_packet", 4, 5, 1024, 0.3, "sgd", "bf16", "bf16", 0),
    ("tiny_packets", 4, 8 * 1000 + 1, 8, 0.1, "sgd", "bf16", "bf16", 0),
    ("heavy_loss_zero_received", 3, 64 * 300, 64, 0.7, "adam", "bf16", "bf16", 0),
    ("heavy_loss_zero_skip", 3, 64 * 300, 64, 0.7, "adam", "bf16", "bf16", SKIP),
    ("self_lossless", 8, 2048 * 9 + 16, 2048, 0.4, "adam", "bf16", "bf16", LOSSLESS),
    ("both_flags_sgd", 2, 128 * 77, 128, 0.6, "sgd", "f32", "f32", LOSSLESS | SKIP),
    ("w64_fp32", 64, 1024 * 20, 1024, 0.05, "sgd", "f32", "f32", 0),
    ("packet_not_multiple_of_chunk", 5, 1000 * 13 + 24, 1000, 0.15, "adam", "bf16", "bf16", 0),
    ("bulk_short_last_tile", 8, 1032 * 40 + 512, 1032, 0.2, "adam", "bf16", "bf16", 0),
    ("bulk_three_tiles_per_packet", 12, 2568 * 17 + 96, 2568, 0.25, "adam", "f32", "bf16", 0),
    ("bulk_w64_heavy_loss", 64, 1024 * 70, 1024, 0.5, "sgd", "bf16", "f32", 0),
    ("bulk_w17_two_groups", 17, 2048 * 33, 2048, 0.3, "adam", "bf16", "bf16", SKIP),
    ("bulk_f32_everything", 9, 1024 * 55 + 1000, 1024, 0.1, "adam", "f32", "f32", LOSSLESS),
    ("bulk_fewer_tiles_than_ctas", 8, 4096 * 3, 4096, 0.3, "adam", "bf16", "bf16", 0),
    ("bulk_zero_skip_w2", 2, 1024 * 40 + 24, 1024, 0.6, "adam", "bf16", "bf16", SKIP),
    ("bulk_zero_received_w3_f32", 3, 2048 * 25, 2048, 0.7, "sgd", "f32", "f32", 0),
    # many workers at high loss: the stale replicas' old copies travel as extra pipeline stages
    ("bulk_w64_stale_stages", 64, 1024 * 70 + 8, 1024, 0.3, "adam", "bf16", "bf16", 0),
    ("bulk_w48_stale_stages_f32", 48, 2048 * 21, 2048, 0.25, "sgd", "f32", "f32", 0),
    ("bulk_w50_stale_stages_mixed", 50, 1032 * 33 + 16, 1032, 0.45, "adam", "f32", "bf16", LOSSLESS),
    # small packets: a tile of the bulk-copy kernel packs several whole packets
    ("bulk_packed_256_w16_last_tile_short", 16, 256 * 37 + 100, 256, 0.2, "adam", "bf16", "bf16", 0),
    ("bulk_packed_128_w40", 40, 128 * 50 + 8, 128, 0.3, "sgd", "bf16", "bf16", 0),
    ("bulk_packed_512_w3_f32", 3, 512 * 21, 512, 0.4, "adam", "f32", "f32", SKIP),
    ("bulk_packed_1024_w16", 16, 1024 * 9 + 512, 1024, 0.1, "adam", "bf16", "bf16", LOSSLESS),
    ("bulk_packed_256_heavy_loss", 8, 256 * 64, 256, 0.6, "adam", "bf16", "bf16", 0),
    ("packed_wide_8_per_tile_low_loss", 16, 256 * 61 + 40, 256, 0.1, "adam", "bf16", "bf16", 0),
    ("packed_wide_4_per_tile_f32", 5, 512 * 27, 512, 0.15, "adam", "f32", "f32", SKIP),
    ("packed_twin_w24_two_per_tile", 24, 512 * 45 + 8, 512, 0.05, "sgd", "bf16", "bf16", 0),
    ("packed_128_elements_any_loss", 40, 128 * 90, 128, 0.4, "adam", "bf16", "f32", LOSSLESS),
    ("packed_128_w4", 4, 128 * 33 + 16, 128, 0.1, "sgd", "f32", "bf16", 0),
    # the gather pipeline where the policy would pick the register kernel: many stale copies per sub-packet
    ("gather_forced_w24_high_loss", 24, 256 * 70 + 8, 256, 0.4, "adam", "bf16", "bf16", L.LOSSY_GATHER_PATH),
    ("gather_forced_w64_f32_replicas", 64, 512 * 33, 512, 0.3, "sgd", "bf16", "f32", L.LOSSY_GATHER_PATH),
    # the wide gather build with drift warps: replica rows cut into halves (W = 12) and quarters (W = 5, W = 4), whole
    # rows with more stale chunks than the scratch holds (W = 24), fp32 replicas (sixteen chunks per row)
    ("packed_drift_warps_w12_halves", 12, 256 * 67 + 9, 256, 0.3, "adam", "bf16", "bf16", 0),
    ("packed_drift_warps_w5_quarters_512", 5, 512 * 41, 512, 0.2, "sgd", "f32", "bf16", 0),
    ("packed_drift_warps_w24_scratch_overflow", 24, 256 * 130 + 8, 256, 0.3, "adam", "bf16", "bf16", 0),
    ("packed_drift_warps_w7_f32_replicas", 7, 256 * 90, 256, 0.45, "adam", "bf16", "f32", L.LOSSY_GATHER_PATH),
    ("packed_drift_warps_w4_wide", 4, 256 * 75 + 100, 256, 0.3, "adam", "bf16", "bf16", SKIP),
    ("packed_drift_warps_w17_elided", 17, 512 * 40, 512, 0.25, "sgd", "bf16", "bf16", L.LOSSY_REPLICA_SKIP_OWNER),
    # fp32 replicas (the policy gives them to the compute warps; the flag asks for drift warps) leave each drift warp a
    # scratch of four chunks for a mean of 13 stale ones: most come from memory directly
    ("packed_drift_warps_w16_f32_replicas_direct_loads", 16, 256 * 75, 256, 0.45, "adam", "bf16", "f32", L.LOSSY_GATHER_PATH),
    # mostly whole rows: the two gather warps deal out every row's chunks instead of the workers
    ("packed_gather_chunks_dealt_w16", 16, 256 * 70 + 24, 256, 0.03, "adam", "bf16", "bf16", 0),
    ("packed_gather_chunks_dealt_w7_512_f32_grads", 7, 512 * 37, 512, 0.05, "sgd", "f32", "bf16", 0),
]


@pytest.mark.parametrize("case", EDGE, ids=[c[0] for c in EDGE])
@pytest.mark.parametrize("fused", [True, False, "packed_bulk"])
def test_edge_cases(case, fused):
    name, W, n, P, p, opt, gd, rd, flags = case
    if fused == "packed_bulk":
        # small packets have two fused builds: the gather pipeline (default) and the packed bulk-copy build
        if "packed" not in name:
            pytest.skip("not a small-packet case")
        flags |= L.LOSSY_PACKED_BULK
    w = workload.Workload(name, W, n, P, p, opt, 1e-2 if opt == "sgd" else 3e-4, gd, rd, 5, seed=42)
    gpu, orc = run_parity(w, 5, fused=bool(fused), flags=flags)
    if name.startswith("heavy_loss") or name.startswith("bulk_zero"):
        assert int((gpu.count == 0).sum()) > 0          # the nothing-received fallback was exercised


def test_different_p_grad_and_p_param():
    w = workload.Workload("two_rates", 6, 512 * 40, 512, 0.0, "adam", 3e-4, "bf16", "bf16", 4, seed=3)
    run_parity(w, 4, p_grad=0.25, p_param=0.05)
    run_parity(w, 4, p_grad=0.0, p_param=0.5, fused=False)


def test_fused_equals_unfused_bitwise_and_without_optional_outputs():
    w = workload.scaled(CFG["cfg2_w8_layer_adam"], 2048 * 50 + 8 * 11)
    a, b, c = GpuRun(w), GpuRun(w), GpuRun(w)
    for t in range(1, 6):
        gd = [workload.grad_slab(w, t, i, 0, w.n, "cuda") for i in range(w.W)]
        a.step_fused(t, gd)
        b.step_unfused(t, gd)
        c.step_fused(t, gd, outputs=False)
        torch.cuda.synchronize()
        for x, y in ((a, b), (a, c)):
            assert torch.equal(x.master, y.master) and torch.equal(x.m, y.m) and torch.equal(x.v, y.v)
            for i in range(w.W):
                assert torch.equal(x.replicas[i], y.replicas[i])
            # same numbers summed in another fixed order
            assert torch.allclose(x.norms, y.norms, rtol=2e-6, atol=0)
        assert torch.equal(a.norms, c.norms)
        assert torch.equal(a.ghat, b.ghat) and torch.equal(a.count, b.count)
        assert torch.equal(a.recv, b.recv) and torch.equal(a.stale, b.stale)
        assert torch.allclose(a.sumsq, b.sumsq, rtol=4e-6, atol=0)


def test_checkpoint_resume_is_bit_identical():
    w = workload.scaled(CFG["cfg2_w8_layer_adam"], 2048 * 20)
    a = GpuRun(w)
    for t in range(1, 11):
        a.step_fused(t, [workload.grad_slab(w, t, i, 0, w.n, "cuda") for i in range(w.W)])
    b = GpuRun(w)
    for t in range(1, 6):
        b.step_fused(t, [workload.grad_slab(w, t, i, 0, w.n, "cuda") for i in range(w.W)])
    saved = [b.master.cpu(), b.m.cpu(), b.v.cpu()] + [r.cpu() for r in b.replicas]
    b.close()
    c = GpuRun(w)                                       # fresh context: masks are a function of (seed, step, ...)
    c.master.copy_(saved[0]); c.m.copy_(saved[1]); c.v.copy_(saved[2])
    for i in range(w.W):
        c.replicas[i].copy_(saved[3 + i])
    for t in range(6, 11):
        c.step_fused(t, [workload.grad_slab(w, t, i, 0, w.n, "cuda") for i in range(w.W)])
    torch.cuda.synchronize()
    assert torch.equal(a.master, c.master) and torch.equal(a.v, c.v)
    for i in range(w.W):
        assert torch.equal(a.replicas[i], c.replicas[i])
    assert torch.equal(a.norms, c.norms)


def test_learning_rate_schedule():
    w = workload.Workload("lr_sched", 4, 256 * 30, 256, 0.1, "sgd", 1e-2, "f32", "f32", 4, seed=8)
    gpu, orc = GpuRun(w), make_oracle(w)
    for t, lr in enumerate([1e-2, 5e-3, 2.5e-3, 0.0], start=1):
        L.lossy_set_lr(gpu.ctx, lr)
        orc.set_lr(lr)
        gs = [workload.grad_slab(w, t, i, 0, w.n) for i in range(w.W)]
        gpu.step_fused(t, [g.cuda() for g in gs])
        ref = orc.step(t, [to_np(g) for g in gs])
        compare_outputs(gpu.outputs(), ref, f"lr step {t}")
        compare_state(gpu, orc, f"lr step {t}")


def test_empty_bucket_is_a_noop_and_bad_arguments_are_rejected():
    dev = "cuda"
    ctx = L.lossy_init(W=2, n=0, packet_elems=64, p_grad=0.1, p_param=0.1, seed=0, grad_dtype=torch.float32,
                       replica_dtype=torch.float32, optimizer="sgd", lr=0.1)
    z = [torch.zeros(8, device=dev) for _ in range(2)]
    norms = torch.ones(2, device=dev)
    L.lossy_fused_step(ctx, 1, z, z[0], None, None, z, norms=norms)
    torch.cuda.synchronize()
    assert float(norms.abs().sum()) == 0.0
    assert L.lossy_kernel_launches(ctx) == 0
    L.lossy_destroy(ctx)
    for bad in (dict(W=0), dict(W=65), dict(packet_elems=0), dict(packet_elems=12), dict(p_grad=1.0),
                dict(p_param=-0.1), dict(p_grad=float("nan")), dict(flags=64), dict(optimizer=5)):
        kw = dict(W=2, n=64, packet_elems=64, p_grad=0.1, p_param=0.1, seed=0, grad_dtype=torch.float32,
                  replica_dtype=torch.float32, optimizer="sgd", lr=0.1)
        kw.update(bad)
        with pytest.raises(L.LossyError) as ei:
            L.lossy_init(**kw)
        assert ei.value.code == L.LOSSY_EINVAL
    ctx = L.lossy_init(W=2, n=64, packet_elems=64, p_grad=0.1, p_param=0.1, seed=0, grad_dtype=torch.float32,
                       replica_dtype=torch.float32, optimizer="adam", lr=0.1)
    g = [torch.zeros(64, device=dev) for _ in range(2)]
    r = [torch.zeros(64, device=dev) for _ in range(2)]
    th = torch.zeros(64, device=dev)
    with pytest.raises(L.LossyError):                   # Adam without moments
        L.lossy_fused_step(ctx, 1, g, th, None, None, r)
    with pytest.raises(L.LossyError):                   # step 0
        L.lossy_fused_step(ctx, 0, g, th, th.clone(), th.clone(), r)
    mis = torch.zeros(80, device=dev)[1:65]             # 4-byte offset: not 16-byte aligned
    with pytest.raises(L.LossyError):
        L.lossy_fused_step(ctx, 1, [mis, g[1]], th, th.clone(), th.clone(), r)
    assert L.lossy_kernel_launches(ctx) == 0            # nothing was launched for rejected calls
    L.lossy_destroy(ctx)


@pytest.mark.parametrize("path_flag", [0, REG], ids=["bulk", "reg"])
@pytest.mark.parametrize("opt", ["sgd", "adam"])
def test_extreme_magnitudes_stay_bit_identical(path_flag, opt):
    """Gradients spanning 2^-120 .. 2^100 (denormal sums, overflowing squares, infinities and the NaNs Adam
    then produces): IEEE division, square root and the bf16 cast agree bit for bit on both sides."""
    W, P, K = 5, 1024, 24
    n = P * K
    w = workload.Workload("extreme_" + opt, W, n, P, 0.2, opt, 1e-2 if opt == "sgd" else 3e-4, "bf16", "bf16", 4,
                          seed=77)
    gpu, orc = GpuRun(w, flags=path_flag), make_oracle(w)
    gen = torch.Generator().manual_seed(5)
    for t in range(1, 5):
        gs = []
        for i in range(W):
            base = workload.grad_slab(w, t, i, 0, n).float()
            expo = torch.randint(-120, 101, (n,), generator=gen)
            gs.append((base * 1e3 * torch.pow(2.0, expo.float())).to(torch.bfloat16))
        gpu.step_fused(t, [g.cuda() for g in gs])
        orc.step(t, [to_np(g) for g in gs])
        torch.cuda.synchronize()
        for name, a, b in (("master", gpu.master, orc.master), ("m", gpu.m, orc.m), ("v", gpu.v, orc.v)):
            if opt == "sgd" and name != "master":
                continue
            ga, gb = to_np(a).view(np.uint32), b.view(np.uint32)
            nan_a, nan_b = np.isnan(to_np(a)), np.isnan(b)
            assert np.array_equal(nan_a, nan_b), f"{name}: NaN positions differ at step {t}"
            assert np.array_equal(ga[~nan_a], gb[~nan_b]), f"{name}: bits differ at step {t}"
        for i in range(W):
            ra, rb = to_np(gpu.replicas[i]), orc.replicas[i]
            nan = (ra & 0x7FFF) > 0x7F80
            assert np.array_equal(nan, (rb & 0x7FFF) > 0x7F80)
            assert np.array_equal(ra[~nan], rb[~nan]), f"replica {i}: bits differ at step {t}"
    if opt == "adam":
        assert np.isnan(orc.master).any() or np.isinf(orc.v).any()      # the overflow paths were reached


def test_ten_steps_captured_in_a_cuda_graph_replay_bit_identically():
    """The calls are stream-asynchronous and synchronise nothing, so a launch-bound loop (config 1: 40 MB per
    step) can be captured once and replayed as one graph launch."""
    w = CFG["cfg1_w4_sgd_f32"]
    eager, graphed = GpuRun(w), GpuRun(w)
    grads = [[workload.grad_slab(w, t, i, 0, w.n, "cuda") for i in range(w.W)] for t in range(1, 11)]
    for t in range(1, 11):
        eager.step_fused(t, grads[t - 1], outputs=False)
    saved = [graphed.master.clone()] + [r.clone() for r in graphed.replicas]
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        graphed.step_fused(1, grads[0], outputs=False)          # first use outside capture (one-time set-up)
        for dst, src in zip([graphed.master] + graphed.replicas, saved):
            dst.copy_(src)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for t in range(1, 11):
                graphed.step_fused(t, grads[t - 1], outputs=False)
    for _ in range(2):                                           # replay twice from the same start
        for dst, src in zip([graphed.master] + graphed.replicas, saved):
            dst.copy_(src)
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(graphed.master, eager.master) and torch.equal(graphed.norms, eager.norms)
        for a, b in zip(graphed.replicas, eager.replicas):
            assert torch.equal(a, b)
    L.lossy_device_status(graphed.ctx)


def test_host_gradient_entry_point_zero_copy_and_staged_match_the_device_path():
    """lossy_fused_step_host: pinned host gradients are read in place by the kernel, pageable ones are staged;
    both leave exactly the state of lossy_fused_step on device-resident gradients."""
    w = workload.scaled(CFG["cfg2_w8_layer_adam"], 2048 * 41 + 1003)
    ref, pinned, paged = GpuRun(w), GpuRun(w), GpuRun(w)
    staging = [torch.empty(w.n, dtype=torch.bfloat16, device="cuda") for _ in range(w.W)]
    host_norms = torch.zeros(w.W)
    for t in range(1, 5):
        gs = [workload.grad_slab(w, t, i, 0, w.n) for i in range(w.W)]
        ref.step_fused(t, [g.cuda() for g in gs], outputs=False)
        L.lossy_fused_step_host(pinned.ctx, t, [g.pin_memory() for g in gs], None, pinned.master, pinned.m, pinned.v,
                                pinned.replicas, pinned.norms, host_norms)
        assert torch.equal(host_norms, ref.norms.cpu())
        L.lossy_fused_step_host(paged.ctx, t, gs, staging, paged.master, paged.m, paged.v, paged.replicas,
                                paged.norms, host_norms)
        assert torch.equal(host_norms, ref.norms.cpu())
        for run in (pinned, paged):
            assert torch.equal(run.master, ref.master) and torch.equal(run.v, ref.v)
            for a, b in zip(run.replicas, ref.replicas):
                assert torch.equal(a, b)
    with pytest.raises(L.LossyError):                      # pageable memory without staging buffers
        L.lossy_fused_step_host(paged.ctx, 5, gs, None, paged.master, paged.m, paged.v, paged.replicas, paged.norms,
                                host_norms)


def test_launch_policy_picks_the_expected_build_for_the_benchmark_configurations():
    """lossy_describe_plan names the kernel build the fused step launches; the choices below are the
    measured policy for the benchmark's configurations and for its corner cases."""
    def plan(W, P, p, n=None, gd="bf16", rd="bf16", flags=0):
        n = P * 4000 if n is None else n
        ctx = L.lossy_init(W=W, n=n, packet_elems=P, p_grad=p, p_param=p, seed=1, grad_dtype=torch.bfloat16 if gd == "bf16" else torch.float32,
                           replica_dtype=torch.bfloat16 if rd == "bf16" else torch.float32, optimizer="adam", lr=1e-3, flags=flags)
        try:
            return L.lossy_describe_plan(ctx, True), L.lossy_describe_plan(ctx, False)
        finally:
            L.lossy_destroy(ctx)

    assert plan(8, 2048, 0.1)[0] == "bulk-copy wide group=4 stale=late stages=4"          # config 2
    assert plan(64, 4096, 0.1)[0] == "bulk-copy twin group=8 stale=late stages=3"         # config 3
    assert plan(4, 1024, 0.1, gd="f32", rd="f32")[0].startswith("bulk-copy twin group=4")  # config 1
    assert plan(16, 1024, 0.3)[0] == "bulk-copy twin group=8 stale=early stages=3"        # config 5, P = 1024
    assert plan(16, 256, 0.1)[0] == "gather wide packets/tile=8 stages=3"                  # config 5, small packets, low loss
    assert plan(16, 1024, 0.05)[0].startswith("bulk-copy wide group=8 stale=late packed")  # config 5, P = 1024, low loss: two packets per wide tile
    assert plan(16, 256, 0.3)[0] == "gather wide packets/tile=8 stages=3 drift-warps"      # ... at high loss: drift warps
    assert plan(16, 256, 0.3)[1] == "gather wide packets/tile=8 stages=3"                  # no drift norms asked for
    assert plan(17, 256, 0.5)[0] == "register kernel"                                     # eight stale replicas per sub-packet
    assert plan(32, 256, 0.05)[0] == "gather wide packets/tile=8 stages=3"                 # many workers: the compute warps read the stale copies
    assert plan(32, 256, 0.2)[0] == "register kernel"
    assert plan(8, 256, 0.3)[0] == "gather wide packets/tile=8 stages=3 drift-warps"
    assert plan(4, 256, 0.3)[0] == "gather wide packets/tile=8 stages=4 drift-warps"
    assert plan(3, 256, 0.3)[0] == "gather twin packets/tile=4 stages=4"                  # two or three workers: twin geometry
    assert plan(40, 128, 0.1)[0].startswith("gather twin packets/tile=8")                 # 128 elements: only the twin tile packs them
    assert plan(16, 256, 0.1, flags=L.LOSSY_PACKED_BULK)[0].startswith("bulk-copy wide group=8 stale=late packed")
    assert plan(64, 4096, 0.3)[0] == "bulk-copy twin group=8 stale=staged split stages=4"
    assert plan(24, 2048, 0.2)[0] == "bulk-copy twin group=8 stale=early split stages=3"
    # fp32 replicas do not fit bf16 gradient slots: early requests instead of staged copies
    assert plan(64, 4096, 0.3, rd="f32")[0] == "bulk-copy twin group=8 stale=early split stages=4"
    assert plan(64, 4096, 0.3)[1] == "bulk-copy twin group=8 stale=late split stages=4"   # no drift norms asked for
    assert plan(8, 2048, 0.1, flags=L.LOSSY_REGISTER_PATH)[0] == "register kernel"
    assert plan(8, 2048, 0.1, n=1000)[0] == "register kernel"                             # no complete packet


def test_packed_build_many_tiles_per_cta_with_skewed_stale_sets():
    """The PACKED build shares a tile's masks between its compute warps through two alternating buffers.
    Many tiles per CTA (forty) and sub-packets whose stale sets differ wildly (every fourth packet of a tile
    has a reliable broadcast, the others lose most of theirs) let the warps of a CTA drift far apart; the
    whole state must still match the oracle element by element."""
    W, P = 8, 256
    n = 2048 * 148 * 40 + 256 * 3
    w = workload.Workload("packed_skew", W, n, P, 0.0, "adam", 3e-4, "bf16", "bf16", 4, seed=77)
    gpu = GpuRun(w, flags=L.LOSSY_PACKED_BULK, p_grad=0.2, p_param=0.7)
    assert "packed" in L.lossy_describe_plan(gpu.ctx)
    orc = make_oracle(w, p_grad=0.2, p_param=0.7)
    K = w.K
    rel = np.zeros((2, K), np.uint64)
    rel[1, ::4] = np.uint64((1 << W) - 1)                 # these broadcasts always arrive
    rel_d = torch.from_numpy(rel.view(np.int64)).cuda()
    L.lossy_set_reliable(gpu.ctx, rel_d)
    for t in range(1, 4):
        gs = [workload.grad_slab(w, t, i, 0, n, "cuda") for i in range(W)]
        gpu.step_fused(t, gs)
        ref = orc.step(t, [to_np(g) for g in gs], reliable=rel)
        compare_outputs(gpu.outputs(), ref, f"packed skew step {t}")
        compare_state(gpu, orc, f"packed skew step {t}")
    L.lossy_device_status(gpu.ctx)


@pytest.mark.parametrize("W,P,p,plan", [
    (8, 256, 0.3, "gather wide packets/tile=8 stages=3 drift-warps"),
    (16, 512, 0.05, "gather wide packets/tile=4 stages=3"),
    (3, 256, 0.3, "gather twin packets/tile=4 stages=4"),
])
def test_gather_pipeline_rings_wrap_element_by_element(W, P, p, plan):
    """Ten tiles and more per CTA (148 CTAs of 2048-element tiles, or 296 of 1024): the mask ring, the wire ring and
    the stage ring wrap and their phase bits flip, compared with the oracle element by element over the whole bucket
    (the full-size tests compare sampled slabs)."""
    n = 2048 * 148 * 10 + P * 3 + 17
    w = workload.Workload(f"rings_w{W}_P{P}", W, n, P, p, "adam", 3e-4, "bf16", "bf16", 2, seed=21)
    gpu, _ = run_parity(w, 2)
    assert L.lossy_describe_plan(gpu.ctx) == plan
