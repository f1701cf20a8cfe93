"""CUDA path vs the float64 oracle, element by element, through the C ABI."""
import numpy as np
import pytest

from paper_2502_20168_b200 import inputs as I
from tests.util import TOL, assert_close, compare_layer, oracle_layer

pytestmark = pytest.mark.gpu


def run(w, with_x0=False, with_gxT=False, mutate=None):
    from paper_2502_20168_b200 import harness
    d = I.draw_layer(w, with_x0=with_x0, with_gxT=with_gxT)
    if mutate:
        mutate(d)
    res = harness.run_layer(d, w.io_dtype, with_x0=with_x0, with_gxT=with_gxT)
    ref = oracle_layer(d, with_x0, with_gxT)
    keys = ["y", "xT", "du", "dLambda", "dDelta", "dB", "dC", "dD"] + (["dx0"] if with_x0 else [])
    errs = compare_layer(res, ref, w.io_dtype, keys)
    print(w.name, {k: f"{v:.1e}" for k, v in errs.items()})
    return errs


def test_c0_tiny_fp32():
    run(I.C0)


def test_c1_world_model_batch_fp32_with_resets():
    run(I.C1)


def test_c3_long_horizon_bf16():
    run(I.C3)


def test_paper_training_batches_bf16():
    # 32 x 128 batches at the sizes of the paper's state task (512 / 256) and vision task (1024 / 512)
    run(I.PAPER_STATE)
    run(I.PAPER_VISION)


@pytest.mark.parametrize("io", ["f32", "bf16"])
@pytest.mark.parametrize("B,T,H,P", [(3, 1, 8, 8), (2, 7, 24, 8), (5, 33, 40, 24), (2, 130, 72, 56),
                                     (1, 300, 64, 128), (9, 64, 128, 64)])
def test_ragged_shapes_with_resets_x0_and_gxT(io, B, T, H, P):
    w = I.Workload("edge", B=B, T=T, H=H, P=P, io_dtype=io, p_done=0.15, seed=B * 1000 + T)

    def flags(d):
        d["done"][0, 0] = 1          # flag on the first step beats x0
        d["done"][-1, -1] = 1        # flag on the last step
    run(w, with_x0=True, with_gxT=True, mutate=flags)


@pytest.mark.parametrize("B,T,H,P", [(1, 1, 256, 128), (2, 100, 256, 128), (3, 333, 512, 128),
                                     (5, 77, 256, 384), (700, 66, 256, 128),
                                     # H a multiple of 128 only: the last 256-column tile of y and du is half empty
                                     (3, 200, 384, 128), (90, 128, 128, 64), (400, 96, 384, 192),
                                     # long sequences, too few for the fused kernels: the streaming scans' tall reverse tiles, bf16 planes
                                     (2, 2304, 256, 128), (3, 2100, 256, 64)])
def test_tensor_core_path_shapes_bf16(B, T, H, P):
    # tile-sized H and P take the tcgen05 projections; B*T is ragged against the 128-row tiles
    w = I.Workload("tc", B=B, T=T, H=H, P=P, io_dtype="bf16", p_done=0.02, seed=B + T)
    run(w, with_x0=True, with_gxT=True)


@pytest.mark.parametrize("B,T,H,P", [(1, 1, 256, 128), (2, 100, 256, 128), (3, 333, 512, 128), (5, 77, 256, 384),
                                     (300, 66, 256, 128)])
def test_plane_path_shapes_fp32(B, T, H, P):
    # fp32 I/O with tile-sized H and P: the projections run on the tensor cores as sums of products of bf16
    # planes (three planes per fp32 value); B*T is ragged against the 128-row tiles.  fp32 tolerance.
    w = I.Workload("planes", B=B, T=T, H=H, P=P, io_dtype="f32", p_done=0.02, seed=B + T)
    run(w, with_x0=True, with_gxT=True)


@pytest.mark.parametrize("B,T,H,P", [(81, 128, 256, 128), (150, 256, 256, 64), (76, 384, 512, 128),
                                     (301, 64, 256, 128), (601, 32, 256, 128), (2403, 16, 256, 64),
                                     # chains of 64 states would occupy at most half of the CTA pairs: chains of 32 states
                                     (33, 64, 256, 256), (130, 16, 256, 256), (33, 128, 512, 128),
                                     # few long sequences: both CTAs of a pair on one sequence, tile by tile in turn
                                     (17, 256, 256, 256), (8, 768, 256, 512), (15, 512, 512, 256), (16, 2048, 256, 256),
                                     # the same with several chains per CTA pair (taken where it fills the last round better)
                                     (48, 256, 256, 256), (41, 512, 256, 256)])
def test_fused_projection_and_scan_shapes_bf16(B, T, H, P):
    # Enough (sequence, 64 states) chains and T a multiple of 128, or T = 16, 32, 64 (a 128-row tile
    # then holds whole sequences; odd B leaves the last tile ragged): the input projection and the
    # forward scan run as one kernel.  Odd B leaves one CTA of the last pair without work.
    w = I.Workload("fused", B=B, T=T, H=H, P=P, io_dtype="bf16", p_done=0.02, seed=B + T)

    def flags(d):
        d["done"][0, 0] = 1
        d["done"][-1, -1] = 1
        d["done"][1, min(127, T - 1)] = 1   # last row of a tile
        d["done"][2, 128 % T] = 1           # first row of a tile
        if T >= 512:
            d["done"][3, 255] = 1           # last row of a pair of tiles
            d["done"][4, 256] = 1           # first row of the next pair
            d["done"][5, 300:400] = 1       # a tile and its neighbour full of flags
    run(w, with_x0=True, with_gxT=True, mutate=flags)
    run(I.small_variant(w, p_done=0.0))


@pytest.mark.parametrize("io,B,T,H,P", [("f32", 3, 50, 40, 48), ("bf16", 80, 128, 256, 128), ("bf16", 5, 77, 256, 256)])
def test_conjugate_symmetric_variant_is_the_layer_with_half_the_states_and_doubled_C(io, B, T, H, P):
    """A system whose P states come in conjugate pairs is stored as its first P/2 states and run as
    this layer with C doubled (y = 2 Re(C_half x_half)).  The CUDA layer called that way is compared
    with the oracle on the FULL P-state system: y and du as they are, x_T on the stored half, and the
    half system's parameter gradients as the sums over each pair (g and conj(g)); the gradient with
    respect to C_half is twice the gradient the layer returns for the doubled C."""
    from oracle import ssm_oracle as O
    from paper_2502_20168_b200 import harness
    Ph = P // 2
    w = I.Workload("conj", B=B, T=T, H=H, P=Ph, io_dtype=io, p_done=0.03, seed=B + T + P)
    d = I.draw_layer(w, with_x0=True, with_gxT=False)
    Lam = np.concatenate([d["Lambda"], np.conj(d["Lambda"])])
    Dl = np.concatenate([d["Delta"], d["Delta"]])
    Bc = np.concatenate([d["Bc"], np.conj(d["Bc"])], axis=0)
    Cc = np.concatenate([d["Cc"], np.conj(d["Cc"])], axis=1)
    x0 = np.concatenate([d["x0"], np.conj(d["x0"])], axis=1)
    y, xT, _ = O.ssm_layer_fwd(Lam, Dl, Bc, Cc, d["D"], d["u"], d["done"], x0)
    g = O.ssm_layer_bwd(Lam, Dl, Bc, Cc, d["D"], d["u"], d["done"], x0, d["gy"])
    half = dict(d)
    half["Cc"] = (2.0 * d["Cc"]).astype(np.complex64)      # exact in fp32
    res = harness.run_layer(half, io, with_x0=True)
    tol = TOL[io]
    pair = lambda a, ax: np.take(a, range(Ph), axis=ax) + np.conj(np.take(a, range(Ph, P), axis=ax))
    errs = {
        "y": assert_close("y", res["y"], y, tol),
        "xT": assert_close("xT", res["xT"], xT[:, :Ph], tol),
        "du": assert_close("du", res["du"], g["du"], tol),
        "dD": assert_close("dD", res["dD"], g["dD"], tol),
        "dB": assert_close("dB", res["dB"], pair(g["dB"], 0), tol),
        "dLambda": assert_close("dLambda", res["dLambda"], pair(g["dLambda"], 0), tol),
        "dDelta": assert_close("dDelta", res["dDelta"], g["dDelta"][:Ph] + g["dDelta"][Ph:], tol),
        "dC_half": assert_close("dC_half", 2.0 * res["dC"], pair(g["dC"], 1), tol),
        "dx0": assert_close("dx0", res["dx0"], pair(g["dx0"], 1), tol),
    }
    print(w.name, {k: f"{v:.1e}" for k, v in errs.items()})


@pytest.mark.parametrize("io", ["f32", "bf16"])
def test_every_step_flagged_and_no_flags(io):
    w = I.Workload("all", B=2, T=40, H=32, P=16, io_dtype=io, p_done=0.5, seed=5)
    run(w, with_x0=True, mutate=lambda d: d["done"].fill(1))
    run(w, with_x0=True, mutate=lambda d: d["done"].fill(0))
    run(I.small_variant(w, p_done=0.0), with_gxT=True)


def test_very_many_short_sequences_fp32():
    # more than 512 * 64 sequences: the per-sequence partial sums of gAbar take two passes of the row reduction
    # (alternating between its two buffers) before the last kernel of the backward pass adds what is left
    w = I.Workload("many", B=33000, T=2, H=8, P=8, io_dtype="f32", p_done=0.1, seed=78)
    run(w, with_x0=True, with_gxT=True)


def test_long_sequence_small_batch_fp32():
    # long enough that a sequence is many tiles, with the state carried from tile to tile
    w = I.Workload("long", B=2, T=2500, H=16, P=24, io_dtype="f32", p_done=0.003, seed=77)
    run(w, with_x0=True, with_gxT=True)


def test_forward_backward_twice_is_bitwise_repeatable_and_workspace_reusable():
    import torch
    from paper_2502_20168_b200 import harness
    # Every sum has a fixed order: results repeat bit for bit.
    d = I.draw_layer(I.Workload("rep", B=160, T=24, H=64, P=256, io_dtype="f32", p_done=0.05, seed=9))
    buf = harness.LayerBuffers(d, "f32")
    buf.forward(); buf.backward()
    first = buf.results()
    buf.forward(); buf.backward()
    torch.cuda.synchronize()
    second = buf.results()
    for k in ("y", "du", "dB", "dC", "dLambda", "dDelta", "dD"):
        assert np.array_equal(first[k], second[k]), k
    # Few sequences, narrow tiles: the order of every sum is still fixed by the shape alone.
    d = I.draw_layer(I.C1)
    buf = harness.LayerBuffers(d, "f32")
    buf.forward(); buf.backward()
    first = buf.results()
    buf.forward(); buf.backward()
    torch.cuda.synchronize()
    second = buf.results()
    for k in ("y", "du", "dB", "dC", "dLambda", "dDelta", "dD"):
        assert np.array_equal(first[k], second[k]), k
    # Few long sequences, bf16: the two CTAs of a pair hand the state to each other tile by tile; the values
    # handed over do not depend on which of them runs ahead.  Five runs, all equal to the first.
    d = I.draw_layer(I.Workload("rep_pairs", B=16, T=1024, H=256, P=256, io_dtype="bf16", p_done=0.003, seed=11),
                     with_x0=True, with_gxT=True)
    buf = harness.LayerBuffers(d, "bf16", with_x0=True, with_gxT=True)
    buf.forward(); buf.backward()
    first = buf.results()
    for _ in range(4):
        buf.forward(); buf.backward()
        torch.cuda.synchronize()
        again = buf.results()
        for k in ("y", "xT", "du", "dx0", "dB", "dC", "dLambda", "dDelta", "dD"):
            assert np.array_equal(first[k], again[k]), k


def test_layer_step_replays_from_a_cuda_graph():
    """After a warm-up call, forward + backward issue only stream work (kernels, memsets), so a
    step can be captured once and replayed: the replay gives the results of the eager run."""
    import torch
    from paper_2502_20168_b200 import harness
    for w in (I.C1, I.Workload("paper_batch", B=32, T=128, H=512, P=256, io_dtype="bf16", p_done=0.01, seed=9)):
        d = I.draw_layer(w)
        buf = harness.LayerBuffers(d, w.io_dtype)
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            buf.forward(s); buf.backward(s)
        torch.cuda.synchronize()
        eager = buf.results()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            buf.forward(s); buf.backward(s)
        for k in ("y", "du", "dLambda", "dB", "dC"):
            getattr(buf, k).zero_()
        g.replay()
        torch.cuda.synchronize()
        sb_res = buf.results()
        for k in ("y", "du", "dLambda", "dDelta", "dB", "dC", "dD"):
            assert np.array_equal(eager[k], sb_res[k]), k


def test_backward_results_do_not_depend_on_a_kernel_running_beside_it():
    """Another stream keeps the GPU busy with reductions over the same gy and u while the backward
    pass runs: every result has to come out bit for bit as in a quiet run.  (Shared-memory buffers
    that the TMA unit refills right after the lanes have read them are where timing could show:
    the sweep point with 64 long sequences is the one where it once did.)"""
    import torch
    from paper_2502_20168_b200 import binding as sb, harness
    w = [c for c in I.C4 if c.T == 4096][0]
    buf = harness.LayerBuffers(I.draw_layer(w), w.io_dtype)
    main, side = torch.cuda.Stream(), torch.cuda.Stream()
    with torch.cuda.stream(main):
        buf.forward(main); buf.backward(main)
    torch.cuda.synchronize()
    sb.ssm_check(buf.ws)
    quiet = buf.results()
    acc = torch.zeros(w.H, dtype=torch.float32, device="cuda")
    for rep in range(6):
        for k in ("du", "dLambda", "dB", "dC", "dD"):
            getattr(buf, k).zero_()
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            for _ in range(8 + 3 * rep):
                acc += torch.sum(buf.gy.view(-1, w.H) * buf.u.view(-1, w.H), dim=0, dtype=torch.float32)
        with torch.cuda.stream(main):
            buf.backward(main)
        torch.cuda.synchronize()
        sb.ssm_check(buf.ws)
        busy = buf.results()
        for k in ("du", "dLambda", "dDelta", "dB", "dC", "dD"):
            assert np.array_equal(quiet[k], busy[k]), (rep, k)


@pytest.mark.parametrize("B,T,H,P,io", [(16, 1024, 256, 256, "bf16"), (80, 128, 256, 128, "bf16"), (4, 256, 256, 256, "bf16"),
                                        (16, 64, 256, 128, "f32"), (2, 40, 32, 16, "f32")])
def test_plan_string_names_the_stages_that_run(B, T, H, P, io):
    """ssm_layer_plan_string against the stages the library's own timers see for the same shape."""
    import torch
    from paper_2502_20168_b200 import binding as sb, harness
    w = I.Workload("plan", B=B, T=T, H=H, P=P, io_dtype=io, seed=3)
    buf = harness.LayerBuffers(harness.device_drawn(w), io)
    buf.forward(); buf.backward()
    torch.cuda.synchronize()
    sb.ssm_profile_begin()
    buf.forward(); buf.backward()
    torch.cuda.synchronize()
    stages = set(sb.ssm_profile_end())
    sb.ssm_check(buf.ws)
    plan = sb.ssm_layer_plan_string(sb.make_shape(B, T, H, P, io))
    fused = "scans=fused" in plan
    assert fused == ("gemm_Bu_scan_fwd" in stages) == ("gemm_gx_scan_bwd" in stages), (plan, stages)
    assert fused != ("scan_fwd" in stages), (plan, stages)
