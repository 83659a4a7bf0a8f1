"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU
oracle on the same seeded inputs.  Small cases are compared element by element;
the full-size benchmark configurations on sampled outputs and on properties."""
import numpy as np
import pytest
import torch

import oracle
from paper_2301_00330_b200 import workloads
from paper_2301_00330_b200.workloads import Layer

from parity_util import TOL, check_layer_full, check_layer_sampled, f64, relerr, run_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(params=["auto", "fused"])
def dense_path(gf, request):
    """Both ways a dense layer can be computed: the library's own choice per layer, and the fused
    gradient-filter + g_X kernel forced wherever it can run (layers it cannot take fall back to the
    separate kernels).  The library's choice is restored afterwards."""
    gf.gf_set_dense_path(gf.GF_PATH_FUSED if request.param == "fused" else gf.GF_PATH_AUTO)
    yield request.param
    gf.gf_set_dense_path(gf.GF_PATH_AUTO)


def L(name, N, Cin, Cout, H, W, K, G, r, dtype="f32", x_dist="relu", gy_std=1e-2, idx=0):
    return Layer(name, 0, idx, N, Cin, Cout, H, W, K, G, r, dtype, x_dist, gy_std)


SMALL = [
    L("tile_multi", 3, 24, 40, 14, 14, 3, 1, 2),
    L("partial_patches_r4", 3, 24, 40, 14, 14, 3, 1, 4),
    L("odd_map_7x7", 2, 8, 8, 7, 7, 3, 1, 2),
    L("ragged_channels", 2, 70, 130, 9, 11, 3, 1, 2),
    L("ragged_channels_1x1", 2, 130, 70, 12, 20, 1, 1, 4),
    L("r_gt_H", 1, 6, 4, 5, 5, 1, 2, 8),
    L("r3_generic", 2, 16, 16, 12, 9, 3, 1, 3),
    L("r7", 2, 16, 24, 32, 32, 3, 1, 7),
    L("k5", 2, 8, 12, 16, 16, 5, 1, 4),
    L("groups2", 2, 16, 24, 10, 10, 3, 2, 2),
    L("groups4_ragged", 3, 20, 12, 9, 9, 3, 4, 2),
    L("dw_r2", 2, 12, 12, 28, 28, 3, 12, 2),
    L("dw_r4", 2, 12, 12, 28, 28, 3, 12, 4),
    L("dw_r7", 2, 12, 12, 20, 20, 3, 12, 7),
    L("dw_odd", 3, 5, 5, 7, 9, 3, 5, 2),
    L("band_mode", 1, 3, 2, 160, 120, 3, 1, 2),
    L("band_mode_r8_ragged", 1, 2, 3, 100, 120, 3, 1, 8),
    L("dw_band_mode", 1, 4, 4, 160, 120, 3, 4, 4),
    L("big_patch", 1, 2, 2, 16, 600, 3, 1, 8),
    L("dw_big_patch", 1, 3, 3, 40, 4100, 3, 3, 40),
    L("n1", 1, 32, 32, 16, 16, 3, 1, 2),
    L("wide_map", 1, 8, 8, 6, 200, 3, 1, 2),
    L("odd_planes", 1, 3, 5, 14, 14, 3, 1, 2),
    L("many_small_planes", 5, 33, 47, 6, 6, 3, 1, 2),
    L("r8_16x16", 3, 20, 36, 16, 16, 3, 1, 8),
    L("r4_32x32", 2, 20, 12, 32, 32, 1, 1, 4),
    # narrow power-of-two maps: the pooling kernel's shuffle mode at its extremes
    L("lin_8x8_r8", 3, 16, 24, 8, 8, 3, 1, 8),
    L("lin_8x8_r2", 3, 16, 24, 8, 8, 1, 1, 2),
    L("lin_32x32_r8", 2, 8, 16, 32, 32, 3, 1, 8),
    L("lin_16x64_r2", 2, 8, 8, 16, 64, 3, 1, 2),
    L("lin_many_tiles", 8, 256, 128, 16, 16, 1, 1, 4),
    # long contraction over many input channels: the 128 x 256 output tiles of the g_W kernel (bf16),
    # with a ragged last tile
    L("gw_wide_tile", 200, 700, 72, 16, 16, 1, 1, 2),
    # many output channels: the 128-wide column tiles of the g_X kernel (bf16), ragged in every direction
    L("gx_wide_tile", 3, 40, 1032, 16, 16, 1, 1, 2),
    L("gx_wide_tile_partial", 2, 24, 1024, 14, 14, 1, 1, 4),
    L("gx_wide_tile_7x7", 5, 136, 1024, 14, 14, 1, 1, 2),
    # depthwise, streamed kernel: ring wrap-around (more tiles per CTA than ring slots), bands of
    # large planes, r = 8, 7-wide patch rows
    L("dw_ring_wrap", 16, 640, 640, 28, 28, 3, 640, 2),
    L("dw_band_ring", 4, 64, 64, 160, 120, 3, 64, 2),
    L("dw_r8", 2, 12, 12, 32, 32, 3, 12, 8),
    L("dw_14x14", 3, 40, 40, 14, 14, 3, 40, 2),
    L("dw_k5_r4", 2, 24, 24, 16, 48, 5, 24, 4),
    # patch planes whose size is not a multiple of 4: the tensor-core operands get a padded pitch
    L("pitch_rows_multi", 3, 24, 40, 30, 30, 3, 1, 2),      # 15x15 patches, several row tiles per image
    L("pitch_generic", 2, 16, 16, 9, 11, 3, 1, 2),          # 5x6 patches, partial patches
    L("pitch_r4_28x28", 2, 24, 16, 28, 28, 1, 1, 4),        # 7x7 patches
    L("pitch_wide_rows", 1, 8, 8, 6, 118, 3, 1, 2),         # 3x59 patches: rows too wide for a row tile
    L("pitch_many_images", 37, 136, 72, 14, 14, 1, 1, 2),   # 7x7 patches, two c_i tiles, many items per CTA
    # long contractions (C_out >= 512) on patch planes whose rows start on 16-byte boundaries: both
    # operands of both contractions through the copy engine, 64-patch units
    L("tma_pair_r2", 3, 72, 520, 16, 24, 1, 1, 2),          # 96 patches: units 3/4 full; ragged contraction tail
    L("tma_pair_generic_r3", 2, 264, 512, 24, 24, 3, 1, 3), # r = 3: element-wise stores; two c_i tiles
    L("tma_pair_partial", 2, 16, 512, 15, 31, 1, 1, 2),     # clipped patches at the right and bottom edges
    L("tma_pair_r8", 2, 24, 512, 64, 64, 1, 1, 8),
    L("tma_pair_r4_multi_ci", 2, 520, 512, 32, 32, 1, 1, 4),  # three c_i tiles of 176
    L("tma_pair_odd_units", 5, 40, 640, 16, 16, 3, 1, 2),   # five units: the last CTA's second unit is empty
    # 28-wide fp32 maps at r = 2 (14 patches per row): the fused kernel's row-aligned slot order, two whole patch rows
    # per 32 accumulator rows; 8-row and 6-row tiles, several c_i groups, a ragged c_o chunk
    L("row_aligned_slots", 3, 24, 40, 28, 28, 3, 1, 2),
    L("row_aligned_slots_groups", 2, 300, 72, 28, 28, 1, 1, 2),
    L("row_aligned_slots_w20", 2, 16, 24, 32, 20, 3, 1, 2),     # 10 patches per row: three rows per 32 slots
    L("tma_pair_ragged_ci", 2, 70, 512, 16, 16, 1, 1, 2),   # C_in neither a multiple of 16 nor of 4: scalar additions into g_W
    L("tma_pair_many_tiles", 56, 24, 64, 40, 48, 3, 1, 2),  # short contraction, 224 row tiles: the second arm of the rule
]


@pytest.mark.parametrize("layer", SMALL, ids=lambda l: l.name)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_small_shapes_element_by_element(gf, layer, dtype, dense_path):
    check_layer_full(gf, layer.with_(dtype=dtype))


def test_config1_r2_and_r1_exact(gf):
    (l2,) = workloads.config1(2)
    check_layer_full(gf, l2)
    (l1,) = workloads.config1(1)
    errs = check_layer_full(gf, l1)
    assert errs["stash"] == 0.0          # r == 1: the stash is x itself


def test_r1_exact_other_shapes(gf):
    for layer in (L("r1_groups", 2, 8, 12, 9, 7, 3, 2, 1), L("r1_k5", 1, 4, 4, 8, 8, 5, 1, 1),
                  L("r1_dw", 2, 6, 6, 8, 8, 3, 6, 1), L("r1_bf16", 2, 8, 8, 8, 8, 3, 1, 1, "bf16")):
        check_layer_full(gf, layer)


def test_nullable_outputs_and_repeatability(gf):
    layer = L("nullable", 2, 24, 40, 14, 14, 3, 1, 2)
    x, gy, w = workloads.make_inputs(layer)
    _, gW_a, gX_a = run_gpu(gf, layer, x, gy, w)
    _, gW_b, _ = run_gpu(gf, layer, x, gy, w, need_gx=False)
    _, _, gX_c = run_gpu(gf, layer, x, gy, w, need_gw=False)
    assert relerr(f64(gW_b), f64(gW_a)) <= TOL["f32"]
    assert torch.equal(gX_a, gX_c)
    for _ in range(2):
        _, gW_d, gX_d = run_gpu(gf, layer, x, gy, w)
        assert relerr(f64(gW_d), f64(gW_a)) <= TOL["f32"] and torch.equal(gX_d, gX_a)


def test_host_buffer_step_matches_device_path(gf):
    layer = L("host_step", 2, 24, 40, 14, 14, 3, 1, 2, "bf16")
    x, gy, w = workloads.make_inputs(layer)
    desc = gf.desc_for(layer)
    _, gW_dev, gX_dev = run_gpu(gf, layer, x, gy, w)
    hx, hgy, hw = x.pin_memory(), gy.pin_memory(), w.pin_memory()
    h_gW = torch.empty(gW_dev.shape, dtype=torch.float32).pin_memory()
    h_gX = torch.empty(gX_dev.shape, dtype=torch.bfloat16).pin_memory()
    arena = torch.empty(gf.gf_host_step_arena_bytes(desc), dtype=torch.uint8, device="cuda")
    gf.gf_layer_step_host(desc, hx, hgy, hw, h_gW, h_gX, arena)
    torch.cuda.synchronize()
    assert relerr(f64(h_gW), f64(gW_dev)) <= 1e-6
    assert torch.equal(h_gX, gX_dev.cpu())


# ---- the benchmark configurations at full size, in the launch configuration bench.py times ----
# Configurations 2, 3 and 4: every element of the stash, g_W and g_X against the checker (it needs
# a few seconds per layer).  Configuration 5 (up to 69 GFLOP of fp64 per layer): sampled outputs.
FULL_ELEMENTWISE = workloads.config2() + workloads.config3(2) + workloads.config3(4) + workloads.config4()
FULL_SAMPLED = [l for dt in ("f32", "bf16") for r in (2, 4, 8) for l in workloads.config5(r, dt)]


@pytest.mark.parametrize("layer", FULL_ELEMENTWISE, ids=lambda l: f"{l.name}_r{l.r}_{l.dtype}")
def test_full_size_configs_element_by_element(gf, layer):
    check_layer_full(gf, layer, isolate=False)


@pytest.mark.parametrize("layer", workloads.config2() + workloads.config3(2)[::2], ids=lambda l: f"{l.name}_r{l.r}_{l.dtype}")
def test_full_size_fused_path_element_by_element(gf, layer):
    """The fused kernels at full size on layers the library would give to the separate kernels."""
    gf.gf_set_dense_path(gf.GF_PATH_FUSED)
    try:
        check_layer_full(gf, layer, isolate=False)
    finally:
        gf.gf_set_dense_path(gf.GF_PATH_AUTO)


@pytest.mark.parametrize("layer", FULL_SAMPLED, ids=lambda l: f"{l.name}_r{l.r}_{l.dtype}")
def test_full_size_configs_sampled(gf, layer):
    check_layer_sampled(gf, layer)


# ---- exact arithmetic: inputs for which every intermediate of the method is an integer that the
# kernels' number formats hold exactly, so the results must equal the checker's BIT FOR BIT ----
# x in {0..3}: patch sums <= 3 r^2 (exact in bf16 up to 256).  g_y is patch-constant with integer
# values in {-3..3}: its patch means are those integers.  W in {-1, 0, 1}: kernel sums are integers
# of magnitude <= KH*KW.  Every product and every partial sum of either contraction is then an
# integer below 2^24, exact in fp32 in any order of summation; g_W (fp32) must equal the checker's
# integer and g_X must equal the checker's integer after ONE rounding to the output dtype.  A dropped
# K chunk, a wrong tile edge or a swapped column changes an integer and cannot hide under a tolerance.
EXACT = [
    L("exact_gw_wide_tile", 200, 700, 72, 16, 16, 1, 1, 2),        # bf16: 128 x 256 output tiles of the g_W kernel
    L("exact_gx_wide_tile", 3, 40, 1032, 16, 16, 1, 1, 2),         # bf16: 128-wide column tiles of the g_X kernel
    L("exact_gx_tile64", 3, 24, 40, 14, 14, 3, 1, 2),              # 64-wide column tiles, 3x3 kernel sums
    L("exact_two_ci_tiles", 5, 136, 264, 28, 28, 1, 1, 2),         # two c_i tiles, five K chunks, row tiles
    L("exact_r4_ragged_k", 9, 72, 200, 32, 32, 3, 1, 4),           # r = 4, C_out not a multiple of 64
    L("exact_many_items", 37, 96, 576, 28, 28, 1, 1, 2),           # many column tiles per CTA
    L("exact_wide_ci", 6, 576, 96, 28, 28, 1, 1, 2),               # C_in far above one accumulator
    L("exact_r8", 4, 128, 64, 32, 32, 3, 1, 8),
    L("exact_dw", 3, 40, 40, 28, 28, 3, 40, 2),                    # depthwise streamed kernel
    L("exact_groups", 3, 32, 48, 16, 16, 3, 4, 2),                 # grouped layer, CUDA-core path
]


def _integer_inputs(layer, seed):
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    assert layer.H % layer.r == 0 and layer.W % layer.r == 0
    x = torch.randint(0, 4, (layer.N, layer.C_in, layer.H, layer.W), generator=g).to(torch.float32)
    gbar = torch.randint(-3, 4, (layer.N, layer.C_out, layer.Hp, layer.Wp), generator=g).to(torch.float32)
    gy = gbar.repeat_interleave(layer.r, 2).repeat_interleave(layer.r, 3).contiguous()
    w = torch.randint(-1, 2, (layer.C_out, layer.C_ig, layer.K, layer.K), generator=g).to(torch.float32)
    dt = workloads.torch_dtype(layer.dtype)
    return x.to(dt), gy.to(dt), w.to(dt)


@pytest.mark.parametrize("layer", EXACT, ids=lambda l: l.name)
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_exact_arithmetic_bit_for_bit(gf, layer, dtype, dense_path):
    layer = layer.with_(dtype=dtype)
    x, gy, w = _integer_inputs(layer, seed=4242)
    stash_ref = oracle.stash_forward(f64(x), layer.r)
    gw_ref, gx_ref = oracle.backward(f64(gy), stash_ref, f64(w), layer.r, groups=layer.groups)
    assert np.abs(gw_ref).max() < 2 ** 24 and np.abs(gx_ref).max() < 2 ** 24
    stash, gW, gX = run_gpu(gf, layer, x, gy, w)
    assert np.array_equal(f64(stash), stash_ref)
    assert np.array_equal(f64(gW), gw_ref)
    gx_once_rounded = torch.from_numpy(gx_ref).to(workloads.torch_dtype(dtype))
    assert torch.equal(gX.cpu(), gx_once_rounded)


def test_error_word_is_reported_and_cleared(gf):
    """The report path of the bounded device-side waits, driven from the host: a non-zero error word
    copied into the workspace header reads back as GF_ERR_TIMEOUT; the next gf_backward on that
    workspace clears it before any of its kernels run, and a completed call reports GF_OK."""
    layer = L("err_word", 2, 24, 40, 14, 14, 3, 1, 2)
    x, gy, w = workloads.make_inputs(layer)
    desc = gf.desc_for(layer)
    buf = gf.alloc_layer(desc)
    xd, gyd, wd = x.cuda(), gy.cuda(), w.cuda()
    gf.gf_stash_forward(desc, xd, buf.stash)
    gf.gf_backward(desc, gyd, buf.stash, wd, buf.g_W, buf.g_X, buf.workspace)
    assert gf.gf_last_async_status(buf.workspace) == gf.GF_OK
    buf.workspace[:4].copy_(torch.tensor([2, 0, 0, 0], dtype=torch.uint8))      # as a timed-out wait would leave it
    torch.cuda.synchronize()
    assert gf.gf_last_async_status(buf.workspace) == gf.GF_ERR_TIMEOUT
    assert gf.gf_last_async_status(buf.workspace) == gf.GF_ERR_TIMEOUT          # reading does not clear a workspace's word
    gf.gf_backward(desc, gyd, buf.stash, wd, buf.g_W, buf.g_X, buf.workspace)
    assert gf.gf_last_async_status(buf.workspace) == gf.GF_OK


def test_a_device_wait_that_runs_out_is_reported(gf):
    """The bounded wait itself, on the GPU: a block waits (a millisecond's worth of clocks) on a barrier
    that nothing arrives on; the wait gives up, the block ends normally and records it, the host
    reads GF_ERR_TIMEOUT, and the context stays usable: the next backward on the same workspace
    clears the word, completes and matches the call made before."""
    layer = L("wait_runs_out", 2, 24, 40, 14, 14, 3, 1, 2)
    x, gy, w = workloads.make_inputs(layer)
    desc = gf.desc_for(layer)
    buf = gf.alloc_layer(desc)
    xd, gyd, wd = x.cuda(), gy.cuda(), w.cuda()
    gf.gf_stash_forward(desc, xd, buf.stash)
    gf.gf_backward(desc, gyd, buf.stash, wd, buf.g_W, buf.g_X, buf.workspace)
    assert gf.gf_last_async_status(buf.workspace) == gf.GF_OK
    gW0, gX0 = buf.g_W.clone(), buf.g_X.clone()
    gf.gf_selftest_bounded_wait(buf.workspace, 2_000_000)
    assert gf.gf_last_async_status(buf.workspace) == gf.GF_ERR_TIMEOUT
    gf.gf_backward(desc, gyd, buf.stash, wd, buf.g_W, buf.g_X, buf.workspace)
    assert gf.gf_last_async_status(buf.workspace) == gf.GF_OK
    assert torch.equal(buf.g_X, gX0) and relerr(f64(buf.g_W), f64(gW0)) <= 1e-6


def test_ondevice_table_shapes_sampled(gf):
    """The seven layer shapes of the paper's on-device latency table (batch 32,
    3x3, stride 1, pad 1); 14x14 with r = 4 has partial patches."""
    for layer in workloads.ondevice_table(r=4, N=8):
        check_layer_sampled(gf, layer, n_ch=4, n_img=1)


def test_oracle_disagrees_when_a_mistake_is_planted(gf):
    """The comparison is sharp enough to see a wrong patch divisor planted on the
    CPU side: the zero-padded average (divide by r^2 on partial patches)."""
    layer = L("planted", 2, 8, 8, 7, 7, 3, 1, 2)
    x, gy, w = workloads.make_inputs(layer)
    _, _, gX = run_gpu(gf, layer, x, gy, w)
    gsum = oracle.patch_sum(f64(gy), 2)
    wrong_mean = gsum / 4.0
    gx_wrong = oracle.reduced_gx(wrong_mean, oracle.kernel_sum(f64(w)), 1, 7, 7, 2)
    assert relerr(f64(gX), gx_wrong) > 100 * TOL["f32"]


def test_back_to_back_steps_in_a_cuda_graph(gf):
    """Steps replayed from a CUDA graph on ONE set of buffers (every kernel of a step starts as
    early as the dependency rules of the library allow) give what a single eager call gives."""
    layer = L("graph_steps", 8, 256, 256, 28, 28, 3, 1, 2, "bf16")
    x, gy, w = workloads.make_inputs(layer)
    desc = gf.desc_for(layer)
    xd, gyd, wd = x.cuda(), gy.cuda(), w.cuda()
    buf = gf.alloc_layer(desc)
    ws_bytes = gf.gf_backward_workspace_bytes(desc)
    stream = torch.cuda.Stream()

    def step():
        gf.gf_stash_forward(desc, xd, buf.stash, stream)
        gf.gf_backward(desc, gyd, buf.stash, wd, buf.g_W, buf.g_X, buf.workspace, ws_bytes, stream)

    with torch.cuda.stream(stream):
        step()
    torch.cuda.synchronize()
    gW_ref, gX_ref = buf.g_W.clone(), buf.g_X.clone()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        for _ in range(4):
            step()
    for _ in range(5):
        buf.g_W.zero_()
        buf.g_X.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert gf.gf_last_async_status(buf.workspace) == gf.GF_OK
        assert torch.equal(buf.g_X, gX_ref)
        assert relerr(f64(buf.g_W), f64(gW_ref)) <= 1e-5
