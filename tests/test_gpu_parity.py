"""Parity of the CUDA path (through the C ABI) with the oracle, element by element, on seeded inputs.

Tolerances: selection indices bit-exact; fp32 inputs within 1e-5 and bf16 inputs within 2e-2 of the
sum of |products| per output element; selection sums within 1e-6 of sum |dY| of the map."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_1908_05460_b200 import binding as B
from paper_1908_05460_b200 import inputs as I
from paper_1908_05460_b200.layers import ConvLayer, config1_layer, resnet20_layers, vgg19_layers, cnn2_layers
from helpers import GpuLayer, norm_err, oshape, to_f64, TOL_F32, TOL_BF16, TOL_SUM

pytestmark = pytest.mark.gpu

DTYPES = [torch.float32, torch.bfloat16]


def tol(dtype):
    return TOL_F32 if dtype == torch.float32 else TOL_BF16


def top1_bound(layer, dtype):
    """What the top-1 output must really meet, tighter than the class tolerance.  The products sum * x are formed in
    fp32 from exactly widened inputs, and the map's sum is an fp32 tree sum (error ~1e-7 of sum|dY|), so the patch
    accumulation meets the fp32 class whatever the input type.  Only bf16 layers with at most 16 pixels per map and
    at least 128 input channels take the route 'sparse dY + dense tensor-core kernel', which rounds each sum to
    bf16 once (8 significant bits, round to nearest: at most 2^-8 |sum| <= 2^-8 sum|dY| per image, i.e. 2^-8 of the
    normaliser), plus the fp32 terms."""
    pq = layer.p * layer.q
    dense = dtype == torch.bfloat16 and ((pq <= 16 and layer.c >= 128) or (pq <= 64 and layer.c >= 256))
    return 2.0 ** -8 + 1e-4 if dense else 1e-5


# small cases spanning several tiles with ragged tails: C=3, W=2, stride 2, 5x5, odd sizes
SMALL = [
    config1_layer(),
    ConvLayer("c3 stem", 5, 3, 32, 32, 16, 3, 3, 1, 1, dy_std=1.0),
    ConvLayer("stride2", 6, 16, 32, 32, 32, 3, 3, 2, 1),
    ConvLayer("5x5", 4, 3, 32, 32, 64, 5, 5, 1, 2, x_dist="uniform_pm1"),
    ConvLayer("5x5 c64", 3, 64, 16, 16, 64, 5, 5, 1, 2),
    ConvLayer("ragged", 3, 19, 13, 11, 21, 3, 3, 1, 1, dy_std=1.0),
    ConvLayer("ragged s2 nopad", 2, 7, 15, 9, 5, 3, 3, 2, 0, dy_std=1.0),
    ConvLayer("w2", 9, 40, 2, 2, 24, 3, 3, 1, 1),
    ConvLayer("4x4", 8, 48, 4, 4, 80, 3, 3, 1, 1),
    ConvLayer("8x8", 8, 64, 8, 8, 64, 3, 3, 1, 1),
    ConvLayer("8x8 c128", 6, 128, 8, 8, 96, 3, 3, 1, 1),
    ConvLayer("8x8 c256 k40 n19 (ragged)", 19, 256, 8, 8, 40, 3, 3, 1, 1),
    ConvLayer("4x4 c128 k40 n19 (top-1 via sparse dY + dense kernel, ragged)", 19, 128, 4, 4, 40, 3, 3, 1, 1),
    ConvLayer("4x4 c256 (top-1 via sparse dY + dense kernel)", 5, 256, 4, 4, 64, 3, 3, 1, 1),
    ConvLayer("1x1", 4, 20, 9, 9, 12, 1, 1, 1, 0, dy_std=1.0),
    ConvLayer("7x7 filter", 2, 5, 12, 12, 6, 7, 7, 1, 3, dy_std=1.0),
    ConvLayer("one image one channel", 1, 1, 5, 5, 1, 3, 3, 1, 1, dy_std=1.0),
]


def _inputs(layer, dtype, tag):
    return I.make_layer_inputs(layer, dtype, config=9, layer_index=tag)


@pytest.mark.parametrize("dtype", DTYPES, ids=["f32", "bf16"])
@pytest.mark.parametrize("li", range(len(SMALL)), ids=[l.name for l in SMALL])
def test_exact_matches_oracle(li, dtype):
    layer = SMALL[li]
    x, dy = _inputs(layer, dtype, li)
    ref, dn = oracle.dw_exact(to_f64(x), to_f64(dy), oshape(layer), 0.5)
    g = GpuLayer(layer, dtype, x, dy, alpha=0.5)
    assert norm_err(g.exact(), ref, dn) <= tol(dtype)


@pytest.mark.parametrize("dtype", DTYPES, ids=["f32", "bf16"])
@pytest.mark.parametrize("li", range(len(SMALL)), ids=[l.name for l in SMALL])
def test_top1_matches_oracle(li, dtype):
    layer = SMALL[li]
    x, dy = _inputs(layer, dtype, li)
    xd, dyd = to_f64(x), to_f64(dy)
    idx_ref, sum_ref, abs_ref = oracle.top1_select(dyd)
    ref, dn = oracle.dw_top1(xd, dyd, oshape(layer), 1.0 / 128)
    g = GpuLayer(layer, dtype, x, dy, alpha=1.0 / 128)
    idx, s, sparse = g.select(want_sparse=True)
    np.testing.assert_array_equal(idx, idx_ref)                       # bit-exact selection
    assert np.max(np.abs(s - sum_ref) / np.maximum(abs_ref, 1e-300)) <= TOL_SUM
    # the dense sparse tensor: the (rounded) sum at the selected position, zero elsewhere
    sp = sparse.to(torch.float64).numpy().reshape(layer.n, layer.k, -1)
    want = np.zeros_like(sp)
    np.put_along_axis(want, idx_ref[..., None].astype(np.int64),
                      torch.from_numpy(s).to(dtype).to(torch.float64).numpy()[..., None], axis=2)
    np.testing.assert_array_equal(sp, want)
    e1 = norm_err(g.approx(B.METHOD_TOP1), ref, dn)                                  # one-launch cluster kernel, or sparse dY + dense kernel
    g2 = GpuLayer(layer, dtype, x, dy, alpha=1.0 / 128, algo=B.ALGO_DIRECT)
    e2 = norm_err(g2.approx(B.METHOD_TOP1), ref, dn)                                 # select + gather kernels
    print("top-1 normalised error: auto route %.3g (bound %.3g), select+gather %.3g (bound 1e-5)" % (e1, top1_bound(layer, dtype), e2))
    assert e1 <= top1_bound(layer, dtype) and e2 <= 1e-5


@pytest.mark.parametrize("x_layout,dw_layout", [(B.X_NCHW, B.DW_KCRS), (B.X_NHWC, B.DW_KCRS), (B.X_NCHW, B.DW_KRSC)])
def test_other_layouts(x_layout, dw_layout):
    layer = SMALL[5]
    x, dy = _inputs(layer, torch.float32, 40)
    xd, dyd = to_f64(x), to_f64(dy)
    g = GpuLayer(layer, torch.float32, x, dy, x_layout=x_layout, dw_layout=dw_layout)
    ref, dn = oracle.dw_exact(xd, dyd, oshape(layer))
    assert norm_err(g.exact(), ref, dn) <= TOL_F32
    ref, dn = oracle.dw_top1(xd, dyd, oshape(layer))
    assert norm_err(g.approx(B.METHOD_TOP1), ref, dn) <= TOL_F32
    z = oracle.dw_random(ref.size, 5, 0.25).reshape(ref.shape)
    assert np.max(np.abs(g.approx(B.METHOD_RANDOM, seed=5) * (0.25 * 128) - z)) < 1e-5 * 0.25 * 8


# ---- N x C x H x W activations on shapes the fast kernels serve: one transposing pass, then the channels-last route ----
NCHW_SHAPES = [
    ConvLayer("nchw 16->16@32", 6, 16, 32, 32, 16, 3, 3, 1, 1),
    ConvLayer("nchw 64->64@8", 9, 64, 8, 8, 64, 3, 3, 1, 1),
    ConvLayer("nchw 3->16@32 stem", 5, 3, 32, 32, 16, 3, 3, 1, 1),
    ConvLayer("nchw 40->24@16 ragged channels", 4, 40, 16, 16, 24, 3, 3, 1, 1),
    ConvLayer("nchw 256->64@4 small maps", 5, 256, 4, 4, 64, 3, 3, 1, 1),
]


@pytest.mark.parametrize("dtype", DTYPES, ids=["f32", "bf16"])
@pytest.mark.parametrize("li", range(len(NCHW_SHAPES)), ids=[l.name for l in NCHW_SHAPES])
def test_nchw_activations_take_the_fast_kernels_through_one_transposing_pass(li, dtype):
    layer = NCHW_SHAPES[li]
    x, dy = _inputs(layer, dtype, 45 + li)
    xd, dyd = to_f64(x), to_f64(dy)
    g = GpuLayer(layer, dtype, x, dy, x_layout=B.X_NCHW, alpha=0.5, topk=3)
    nhwc = GpuLayer(layer, dtype, x, dy, alpha=0.5, topk=3)
    ref, dn = oracle.dw_exact(xd, dyd, oshape(layer), 0.5)
    got = g.exact()
    assert norm_err(got, ref, dn) <= tol(dtype)
    np.testing.assert_array_equal(got, nhwc.exact())                 # the same kernels on the same values
    ref, dn = oracle.dw_top1(xd, dyd, oshape(layer), 0.5)
    got = g.approx(B.METHOD_TOP1)
    assert norm_err(got, ref, dn) <= top1_bound(layer, dtype)
    np.testing.assert_array_equal(got, nhwc.approx(B.METHOD_TOP1))
    ref, dn = oracle.dw_topk(xd, dyd, oshape(layer), 3, 0.5)
    assert norm_err(g.approx(B.METHOD_TOPK), ref, dn) <= TOL_F32
    assert B.gaconv_poll_async_status(g.desc) == B.OK
    # read in place when asked for the FP32-pipe kernel
    inplace = GpuLayer(layer, dtype, x, dy, x_layout=B.X_NCHW, alpha=0.5, algo=B.ALGO_DIRECT)
    ref, dn = oracle.dw_exact(xd, dyd, oshape(layer), 0.5)
    assert norm_err(inplace.exact(), ref, dn) <= tol(dtype)


# ---- N x P x Q x K output gradients (channels last): transposed once into the workspace, every method ----
@pytest.mark.parametrize("dtype", DTYPES, ids=["f32", "bf16"])
@pytest.mark.parametrize("li", [0, 1, 3, 4], ids=lambda i: NCHW_SHAPES[i].name.replace("nchw", "npqk"))
@pytest.mark.parametrize("x_layout", [B.X_NHWC, B.X_NCHW], ids=["x-nhwc", "x-nchw"])
def test_channels_last_output_gradients(li, dtype, x_layout):
    layer = NCHW_SHAPES[li]
    x, dy = _inputs(layer, dtype, 145 + li)
    g = GpuLayer(layer, dtype, x, dy, x_layout=x_layout, dy_layout=B.DY_NPQK, alpha=0.5, topk=2)
    plain = GpuLayer(layer, dtype, x, dy, alpha=0.5, topk=2)
    np.testing.assert_array_equal(g.exact(), plain.exact())           # the same kernels on the same values
    np.testing.assert_array_equal(g.approx(B.METHOD_TOP1), plain.approx(B.METHOD_TOP1))
    np.testing.assert_array_equal(g.approx(B.METHOD_TOPK), plain.approx(B.METHOD_TOPK))
    ref, dn = oracle.dw_exact(to_f64(x), to_f64(dy), oshape(layer), 0.5)
    assert norm_err(g.exact(), ref, dn) <= tol(dtype)
    with pytest.raises(B.GaconvError) as e:                            # the selection-only entry has no scratch to transpose into
        g.select()
    assert e.value.status == B.ERR_UNSUPPORTED
    assert B.gaconv_poll_async_status(g.desc) == B.OK


def test_selection_ties_and_planted_maxima():
    layer = ConvLayer("ties", 4, 2, 32, 32, 8, 3, 3, 1, 1)
    for dtype in DTYPES:
        x, dy = _inputs(layer, dtype, 50)
        dy = dy.clone()
        dy[0, 0].zero_()                                   # all-zero map -> index 0
        dy[0, 1, 31, 31] = 64.0; dy[0, 1, 3, 7] = -64.0    # equal magnitudes -> the earlier one
        dy[1, 2, 0, 0] = -77.0                             # first element
        dy[1, 3, 31, 31] = 77.0                            # last element
        dy[2, 4] = 1.0                                     # constant map -> index 0
        dy[3, 5, 10, :] = -3.0                             # a row of equal maxima -> its first
        g = GpuLayer(layer, dtype, x, dy)
        idx, s, _ = g.select()
        idx_ref, sum_ref, abs_ref = oracle.top1_select(to_f64(dy))
        np.testing.assert_array_equal(idx, idx_ref)
        assert idx[0, 0] == 0 and idx[0, 1] == 3 * 32 + 7 and idx[1, 2] == 0 and idx[1, 3] == 1023
        assert idx[2, 4] == 0 and idx[3, 5] == 320
        assert np.max(np.abs(s - sum_ref) / np.maximum(abs_ref, 1e-30)) <= TOL_SUM


def test_bf16_ties_occur_naturally_and_match():
    """bf16 gradients collide often; the tie rule is exercised on plain random inputs too."""
    layer = ConvLayer("bf16 ties", 64, 4, 32, 32, 32, 3, 3, 1, 1)
    _, dy = _inputs(layer, torch.bfloat16, 51)
    d = to_f64(dy).reshape(layer.n * layer.k, -1)
    top2 = np.sort(np.abs(d), axis=1)[:, -2:]
    assert np.count_nonzero(top2[:, 0] == top2[:, 1]) >= 5
    g = GpuLayer(layer, torch.bfloat16, torch.zeros(layer.n, layer.c, layer.h, layer.w, dtype=torch.bfloat16), dy)
    np.testing.assert_array_equal(g.select()[0], oracle.top1_select(to_f64(dy))[0])


def test_zero_and_random_methods():
    layer = config1_layer()
    x, dy = _inputs(layer, torch.float32, 60)
    g = GpuLayer(layer, torch.float32, x, dy, rand_std=1.0 / 128)
    z = g.approx(B.METHOD_ZERO)
    assert np.all(z == 0) and not np.any(np.signbit(z))
    count = z.size
    for seed in (0, 1, 0xDEADBEEFCAFEF00D):
        got = g.approx(B.METHOD_RANDOM, seed=seed).reshape(-1)
        ref = oracle.dw_random(count, seed, 1.0 / 128)
        assert np.max(np.abs(got - ref) / ((1.0 / 128) * np.maximum(1.0, np.abs(ref) * 128))) <= 1e-5
    # a count that is not a multiple of four, written through the strided (KRSC) path
    odd = ConvLayer("odd", 1, 3, 5, 5, 5, 3, 3, 1, 1)
    xo, dyo = _inputs(odd, torch.float32, 61)
    go = GpuLayer(odd, torch.float32, xo, dyo, rand_std=2.0)
    got = go.approx(B.METHOD_RANDOM, seed=9).reshape(-1)
    assert np.max(np.abs(got - oracle.dw_random(got.size, 9, 2.0))) <= 1e-5 * 2.0 * 6
    big = ConvLayer("big", 1, 256, 4, 4, 256, 3, 3, 1, 1)
    gb = GpuLayer(big, torch.float32, torch.zeros(1, 256, 4, 4), torch.zeros(1, 256, 4, 4), dw_layout=B.DW_KCRS)
    v = gb.approx(B.METHOD_RANDOM, seed=77).reshape(-1) * 128
    assert abs(v.mean()) < 4 / np.sqrt(v.size) and abs(v.std() - 1) < 0.01
    # every value of a large layer (2.4 million draws reach u1 within 1e-6 of 0 and of 1), both storage orders
    wide = ConvLayer("wide", 1, 512, 4, 4, 512, 3, 3, 1, 1)
    for layout in (B.DW_KCRS, B.DW_KRSC):
        gw = GpuLayer(wide, torch.float32, torch.zeros(1, 512, 4, 4), torch.zeros(1, 512, 4, 4), dw_layout=layout, rand_std=1.0)
        got = gw.approx(B.METHOD_RANDOM, seed=2024).reshape(-1)
        ref = oracle.dw_random(got.size, 2024, 1.0)
        assert np.max(np.abs(got - ref) / np.maximum(1.0, np.abs(ref))) <= 1e-5
        assert np.abs(ref).max() > 4.5 and np.abs(ref).min() < 1e-5          # the sample does reach both tails


def test_runs_are_bitwise_reproducible():
    layer = SMALL[2]
    x, dy = _inputs(layer, torch.bfloat16, 70)
    g = GpuLayer(layer, torch.bfloat16, x, dy)
    a, b = g.exact(), g.exact()
    np.testing.assert_array_equal(a, b)
    a, b = g.approx(B.METHOD_TOP1), g.approx(B.METHOD_TOP1)
    np.testing.assert_array_equal(a, b)


def test_full_selection_invariant_on_gpu():
    """With one output pixel per map the top-1 method keeps everything, so it must equal exact dW."""
    layer = ConvLayer("p=q=1", 16, 8, 3, 3, 8, 3, 3, 1, 0, dy_std=1.0)
    x, dy = _inputs(layer, torch.float32, 71)
    g = GpuLayer(layer, torch.float32, x, dy)
    ref, dn = oracle.dw_exact(to_f64(x), to_f64(dy), oshape(layer))
    assert norm_err(g.approx(B.METHOD_TOP1), ref, dn) <= TOL_F32
    assert norm_err(g.exact(), ref, dn) <= TOL_F32


def test_from_host_entry_point():
    layer = config1_layer()
    x, dy = _inputs(layer, torch.float32, 72)
    g = GpuLayer(layer, torch.float32, x, dy)
    xh = I.to_nhwc(x).pin_memory(); dyh = dy.contiguous().pin_memory()
    out = torch.empty(layer.k, layer.r, layer.s, layer.c, dtype=torch.float32).pin_memory()
    ref, dn = oracle.dw_exact(to_f64(x), to_f64(dy), oshape(layer))
    g.x.zero_(); g.dy.zero_()
    B.gaconv_dw_from_host(B.METHOD_EXACT, xh, dyh, out, g.x, g.dy, g.dw, g.desc)
    assert norm_err(I.krsc_to_kcrs(out).to(torch.float64).numpy(), ref, dn) <= TOL_F32
    ref, dn = oracle.dw_top1(to_f64(x), to_f64(dy), oshape(layer))
    B.gaconv_dw_from_host(B.METHOD_TOP1, xh, dyh, out, g.x, g.dy, g.dw, g.desc)
    assert norm_err(I.krsc_to_kcrs(out).to(torch.float64).numpy(), ref, dn) <= TOL_F32
    # no host inputs: the staging buffers are used as the previous call left them
    out.fill_(float("nan"))
    B.gaconv_dw_from_host(B.METHOD_TOP1, None, None, out, g.x, g.dy, g.dw, g.desc)
    assert norm_err(I.krsc_to_kcrs(out).to(torch.float64).numpy(), ref, dn) <= TOL_F32
    # the variant that does not wait: the result is on the host once the stream has been synchronised
    out.fill_(float("nan"))
    B.gaconv_dw_from_host_async(B.METHOD_TOP1, xh, dyh, out, g.x, g.dy, g.dw, g.desc)
    torch.cuda.current_stream().synchronize()
    assert norm_err(I.krsc_to_kcrs(out).to(torch.float64).numpy(), ref, dn) <= TOL_F32
    with pytest.raises(B.GaconvError) as e:                               # one host input without the other
        B.gaconv_dw_from_host(B.METHOD_TOP1, xh, None, out, g.x, g.dy, g.dw, g.desc)
    assert e.value.status == B.ERR_NULL_POINTER
    assert B.gaconv_poll_async_status(g.desc) == B.OK


def test_schedule_run_layer_dispatches_the_scheduled_method():
    layer = config1_layer()
    x, dy = _inputs(layer, torch.float32, 73)
    g = GpuLayer(layer, torch.float32, x, dy)
    ref_e, dn_e = oracle.dw_exact(to_f64(x), to_f64(dy), oshape(layer))
    ref_t, dn_t = oracle.dw_top1(to_f64(x), to_f64(dy), oshape(layer))
    s = B.Schedule(2, B.SCHED_LAYER2_ALT_BATCH, B.METHOD_TOP1)
    for step in range(4):
        for l in range(2):
            g.dw.fill_(float("nan"))
            s.run_layer(l, step, g.x, g.dy, g.dw, g.desc)
            if l == 1 and step % 2 == 1:
                assert norm_err(g.logical_dw(), ref_t, dn_t) <= TOL_F32
            else:
                assert norm_err(g.logical_dw(), ref_e, dn_e) <= TOL_F32
    r = B.Schedule(3, B.SCHED_ALL_LAYERS_EVERY_4TH_BATCH, B.METHOD_RANDOM, seed=5)
    r.run_layer(0, 3, g.x, g.dy, g.dw, g.desc); a = g.logical_dw()
    r.run_layer(0, 7, g.x, g.dy, g.dw, g.desc); b = g.logical_dw()
    r.run_layer(1, 7, g.x, g.dy, g.dw, g.desc); c = g.logical_dw()
    assert abs(np.corrcoef(a.ravel(), b.ravel())[0, 1]) < 0.1 and abs(np.corrcoef(b.ravel(), c.ravel())[0, 1]) < 0.1
    assert abs(a.std() * 128 - 1) < 0.1


# ---- full-size layers in the configuration the benchmark times: sampled outputs + whole top-1 ----
# (net, layer index, batch): batch 128 = the benchmark's step, batch 256 = the schedule sweep's launches
FULL = [("resnet", 1, 128), ("resnet", 7, 128), ("resnet", 13, 128), ("resnet", 18, 128), ("vgg", 1, 128), ("vgg", 5, 128),
        ("vgg", 9, 128), ("vgg", 15, 128), ("cnn", 0, 128), ("cnn", 1, 128),
        ("resnet", 8, 256), ("vgg", 3, 256), ("vgg", 6, 256), ("vgg", 12, 256)]


@pytest.mark.parametrize("net,li,batch", FULL, ids=["%s%d_n%d" % f for f in FULL])
@pytest.mark.parametrize("dtype", DTYPES, ids=["f32", "bf16"])
def test_full_size_layers(net, li, batch, dtype):
    layer = {"resnet": resnet20_layers, "vgg": vgg19_layers, "cnn": cnn2_layers}[net](batch)[li]
    if dtype == torch.float32 and (net == "vgg" or batch == 256):
        pytest.skip("VGG-19 and the schedule sweep are bf16 workloads")
    cfg = {"resnet": 2, "cnn": 3, "vgg": 4}[net] if batch == 128 else 5
    x, dy = I.make_layer_inputs(layer, dtype, cfg, li)
    xd, dyd = to_f64(x), to_f64(dy)
    g = GpuLayer(layer, dtype, x, dy)
    sh = oshape(layer)
    # top-1: the oracle covers the whole layer
    idx, s, _ = g.select()
    idx_ref, sum_ref, abs_ref = oracle.top1_select(dyd)
    np.testing.assert_array_equal(idx, idx_ref)
    assert np.max(np.abs(s - sum_ref) / abs_ref) <= TOL_SUM
    ref, dn = oracle.dw_top1(xd, dyd, sh)
    e1 = norm_err(g.approx(B.METHOD_TOP1), ref, dn)
    print("top-1 normalised error %.3g (bound %.3g)" % (e1, top1_bound(layer, dtype)))
    assert e1 <= top1_bound(layer, dtype)
    # exact: sampled output elements, each computed by the oracle on its own
    got = g.exact()
    rng = np.random.default_rng(li)
    picks = {(0, 0, 0, 0), (layer.k - 1, layer.c - 1, layer.r - 1, layer.s - 1), (layer.k - 1, 0, 0, layer.s - 1)}
    while len(picks) < 48:
        picks.add((int(rng.integers(layer.k)), int(rng.integers(layer.c)), int(rng.integers(layer.r)), int(rng.integers(layer.s))))
    worst = 0.0
    for (k, c, r, s_) in picks:
        v, nrm = oracle.dw_exact_at(xd, dyd, sh, k, c, r, s_)
        worst = max(worst, abs(got[k, c, r, s_] - v) / nrm)
    assert worst <= tol(dtype)
    assert np.all(np.isfinite(got))
    # the same layer as the benchmark's step launches it: sized for its share of the SMs (148 * roofline time / 12,
    # between 18 and 74), which changes the splits, the clusters and the top-1 grid
    eb = 2 if dtype == torch.bfloat16 else 4
    t_roof = max(layer.flops_exact() / (1654.6e12 * (1.0 if eb == 2 else 0.5)), layer.bytes_exact(eb) / 6456.2e9) * 1e6
    gb = GpuLayer(layer, dtype, x, dy, sm_budget=max(18, min(74, int(148 * t_roof / 12.0))))
    assert norm_err(gb.approx(B.METHOD_TOP1), ref, dn) <= top1_bound(layer, dtype)
    got = gb.exact()
    worst = 0.0
    for (k, c, r, s_) in picks:
        v, nrm = oracle.dw_exact_at(xd, dyd, sh, k, c, r, s_)
        worst = max(worst, abs(got[k, c, r, s_] - v) / nrm)
    assert worst <= tol(dtype)
    assert np.all(np.isfinite(got)) and B.gaconv_poll_async_status(gb.desc) == B.OK


# ---- tensor-core (tcgen05) exact path, forced, on shapes that exercise each of its tilings ----
TC_SHAPES = [
    ConvLayer("tc 16->16@32 halo M64 ct16", 8, 16, 32, 32, 16, 3, 3, 1, 1),
    ConvLayer("tc 32->32@16 ct32", 6, 32, 16, 16, 32, 3, 3, 1, 1),
    ConvLayer("tc 64->64@8 whole-image chunks", 16, 64, 8, 8, 64, 3, 3, 1, 1),
    ConvLayer("tc 64->64@32 ct64", 4, 64, 32, 32, 64, 3, 3, 1, 1),
    ConvLayer("tc 64->128@16 M128", 8, 64, 16, 16, 128, 3, 3, 1, 1),
    ConvLayer("tc 128->256@8 many tiles", 8, 128, 8, 8, 256, 3, 3, 1, 1),
    ConvLayer("tc 16->32 stride2", 6, 16, 32, 32, 32, 3, 3, 2, 1),
    ConvLayer("tc 32->64 stride2", 5, 32, 16, 16, 64, 3, 3, 2, 1),
    ConvLayer("tc 4x4 maps", 9, 48, 4, 4, 80, 3, 3, 1, 1),
    ConvLayer("tc 5x5 c64", 3, 64, 16, 16, 64, 5, 5, 1, 2),
    ConvLayer("tc ragged channels", 4, 40, 16, 16, 24, 3, 3, 1, 1),
    ConvLayer("tc k72", 4, 16, 8, 8, 72, 3, 3, 1, 1),
    ConvLayer("tc 1x1", 4, 32, 16, 16, 48, 1, 1, 1, 0),
    ConvLayer("tc many splits", 128, 16, 32, 32, 16, 3, 3, 1, 1),
    ConvLayer("tc 2x2 maps (transposed dY), one row per CTA", 40, 64, 2, 2, 128, 3, 3, 1, 1),
    ConvLayer("tc 2x2 maps, narrow", 33, 24, 2, 2, 40, 3, 3, 1, 1),
    ConvLayer("tc 1x1 maps", 70, 32, 1, 1, 64, 1, 1, 1, 0),
    ConvLayer("tc 128->128@16 one row per CTA", 4, 128, 16, 16, 128, 3, 3, 1, 1),
    ConvLayer("tc 512->512@4 one CTA per tile, whole output", 8, 512, 4, 4, 512, 3, 3, 1, 1),
    ConvLayer("tc 512->512@2 one CTA per tile, whole output", 64, 512, 2, 2, 512, 3, 3, 1, 1),
    ConvLayer("tc 256->256@8 several images per chunk, ragged batch", 21, 256, 8, 8, 256, 3, 3, 1, 1),
    # filter rows stacked in M (few output channels, "same" padding)
    ConvLayer("tc stacked rows, k20 (rows of the last block unused)", 4, 24, 16, 16, 20, 3, 3, 1, 1),
    ConvLayer("tc stacked rows, 5x5 k16", 3, 16, 16, 16, 16, 5, 5, 1, 2),
    ConvLayer("tc stacked rows, 8x8 maps, several images per chunk, ragged batch", 21, 32, 8, 8, 24, 3, 3, 1, 1),
    ConvLayer("tc stacked rows, k40 fills M = 128", 3, 16, 32, 32, 40, 3, 3, 1, 1),
    ConvLayer("tc no padding: rows not stacked", 4, 16, 18, 18, 16, 3, 3, 1, 0),
]


@pytest.mark.parametrize("li", range(len(TC_SHAPES)), ids=[l.name for l in TC_SHAPES])
def test_tensor_core_exact_matches_oracle_and_direct(li):
    layer = TC_SHAPES[li]
    x, dy = _inputs(layer, torch.bfloat16, 200 + li)
    g = GpuLayer(layer, torch.bfloat16, x, dy, alpha=0.25, algo=B.ALGO_TENSOR)
    got = g.exact()
    assert B.gaconv_poll_async_status(g.desc) == B.OK
    if layer.n * layer.p * layer.q * layer.k * layer.c <= 4e8:
        ref, dn = oracle.dw_exact(to_f64(x), to_f64(dy), oshape(layer), 0.25)
        assert norm_err(got, ref, dn) <= TOL_BF16
        assert norm_err(got, ref, dn) <= 1e-4        # bf16 products are exact in fp32: far inside the class tolerance
    gd = GpuLayer(layer, torch.bfloat16, x, dy, alpha=0.25, algo=B.ALGO_DIRECT)
    direct = gd.exact()
    scale = np.maximum(np.abs(direct), 1e-3 * np.abs(direct).max())
    assert np.max(np.abs(got - direct) / scale) < 1e-2
    np.testing.assert_array_equal(got, g.exact())                      # reproducible bit for bit


# ---- fp32 inputs: warp-level tensor-core path with split TF32 operands, and the FP32-pipe kernel ----
MMA_SHAPES = [
    ConvLayer("mma 16->16@32", 6, 16, 32, 32, 16, 3, 3, 1, 1),
    ConvLayer("mma 32->32@16 two c tiles", 5, 32, 16, 16, 32, 3, 3, 1, 1),
    ConvLayer("mma 64->64@8", 9, 64, 8, 8, 64, 3, 3, 1, 1),
    ConvLayer("mma stride 2", 4, 16, 32, 32, 32, 3, 3, 2, 1),
    ConvLayer("mma ragged channels", 3, 24, 16, 16, 20, 3, 3, 1, 1),
    ConvLayer("mma 1x1", 4, 32, 16, 16, 48, 1, 1, 1, 0),
    ConvLayer("mma c8", 7, 8, 32, 32, 16, 3, 3, 1, 1),
    ConvLayer("mma 5x5 64->64@16", 3, 64, 16, 16, 64, 5, 5, 1, 2),
    ConvLayer("mma 5x5 ragged", 4, 20, 16, 16, 24, 5, 5, 1, 2),
]


@pytest.mark.parametrize("li", range(len(MMA_SHAPES)), ids=[l.name for l in MMA_SHAPES])
def test_fp32_exact_split_tf32_and_fp32_pipes(li):
    layer = MMA_SHAPES[li]
    x, dy = _inputs(layer, torch.float32, 300 + li)
    ref, dn = oracle.dw_exact(to_f64(x), to_f64(dy), oshape(layer), 0.5)
    auto = GpuLayer(layer, torch.float32, x, dy, alpha=0.5)                       # split-TF32 tensor path
    got = auto.exact()
    assert norm_err(got, ref, dn) <= TOL_F32
    np.testing.assert_array_equal(got, auto.exact())
    pipes = GpuLayer(layer, torch.float32, x, dy, alpha=0.5, algo=B.ALGO_DIRECT)   # FP32 pipes
    assert norm_err(pipes.exact(), ref, dn) <= TOL_F32
    one = GpuLayer(layer, torch.float32, x, dy, alpha=0.5, math=B.MATH_TF32)      # one TF32 pass: its own, looser class
    e1 = norm_err(one.exact(), ref, dn)
    assert e1 <= 4e-3
    assert B.gaconv_poll_async_status(auto.desc) == B.OK


# ---- fp32 inputs on the tcgen05 kernel (kind::tf32), forced: three passes on split operands, and one plain TF32 pass ----
TC_F32_SHAPES = [
    ConvLayer("tcf32 64->64@8 M64", 9, 64, 8, 8, 64, 3, 3, 1, 1),
    ConvLayer("tcf32 64->128@16 M128", 5, 64, 16, 16, 128, 3, 3, 1, 1),
    ConvLayer("tcf32 96->72@8 ragged k, three c tiles", 7, 96, 8, 8, 72, 3, 3, 1, 1),
    ConvLayer("tcf32 32->200@16 two k tiles, ragged", 3, 32, 16, 16, 200, 3, 3, 1, 1),
    ConvLayer("tcf32 32->32@32 rows of 32", 4, 32, 32, 32, 32, 3, 3, 1, 1),
    ConvLayer("tcf32 1x1 64->48@16", 6, 64, 16, 16, 48, 1, 1, 1, 0),
    ConvLayer("tcf32 5x5 64->64@16", 3, 64, 16, 16, 64, 5, 5, 1, 2),
    ConvLayer("tcf32 7x7 32->16@8", 4, 32, 8, 8, 16, 7, 7, 1, 3),
    ConvLayer("tcf32 many images", 200, 32, 8, 8, 32, 3, 3, 1, 1),
]


@pytest.mark.parametrize("li", range(len(TC_F32_SHAPES)), ids=[l.name for l in TC_F32_SHAPES])
def test_fp32_on_tcgen05_matches_oracle(li):
    layer = TC_F32_SHAPES[li]
    x, dy = _inputs(layer, torch.float32, 340 + li)
    ref, dn = oracle.dw_exact(to_f64(x), to_f64(dy), oshape(layer), 0.5)
    g = GpuLayer(layer, torch.float32, x, dy, alpha=0.5, algo=B.ALGO_TENSOR)
    got = g.exact()
    assert B.gaconv_poll_async_status(g.desc) == B.OK
    assert norm_err(got, ref, dn) <= TOL_F32                     # big*big + big*small + small*big, fp32 accumulation
    np.testing.assert_array_equal(got, g.exact())
    one = GpuLayer(layer, torch.float32, x, dy, alpha=0.5, algo=B.ALGO_TENSOR, math=B.MATH_TF32)
    e1 = norm_err(one.exact(), ref, dn)
    assert TOL_F32 < e1 <= 4e-3                                   # one pass really is TF32: outside the fp32 class, inside its own
    kcrs = GpuLayer(layer, torch.float32, x, dy, alpha=0.5, algo=B.ALGO_TENSOR, dw_layout=B.DW_KCRS)
    np.testing.assert_array_equal(kcrs.exact(), got)


def test_tf32_mode_is_refused_where_it_has_no_kernel():
    layer = ConvLayer("7x7", 2, 16, 16, 16, 16, 7, 7, 1, 3)
    x, dy = _inputs(layer, torch.float32, 320)
    g = GpuLayer(layer, torch.float32, x, dy, math=B.MATH_TF32)
    with pytest.raises(B.GaconvError) as e:
        g.exact()
    assert e.value.status == B.ERR_UNSUPPORTED


# ---- few-channel (stem) layers: mma.sync over flattened image rows, both dtypes, against oracle and FP32 pipes ----
STEM_SHAPES = [
    ConvLayer("stem 3->16@32", 6, 3, 32, 32, 16, 3, 3, 1, 1),
    ConvLayer("stem 3->64@32", 3, 3, 32, 32, 64, 3, 3, 1, 1),
    ConvLayer("stem 5x5 3->64@32", 3, 3, 32, 32, 64, 5, 5, 1, 2, x_dist="uniform_pm1"),
    ConvLayer("stem 4 channels k20", 5, 4, 16, 16, 20, 3, 3, 1, 1),
    ConvLayer("stem stride 2", 4, 3, 32, 32, 24, 3, 3, 2, 1),
    ConvLayer("stem 1 channel", 7, 1, 32, 32, 8, 3, 3, 1, 1),
]


@pytest.mark.parametrize("dtype", DTYPES, ids=["f32", "bf16"])
@pytest.mark.parametrize("li", range(len(STEM_SHAPES)), ids=[l.name for l in STEM_SHAPES])
def test_stem_layers(li, dtype):
    layer = STEM_SHAPES[li]
    x, dy = _inputs(layer, dtype, 400 + li)
    ref, dn = oracle.dw_exact(to_f64(x), to_f64(dy), oshape(layer), 2.0)
    auto = GpuLayer(layer, dtype, x, dy, alpha=2.0)
    got = auto.exact()
    assert norm_err(got, ref, dn) <= (TOL_F32 if dtype == torch.float32 else 1e-4)
    np.testing.assert_array_equal(got, auto.exact())
    pipes = GpuLayer(layer, dtype, x, dy, alpha=2.0, algo=B.ALGO_DIRECT)
    assert norm_err(pipes.exact(), ref, dn) <= tol(dtype)
    kcrs = GpuLayer(layer, dtype, x, dy, alpha=2.0, dw_layout=B.DW_KCRS)
    assert norm_err(kcrs.exact(), ref, dn) <= tol(dtype)
    assert B.gaconv_poll_async_status(auto.desc) == B.OK


def test_workspace_control_words_are_left_as_found():
    """Every call must leave the workspace's control block (status word, ticket counters) all zero, so that
    a workspace initialised once serves any number of calls."""
    layer = ConvLayer("tickets", 24, 16, 16, 16, 32, 3, 3, 1, 1)
    for dtype in DTYPES:
        x, dy = _inputs(layer, dtype, 500)
        for algo in (B.ALGO_AUTO, B.ALGO_DIRECT):
            g = GpuLayer(layer, dtype, x, dy, algo=algo)
            g.exact(); g.approx(B.METHOD_TOP1); g.approx(B.METHOD_ZERO); g.approx(B.METHOD_RANDOM, seed=3)
            torch.cuda.synchronize()
            control = g.ws[:256 + 4096 * 4].cpu()
            assert int(control.to(torch.int32).abs().sum()) == 0
            assert B.gaconv_poll_async_status(g.desc) == B.OK


def _fuzz_shapes():
    rng = np.random.default_rng(20261125)
    out = []
    while len(out) < 28:
        r = int(rng.choice([1, 3, 5]))
        hw = int(rng.choice([2, 4, 7, 8, 16, 32]))
        stride = int(rng.choice([1, 2]))
        pad = int(rng.choice([0, r // 2]))
        if hw + 2 * pad < r:
            continue
        out.append(ConvLayer("fuzz%d" % len(out), int(rng.integers(1, 7)), int(rng.choice([1, 3, 8, 16, 24, 32, 64, 72])),
                             hw, hw, int(rng.choice([1, 8, 16, 24, 64, 80, 128])), r, r, stride, pad, dy_std=1.0))
    return out


FUZZ = _fuzz_shapes()


@pytest.mark.parametrize("li", range(len(FUZZ)), ids=["%s c%d k%d hw%d r%d s%d p%d" % (l.name, l.c, l.k, l.h, l.r, l.stride, l.pad) for l in FUZZ])
def test_seeded_random_geometries(li):
    """Planner robustness: whatever kernel a geometry is routed to, exact dW and top-1 match the oracle."""
    layer = FUZZ[li]
    for dtype in DTYPES:
        x, dy = _inputs(layer, dtype, 600 + li)
        xd, dyd = to_f64(x), to_f64(dy)
        g = GpuLayer(layer, dtype, x, dy)
        ref, dn = oracle.dw_exact(xd, dyd, oshape(layer))
        assert norm_err(g.exact(), ref, dn) <= tol(dtype)
        idx, _, _ = g.select()
        np.testing.assert_array_equal(idx, oracle.top1_select(dyd)[0])
        ref, dn = oracle.dw_top1(xd, dyd, oshape(layer))
        assert norm_err(g.approx(B.METHOD_TOP1), ref, dn) <= tol(dtype)
        assert B.gaconv_poll_async_status(g.desc) == B.OK


# ---- inputs the paper does not discuss: NaN, infinities, signed zeros in dY (selection is still defined) ----
def test_selection_of_nan_inf_and_signed_zero_matches_the_oracle():
    layer = ConvLayer("specials", 2, 2, 8, 8, 6, 3, 3, 1, 1, dy_std=1.0)
    for dtype in DTYPES:
        x, dy = _inputs(layer, dtype, 700)
        dy = dy.clone()
        dy[0, 0, 3, 4] = float("inf"); dy[0, 0, 5, 1] = float("-inf")         # two infinities: the earlier
        dy[0, 1, 2, 2] = float("inf"); dy[0, 1, 6, 6] = float("nan")           # NaN sorts above infinity
        dy[0, 2].zero_(); dy[0, 2, 1, 1] = -0.0                                # zeros of either sign: position 0
        dy[0, 3, 7, 7] = float("nan"); dy[0, 3, 0, 3] = float("nan")           # equal NaN payloads: the earlier
        dy[1, 4, 4, 4] = float("-inf")
        g = GpuLayer(layer, dtype, x, dy)
        idx, s, _ = g.select()
        idx_ref, sum_ref, _ = oracle.top1_select(to_f64(dy))
        np.testing.assert_array_equal(idx, idx_ref)
        assert idx[0, 0] == 3 * 8 + 4 and idx[0, 1] == 6 * 8 + 6 and idx[0, 2] == 0 and idx[0, 3] == 3 and idx[1, 4] == 36
        np.testing.assert_array_equal(np.isnan(s), np.isnan(sum_ref))          # the sum propagates as IEEE does
        np.testing.assert_array_equal(np.isinf(s), np.isinf(sum_ref))
        g.desc.topk = 3
        np.testing.assert_array_equal(g.select_topk()[0], oracle.topk_select(to_f64(dy), 3)[0])


# ---- the host half of the bounded-wait report: a raised status word is reported once, then cleared ----
def test_poll_reports_a_raised_status_word_once():
    layer = config1_layer()
    x, dy = _inputs(layer, torch.float32, 710)
    g = GpuLayer(layer, torch.float32, x, dy)
    assert B.gaconv_poll_async_status(g.desc) == B.OK
    g.ws[:4].copy_(torch.tensor([1, 0, 0, 0], dtype=torch.uint8))              # what a kernel's give-up branch writes
    assert B.gaconv_poll_async_status(g.desc) == B.ERR_TIMEOUT
    assert B.gaconv_poll_async_status(g.desc) == B.OK
    assert int(g.ws[:4].cpu().sum()) == 0


# ---- top-k variant (Section 2.3): selection bit-exact, dW within the fp32 class for both input types ----
TOPK_SHAPES = [
    ConvLayer("topk 16->16@32", 4, 16, 32, 32, 16, 3, 3, 1, 1),
    ConvLayer("topk ragged s2", 3, 7, 15, 9, 5, 3, 3, 2, 0, dy_std=1.0),
    ConvLayer("topk 4x4 c48", 6, 48, 4, 4, 40, 3, 3, 1, 1),
    ConvLayer("topk 2x2 (k clamps to 4)", 5, 8, 2, 2, 8, 3, 3, 1, 1),
    ConvLayer("topk 5x5", 2, 3, 16, 16, 8, 5, 5, 1, 2, x_dist="uniform_pm1"),
]


@pytest.mark.parametrize("topk", [1, 2, 5, 16])
@pytest.mark.parametrize("li", range(len(TOPK_SHAPES)), ids=[l.name for l in TOPK_SHAPES])
def test_topk_matches_oracle(li, topk):
    layer = TOPK_SHAPES[li]
    for dtype in DTYPES:
        x, dy = _inputs(layer, dtype, 720 + li)
        xd, dyd = to_f64(x), to_f64(dy)
        g = GpuLayer(layer, dtype, x, dy, alpha=0.5, topk=topk)
        idx, s = g.select_topk()
        idx_ref, sum_ref, abs_ref = oracle.topk_select(dyd, topk)
        np.testing.assert_array_equal(idx, idx_ref)
        assert np.max(np.abs(s - sum_ref) / np.maximum(abs_ref, 1e-300)) <= TOL_SUM
        ref, dn = oracle.dw_topk(xd, dyd, oshape(layer), topk, 0.5)
        got = g.approx(B.METHOD_TOPK)
        assert norm_err(got, ref, dn) <= TOL_F32
        np.testing.assert_array_equal(got, g.approx(B.METHOD_TOPK))             # reproducible
        # the ticketed gather kernel (what shapes beyond the one-launch kernel's shared memory take)
        gd = GpuLayer(layer, dtype, x, dy, alpha=0.5, topk=topk, algo=B.ALGO_DIRECT)
        assert norm_err(gd.approx(B.METHOD_TOPK), ref, dn) <= TOL_F32
        if topk == 1:
            ref1, dn1 = oracle.dw_top1(xd, dyd, oshape(layer), 0.5)
            assert norm_err(got, ref1, dn1) <= TOL_F32
    bad = GpuLayer(layer, torch.float32, *_inputs(layer, torch.float32, 720 + li), topk=0)
    with pytest.raises(B.GaconvError) as e:
        bad.approx(B.METHOD_TOPK)
    assert e.value.status == B.ERR_BAD_DESC


# ---- dW in the K K C_i C_o order (RSCK), through every kernel family ----
@pytest.mark.parametrize("li", [0, 2, 5, 8, 9], ids=lambda i: SMALL[i].name)
def test_rsck_output_layout(li):
    layer = SMALL[li]
    for dtype in DTYPES:
        x, dy = _inputs(layer, dtype, 740 + li)
        xd, dyd = to_f64(x), to_f64(dy)
        ref, dn = oracle.dw_exact(xd, dyd, oshape(layer), 0.5)
        ref1, dn1 = oracle.dw_top1(xd, dyd, oshape(layer), 0.5)
        for algo in (B.ALGO_AUTO, B.ALGO_DIRECT):
            g = GpuLayer(layer, dtype, x, dy, alpha=0.5, dw_layout=B.DW_RSCK, algo=algo)
            assert norm_err(g.exact(), ref, dn) <= tol(dtype)
            assert norm_err(g.approx(B.METHOD_TOP1), ref1, dn1) <= top1_bound(layer, dtype)
        z = oracle.dw_random(ref.size, 3, 1.0 / 128).reshape(ref.shape)
        assert np.max(np.abs(g.approx(B.METHOD_RANDOM, seed=3) - z)) <= 1e-5 * 6 / 128
        assert np.all(g.approx(B.METHOD_ZERO) == 0)


# ---- a whole step on several lanes: every layer's dW is bit for bit the per-layer call's ----
def test_run_step_on_lanes_equals_per_layer_calls():
    layers = [SMALL[0], SMALL[2], SMALL[8], SMALL[9], TC_SHAPES[4], SMALL[5], TC_SHAPES[14], SMALL[12]]
    gs = []
    for li, layer in enumerate(layers):
        x, dy = _inputs(layer, torch.bfloat16, 800 + li)
        gs.append(GpuLayer(layer, torch.bfloat16, x, dy, alpha=0.5))
    sched = B.Schedule(len(gs), B.SCHED_EVERY_4TH_LAYER, B.METHOD_TOP1)           # layers 2 and 6 (1-based) approximated
    want = []
    for li, g in enumerate(gs):
        g.dw.fill_(float("nan"))
        sched.run_layer(li, 5, g.x, g.dy, g.dw, g.desc)
        want.append(g.logical_dw())
    assert [sched.method(l, 5) for l in range(len(gs))].count(B.METHOD_TOP1) == 2
    packed = sched.pack_step([g.x for g in gs], [g.dy for g in gs], [g.dw for g in gs], [g.desc for g in gs])
    for lanes in (1, 3, 8):
        for g in gs:
            g.dw.fill_(float("nan"))
        sched.run_step(5, packed, lanes=lanes)
        for li, g in enumerate(gs):
            np.testing.assert_array_equal(g.logical_dw(), want[li])
    # inside a stream capture the fork and join of the lanes are part of the graph
    for g in gs:
        g.dw.fill_(float("nan"))
    torch.cuda.synchronize()
    gr = torch.cuda.CUDAGraph()
    with torch.cuda.graph(gr):
        sched.run_step(5, packed, lanes=4)
    for g in gs:
        g.dw.fill_(float("nan"))
    gr.replay()
    for li, g in enumerate(gs):
        np.testing.assert_array_equal(g.logical_dw(), want[li])
        assert B.gaconv_poll_async_status(g.desc) == B.OK
    # layers that run next to one another may not share a workspace
    shared = sched.pack_step([gs[0].x, gs[0].x], [gs[0].dy, gs[0].dy], [gs[0].dw, gs[1].dw], [gs[0].desc, gs[0].desc])
    with pytest.raises(B.GaconvError) as e:
        sched.run_step(5, shared, lanes=2)
    assert e.value.status == B.ERR_BAD_DESC


# ---- training-step integration: forward and input gradient from the framework, filter gradient from the library ----
def test_autograd_module_matches_the_frameworks_filter_gradient_and_follows_the_schedule():
    from paper_1908_05460_b200.autograd import GAConv2d
    torch.manual_seed(3)
    torch.backends.cudnn.allow_tf32 = False          # the framework's convolutions in true fp32, so that they can serve as a reference
    sched = B.Schedule(2, B.SCHED_LAYER2_ALT_BATCH, B.METHOD_TOP1)                # layer 2 approximated on odd steps
    conv1 = GAConv2d(3, 16, 3, padding=1, schedule=sched, layer_index=0)
    conv2 = GAConv2d(16, 16, 3, stride=2, padding=1, schedule=sched, layer_index=1)
    x = torch.randn(8, 3, 32, 32, device="cuda")
    for step in (0, 1):
        conv1.step = conv2.step = step
        for m in (conv1, conv2):
            m.weight.grad = None
        xin = x.clone().requires_grad_(True)
        h = torch.relu(conv1(xin))
        y = conv2(h)
        g = torch.randn_like(y)
        y.backward(g)
        # the framework's own gradients of the same graph
        w1 = conv1.weight.detach().clone().requires_grad_(True); w2 = conv2.weight.detach().clone().requires_grad_(True)
        xr = x.clone().requires_grad_(True)
        hr = torch.relu(torch.nn.functional.conv2d(xr, w1, None, 1, 1))
        yr = torch.nn.functional.conv2d(hr, w2, None, 2, 1)
        yr.backward(g)
        assert torch.allclose(xin.grad, xr.grad, rtol=1e-3, atol=1e-4)             # input gradients: framework both times
        assert torch.allclose(conv1.weight.grad, w1.grad, rtol=1e-3, atol=1e-3)    # layer 1 is always exact
        if step == 0:
            assert torch.allclose(conv2.weight.grad, w2.grad, rtol=1e-3, atol=1e-3)
        else:                                                                      # odd step: Algorithm 1 on layer 2
            layer = ConvLayer("l2", 8, 16, 32, 32, 16, 3, 3, 2, 1)
            ref, dn = oracle.dw_top1(to_f64(hr.detach().cpu()), to_f64(g.cpu()), oshape(layer))
            got = conv2.weight.grad.double().cpu().numpy()
            assert norm_err(got, ref, dn) <= 1e-4        # torch's forward runs in TF32/fp32: the activations differ in the last bits
            assert not torch.allclose(conv2.weight.grad, w2.grad, rtol=1e-2, atol=1e-3)
