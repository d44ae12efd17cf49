"""GPU parity of the convolution forms (Section "TSVD in Convolution Layer", Eq. 5): the library's
patch gather and single-stage forward, composed by TSVDConv2d, against the CPU checker's staged
evaluation V(.) -> diag(s)(.) -> U(.), element by element (fp32 outputs: maximum norm, 1e-5)."""
import numpy as np
import pytest

import gen
from oracle import conv as oc

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2308_07641_b200 import build
    build.build()


def _layer(seed, form, C_out, C_in, K1, K2, K, density=0.28):
    M, N = oc.matrix_shape(form, C_out, C_in, K1, K2)
    U = gen.rng.ternary(seed, 1, M * K, density).reshape(M, K)
    V = gen.rng.ternary(seed, 2, K * N, density).reshape(K, N)
    g = np.random.default_rng(seed)
    S = (np.exp(0.5 * g.standard_normal(K)) * g.choice([-1.0, 1.0], K)).astype(np.float32)
    return U, S, V


def _x(seed, shape, x_dtype):
    n = int(np.prod(shape))
    if x_dtype == "i8":
        return gen.rng.int8_uniform(seed, 4, n, -128, 127).reshape(shape)
    v = gen.rng.normal(seed, 4, n).astype(np.float32).reshape(shape)
    return gen.rng.f32_to_bf16_bits(v).reshape(shape) if x_dtype == "bf16" else v


def _run(form, geom, x_dtype, shape=(2, 13, 11), C_in=24, C_out=40, K1=3, K2=3, K=50, flags=0, seed=0):
    import torch
    from paper_2308_07641_b200 import device_activations
    from paper_2308_07641_b200.conv import TSVDConv2d
    stride, pad, dil = geom
    U, S, V = _layer(100 + seed + form, form, C_out, C_in, K1, K2, K)
    x = _x(200 + seed, shape + (C_in,), x_dtype)
    layer = TSVDConv2d(U, S, V, form, C_out, C_in, K1, K2, stride, pad, dil)
    try:
        xt = device_activations(x.reshape(-1, C_in), x_dtype).view(*shape, C_in)
        y = layer.forward(xt, flags).double().cpu().numpy()
        torch.cuda.synchronize()
        assert layer.status() == 0
    finally:
        layer.close()
    ref = oc.conv2d_tsvd(gen.widen_x(x, x_dtype), U, S, V, form, C_out, C_in, K1, K2, stride, pad, dil)
    assert y.shape == ref.shape
    assert np.abs(y - ref).max() <= 1e-5 * np.abs(ref).max(), (form, geom, x_dtype)


GEOMS = [((1, 1), (0, 0), (1, 1)), ((2, 2), (1, 1), (1, 1)), ((1, 2), (2, 0), (2, 1)), ((2, 1), (1, 2), (1, 2))]


@pytest.mark.parametrize("x_dtype", ["f32", "bf16", "i8"])
@pytest.mark.parametrize("geom", GEOMS, ids=lambda g: "s%d%d_p%d%d_d%d%d" % (g[0] + g[1] + g[2]))
@pytest.mark.parametrize("form", [0, 1, 2, 3])
def test_four_forms(form, geom, x_dtype):
    _run(form, geom, x_dtype)


@pytest.mark.parametrize("form", [0, 1, 2, 3])
def test_rectangular_kernels_and_ragged_channels(form):
    _run(form, ((1, 1), (1, 0), (1, 1)), "f32", shape=(1, 9, 17), C_in=7, C_out=13, K1=2, K2=5, K=19, seed=7)


@pytest.mark.parametrize("flags", [0x10, 0x20, 0x40], ids=["simple", "decode", "tensor"])
def test_every_kernel_family_serves_a_stage(flags):
    # one image of 3 x 4 pixels: with a 3x3 kernel and no padding 2 output pixels, within the decode limit
    _run(0, ((1, 1), (0, 0), (1, 1)), "f32", shape=(1, 3, 4), flags=flags, seed=3)
    _run(1, ((1, 1), (1, 1), (1, 1)), "bf16", shape=(1, 2, 3), flags=flags, seed=4)


def test_pointwise_form_is_the_linear_layer():
    """A [1,1] kernel: the convolution is the linear map on every pixel, and costs no patch gather."""
    import torch
    from paper_2308_07641_b200 import TSVDLinear, binding, device_activations
    from paper_2308_07641_b200.conv import TSVDConv2d
    U, S, V = _layer(9, 0, 48, 32, 1, 1, 64)
    x = _x(9, (2, 5, 6, 32), "f32")
    conv = TSVDConv2d(U, S, V, 0, 48, 32, 1, 1)
    lin = TSVDLinear(U, S, V)
    try:
        n0 = binding.tsvd_launch_count()
        y = conv.forward(device_activations(x.reshape(-1, 32), "f32").view(2, 5, 6, 32))
        torch.cuda.synchronize()
        assert binding.tsvd_launch_count() - n0 <= 8          # two stages of at most four kernels, no gather
        y_lin = lin.forward(device_activations(x.reshape(-1, 32), "f32"))
        err = (y.view(-1, 48) - y_lin).abs().max().item()
        assert err <= 1e-5 * y_lin.abs().max().item()
    finally:
        conv.close(); lin.close()


@pytest.mark.parametrize("case", [(12, 1, 1, 7, 7, 5, 0, ((1, 1), (3, 3), (1, 1)), "f32"),      # depth-wise 7x7, rank 5 per channel
                                  (4, 6, 3, 3, 3, 10, 2, ((2, 2), (1, 1), (1, 1)), "bf16"),
                                  (3, 4, 8, 2, 3, 9, 1, ((1, 1), (1, 1), (1, 2)), "i8")],
                         ids=["depthwise_7x7_rank5", "grouped_form2", "grouped_form1"])
def test_grouped_and_depthwise_layers(case):
    import torch
    from paper_2308_07641_b200 import device_activations
    from paper_2308_07641_b200.conv import TSVDConv2d
    G, co, ci, K1, K2, K, form, (stride, pad, dil), x_dtype = case
    layers = [_layer(300 + g, form, co, ci, K1, K2, K) for g in range(G)]
    Us, Ss, Vs = [l[0] for l in layers], [l[1] for l in layers], [l[2] for l in layers]
    x = _x(301, (2, 14, 11, G * ci), x_dtype)
    conv = TSVDConv2d(Us, Ss, Vs, form, G * co, G * ci, K1, K2, stride, pad, dil)
    try:
        y = conv.forward(device_activations(x.reshape(-1, G * ci), x_dtype).view(2, 14, 11, G * ci)).double().cpu().numpy()
        torch.cuda.synchronize()
        assert conv.status() == 0
    finally:
        conv.close()
    ref = oc.conv2d_tsvd_grouped(gen.widen_x(x, x_dtype), Us, Ss, Vs, form, G * co, G * ci, K1, K2, stride, pad, dil)
    assert y.shape == ref.shape
    assert np.abs(y - ref).max() <= 1e-5 * np.abs(ref).max()


@pytest.mark.parametrize("x_dtype", ["f32", "bf16", "i8"])
@pytest.mark.parametrize("geom", GEOMS, ids=lambda g: "s%d%d_p%d%d_d%d%d" % (g[0] + g[1] + g[2]))
@pytest.mark.parametrize("form", [0, 1, 2, 3])
def test_four_forms_with_patches_read_in_place(form, geom, x_dtype):
    """Channels and rank multiples of 16 and more than 16 output pixels: both stages read their patches in
    place (no patch matrix); same comparison with the checker."""
    from paper_2308_07641_b200 import binding
    n0 = binding.tsvd_launch_count()
    _run(form, geom, x_dtype, shape=(2, 13, 11), C_in=32, C_out=40, K=48, seed=11)
    assert binding.tsvd_launch_count() - n0 <= 8              # two stages of at most four kernels, no gather


@pytest.mark.parametrize("x_dtype", ["f32", "bf16", "i8"])
@pytest.mark.parametrize("shape,C,kernel,geom,K", [
    ((3, 20, 17), 48, (3, 3), ((1, 1), (1, 1), (1, 1)), 70),          # 1020 patches of 432 values: warp-per-token conversion
    ((1, 9, 8), 128, (3, 3), ((1, 1), (1, 1), (1, 1)), 33),           # 72 patches of 1152 values: resident conversion
    ((1, 40, 40), 256, (3, 3), ((2, 2), (0, 0), (1, 1)), 20),         # 361 patches of 2304 values
    ((2, 6, 7), 16, (5, 2), ((1, 2), (2, 1), (1, 2)), 9),             # small batch: 16-token tiles
])
def test_patches_in_place_equal_the_gathered_patches_bit_for_bit(shape, C, kernel, geom, K, x_dtype):
    import torch
    from paper_2308_07641_b200 import binding, device_activations
    k1, k2 = kernel
    stride, pad, dil = geom
    N = k1 * k2 * C
    V = gen.rng.ternary(500 + C, 2, K * N, 0.28).reshape(K, N)
    g = np.random.default_rng(C)
    S = (np.exp(0.5 * g.standard_normal(K)) * g.choice([-1.0, 1.0], K)).astype(np.float32)
    x = _x(600 + C, shape + (C,), x_dtype)
    n, H, W = shape
    dt = {"f32": binding.TSVD_F32, "bf16": binding.TSVD_BF16, "i8": binding.TSVD_I8}[x_dtype]
    Ho = (H + 2 * pad[0] - dil[0] * (k1 - 1) - 1) // stride[0] + 1
    Wo = (W + 2 * pad[1] - dil[1] * (k2 - 1) - 1) // stride[1] + 1
    B = n * Ho * Wo
    h = binding.tsvd_pack(np.zeros((1, K), np.int8), S, V)
    try:
        xt = device_activations(x.reshape(-1, C), x_dtype)
        cols = torch.empty((B, N), dtype=xt.dtype, device="cuda")
        binding.tsvd_im2col(xt.data_ptr(), dt, n, H, W, C, k1, k2, stride, pad, dil, cols.data_ptr(), N)
        t_ref = torch.empty((B, K), dtype=torch.float32, device="cuda")
        binding.tsvd_forward_v(h, cols.data_ptr(), N, t_ref.data_ptr(), K, B, dt, binding.TSVD_FLAG_PATH_TENSOR)
        t = torch.full((B, K + 3), -7.0, dtype=torch.float32, device="cuda")
        binding.tsvd_forward_v_patches(h, xt.data_ptr(), dt, n, H, W, C, k1, k2, stride, pad, dil, t.data_ptr(), K + 3,
                                       binding.TSVD_FLAG_PATH_TENSOR)
        torch.cuda.synchronize()
        assert binding.tsvd_last_status(h) in (0, 10)
        assert torch.equal(t[:, :K], t_ref)
        assert bool((t[:, K:] == -7.0).all())                 # padding of the caller's rows untouched
    finally:
        binding.tsvd_destroy(h)


def test_patches_in_place_rejects_what_it_cannot_read():
    import torch
    from paper_2308_07641_b200 import binding
    V = np.zeros((4, 9 * 24), np.int8)
    h = binding.tsvd_pack(np.zeros((1, 4), np.int8), np.ones(4, np.float32), V)
    try:
        x = torch.zeros((1, 8, 8, 24), device="cuda")
        t = torch.zeros((64, 4), device="cuda")
        for args in ((24, 3, 3),        # channels not a multiple of 16
                     (16, 3, 3)):       # 9 * 16 != N
            with pytest.raises(binding.TSVDError) as e:
                binding.tsvd_forward_v_patches(h, x.data_ptr(), binding.TSVD_F32, 1, 8, 8, args[0], args[1], args[2], (1, 1),
                                               (1, 1), (1, 1), t.data_ptr(), 4)
            assert e.value.status == binding.TSVD_E_SHAPE
    finally:
        binding.tsvd_destroy(h)
