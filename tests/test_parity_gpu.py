"""GPU parity: the CUDA library, called through the C ABI, against the CPU checker on the same
seeded inputs.  Small cases are compared element by element over every token; the full-size
configurations are compared on sampled token columns (columns are independent, so the checker
computes each sampled column completely)."""
import numpy as np
import pytest

import gen
import oracle
from tests import _util

pytestmark = pytest.mark.gpu

C = gen.CONFIGS


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2308_07641_b200 import build
    build.build()


def test_pack_roundtrip_and_info():
    from paper_2308_07641_b200 import binding
    for (M, K, N, d) in [(1, 1, 1, 1.0), (130, 63, 345, 0.3), (256, 256, 256, 0.3), (1000, 2415, 96, 0.1)]:
        spec = gen.scaled(C["cfg1"], M=M, K=K, N=N, B=1, density=d, seed=77)
        U, V, S = gen.make_weights(spec)
        h = binding.tsvd_pack(U, S, V)
        try:
            U2, S2, V2 = binding.tsvd_unpack(h)
            assert np.array_equal(U, U2) and np.array_equal(V, V2) and np.array_equal(S, S2)
            info = binding.tsvd_info(h)
            assert (info["M"], info["K"], info["N"]) == (M, K, N)
            assert abs(info["density_u"] - np.count_nonzero(U) / U.size) < 1e-12
            assert abs(info["density_v"] - np.count_nonzero(V) / V.size) < 1e-12
            rp = lambda v: (v + 127) // 128 * 128
            assert info["packed_bytes"] == (rp(M) * rp(K) + rp(K) * rp(N)) // 4 + 4 * K
        finally:
            binding.tsvd_destroy(h)


def test_pack_rejects_non_ternary():
    from paper_2308_07641_b200 import binding
    U = np.zeros((4, 4), np.int8); V = np.zeros((4, 4), np.int8); S = np.ones(4, np.float32)
    V[2, 3] = 2
    with pytest.raises(binding.TSVDError) as e:
        binding.tsvd_pack(U, S, V)
    assert e.value.status == binding.TSVD_E_VALUE
    V[2, 3] = 0; U[0, 0] = -2
    with pytest.raises(binding.TSVDError) as e:
        binding.tsvd_pack(U, S, V)
    assert e.value.status == binding.TSVD_E_VALUE


def test_forward_argument_errors():
    import torch
    from paper_2308_07641_b200 import binding
    U = np.zeros((4, 4), np.int8); V = np.zeros((4, 4), np.int8); S = np.ones(4, np.float32)
    h = binding.tsvd_pack(U, S, V)
    try:
        x = torch.zeros(64, device="cuda"); y = torch.zeros(64, device="cuda")
        L = binding.lib()
        assert L.tsvd_forward(h, x.data_ptr(), y.data_ptr(), 0, 0, None) == binding.TSVD_E_SHAPE
        assert L.tsvd_forward(h, x.data_ptr(), y.data_ptr(), 1, 9, None) == binding.TSVD_E_DTYPE
        assert L.tsvd_forward(h, x.data_ptr() + 4, y.data_ptr(), 1, 0, None) == binding.TSVD_E_ALIGN
        assert L.tsvd_forward_ex(h, x.data_ptr(), 3, y.data_ptr(), 4, 1, 0, 0, None, None) == binding.TSVD_E_SHAPE
        assert L.tsvd_forward_ex(h, x.data_ptr(), 4, y.data_ptr(), 4, 1, 0, 0x30, None, None) == binding.TSVD_E_DTYPE
        assert L.tsvd_forward(h, None, y.data_ptr(), 1, 0, None) == binding.TSVD_E_NULL
        assert binding.tsvd_last_status(h) == binding.TSVD_OK
    finally:
        binding.tsvd_destroy(h)


# ---- small cases, every element --------------------------------------------------------------
SMALL = [
    C["cfg1"],
    gen.scaled(C["cfg1"], name="tiny_1x1x1", M=1, N=1, K=1, B=1, density=1.0),
    gen.scaled(C["cfg1"], name="ragged_f32", M=300, N=333, K=200, B=13, seed=11),
    gen.scaled(C["cfg2"], name="cfg2_small", M=384, N=200, K=130, B=70),
    gen.scaled(C["cfg2"], name="ragged_bf16", M=1000, N=345, K=63, B=37, seed=12),
    gen.scaled(C["cfg3_b4"], name="cfg3_small", M=512, N=640, K=384),
    gen.scaled(C["cfg3_b1"], name="cfg3_small_b1", M=512, N=640, K=384),
    gen.scaled(C["cfg4"], name="cfg4_small", M=640, N=256, K=256, B=160),
    gen.scaled(C["cfg5_d05"], name="cfg5_small_d05", M=256, N=384, K=512, B=40),
    gen.scaled(C["cfg5_d20"], name="cfg5_small_d20", M=256, N=384, K=512, B=40),
    gen.scaled(C["cfg5_d50"], name="cfg5_small_d50", M=129, N=257, K=255, B=33),
    gen.scaled(C["cfg2"], name="all_zero", M=140, N=130, K=150, B=9, density=0.0),
    gen.scaled(C["cfg5_d50"], name="all_nonzero_i8", M=140, N=130, K=150, B=9, density=1.0),
    gen.scaled(C["cfg2"], name="row_density_varies", M=260, N=300, K=280, B=20, row_density_spread=0.9),
]


PATHS = {"simple": 0x10, "tensor": 0x40}


@pytest.mark.parametrize("path", sorted(PATHS))
@pytest.mark.parametrize("spec", SMALL, ids=lambda s: s.name)
def test_small_cases_every_element(spec, path):
    _util.run_and_check(spec, flags=PATHS[path])


# ---- decode kernels: one to four tokens ------------------------------------------------------------
DECODE = [
    gen.scaled(C["cfg1"], name="dec_tiny_1x1x1", M=1, N=1, K=1, B=1, density=1.0),
    gen.scaled(C["cfg1"], name="dec_f32_b3", M=300, N=333, K=200, B=3, seed=21),
    gen.scaled(C["cfg1"], name="dec_f32_b1", M=131, N=1100, K=257, B=1, seed=22),
    gen.scaled(C["cfg3_b1"], name="dec_bf16_b1", M=512, N=640, K=384),
    gen.scaled(C["cfg3_b4"], name="dec_bf16_b2", M=520, N=2100, K=390, B=2, seed=23),
    gen.scaled(C["cfg3_b4"], name="dec_bf16_b4", M=512, N=640, K=384),
    gen.scaled(C["cfg5_d20"], name="dec_i8_b4", M=256, N=384, K=512, B=4),
    gen.scaled(C["cfg5_d50"], name="dec_i8_b1_dense", M=129, N=257, K=255, B=1, density=1.0),
    gen.scaled(C["cfg2"], name="dec_all_zero", M=140, N=130, K=150, B=2, density=0.0),
    gen.scaled(C["cfg1"], name="dec_f32_b8", M=300, N=333, K=200, B=8, seed=24),
    gen.scaled(C["cfg3_b4"], name="dec_bf16_b5", M=520, N=2100, K=390, B=5, seed=25),
    gen.scaled(C["cfg3_b4"], name="dec_bf16_b7", M=512, N=640, K=384, B=7, seed=26),
    gen.scaled(C["cfg5_d20"], name="dec_i8_b8", M=256, N=384, K=512, B=8),
    gen.scaled(C["cfg2"], name="dec_row_density_varies", M=260, N=300, K=280, B=4, row_density_spread=0.9),
]


@pytest.mark.parametrize("spec", DECODE, ids=lambda s: s.name)
def test_decode_cases_every_element(spec):
    _util.run_and_check(spec, flags=0x20)


def test_decode_is_the_default_up_to_four_tokens_and_refuses_more_than_eight():
    import torch
    from paper_2308_07641_b200 import binding
    rng = np.random.default_rng(5)
    U = rng.integers(-1, 2, (40, 24)).astype(np.int8); V = rng.integers(-1, 2, (24, 36)).astype(np.int8)
    S = np.ones(24, np.float32)
    h = binding.tsvd_pack(U, S, V)
    try:
        for B in range(1, 9):
            # contractions under 1024 columns: the decode kernels by default up to four tokens, from five on
            # the cluster kernels of the tensor-core path; the decode kernels on request up to eight
            assert binding.tsvd_plan(h, B, binding.TSVD_BF16)["path"] == ("decode" if B <= 4 else "tensor")
            assert binding.tsvd_plan(h, B, binding.TSVD_BF16, 0x20)["path"] == "decode"
            assert binding.tsvd_plan(h, B, binding.TSVD_BF16, 0x40)["path"] == "tensor"
        assert binding.tsvd_plan(h, 9, binding.TSVD_BF16)["path"] == "tensor"
        plan = binding.tsvd_plan(h, 4, binding.TSVD_I8, 0x20)
        assert (plan["path"], plan["digits_x"], plan["digits_t"]) == ("decode", 1, 4)
        x = torch.zeros(9 * 36, device="cuda"); y = torch.zeros(9 * 40, device="cuda")
        L = binding.lib()
        assert L.tsvd_forward_ex(h, x.data_ptr(), 36, y.data_ptr(), 40, 9, 0, 0x20, None, None) == binding.TSVD_E_TOOBIG
        assert L.tsvd_forward_ex(h, x.data_ptr(), 36, y.data_ptr(), 40, 8, 0, 0x20, None, None) == binding.TSVD_OK
        torch.cuda.synchronize()
    finally:
        binding.tsvd_destroy(h)


def test_decode_and_tensor_paths_agree_bit_for_bit():
    """Below 1024 columns both quantise each token with one scale and add exact integers: identical
    outputs.  (From 1024 columns on the decode kernels scale each quarter of the columns on its own.)"""
    import torch
    from paper_2308_07641_b200 import TSVDLinear
    spec = gen.scaled(C["cfg3_b4"], name="agree", M=700, N=700, K=520, B=4, seed=31)
    U, V, S = gen.make_weights(spec)
    x = _util.torch_x(gen.make_x(spec), spec.x_dtype)
    layer = TSVDLinear(U, S, V)
    try:
        y_dec = layer.forward(x, flags=0x20 | 0x1).clone()
        y_ten = layer.forward(x, flags=0x40 | 0x1).clone()
        torch.cuda.synchronize()
        assert torch.equal(y_dec, y_ten)
    finally:
        layer.close()


@pytest.mark.parametrize("B", [1, 2, 3, 4, 6, 8, 9, 12, 16])
@pytest.mark.parametrize("x_dtype,base", [("bf16", "cfg3_b4"), ("f32", "cfg1"), ("i8", "cfg5_d20")])
def test_decode_cluster_form_long_contractions(B, x_dtype, base):
    """From 1024 columns on four CTAs of a cluster split the contraction of a 128-row tile; ragged
    column counts leave the last quarter short, and 17 or 18 column groups do not divide by four."""
    for (M, N, K) in ((300, 1100, 1030), (200, 2300, 1100)):
        spec = gen.scaled(C[base], name=f"cluster_{x_dtype}_B{B}_{N}", M=M, N=N, K=K, B=B, seed=90 + B)
        _util.run_and_check(spec, flags=0x20)


@pytest.mark.parametrize("B", [1, 2, 4, 7])
@pytest.mark.parametrize("x_dtype,base", [("bf16", "cfg3_b4"), ("i8", "cfg5_d20")])
def test_decode_contractions_longer_than_one_round(B, x_dtype, base):
    """More than 4096 columns: a warp of the single-CTA kernel, and more than 4096 columns per quarter a
    warp of the cluster form, comes back for further rounds of column groups (codes requested one round
    ahead).  9000 columns = 142 groups (three rounds; quarters of 36, 36, 36, 34), 17000 columns per
    quarter more than one round as well."""
    for (M, N, K) in ((150, 9000, 140), (140, 17000, 130)):
        spec = gen.scaled(C[base], name=f"rounds_{x_dtype}_B{B}_{N}", M=M, N=N, K=K, B=B, seed=120 + B, density=0.1)
        _util.run_and_check(spec, flags=0x20)


def test_decode_cluster_form_runs_back_to_back_and_is_deterministic():
    import torch
    from paper_2308_07641_b200 import TSVDLinear
    spec = gen.scaled(C["cfg3_b4"], name="cluster_repeat", M=1000, N=4096, K=2048, B=4, seed=97)
    U, V, S = gen.make_weights(spec)
    x = _util.torch_x(gen.make_x(spec), "bf16")
    layer = TSVDLinear(U, S, V)
    try:
        ys = [layer.forward(x, flags=0x20 | 0x1).clone() for _ in range(6)]
        torch.cuda.synchronize()
        assert all(torch.equal(ys[0], y) for y in ys[1:])
    finally:
        layer.close()


def test_decode_strided_inputs_and_host_entry_point():
    """Row strides larger than the row, fp32 output of bf16 activations, and the host-buffer call."""
    import torch
    from paper_2308_07641_b200 import TSVDLinear, binding
    spec = gen.scaled(C["cfg3_b4"], name="dec_strided", M=260, N=333, K=200, B=3, seed=41)
    U, V, S = gen.make_weights(spec)
    x_np = gen.make_x(spec)
    ref = oracle.forward(U, S, V, _util.oracle_x(x_np, "bf16"))
    layer = TSVDLinear(U, S, V)
    try:
        x = _util.torch_x(x_np, "bf16")
        xs = torch.zeros((spec.B, spec.N + 7), dtype=torch.bfloat16, device="cuda")
        xs[:, :spec.N] = x
        out = torch.full((spec.B, spec.M + 5), 7.0, dtype=torch.float32, device="cuda")
        layer.forward(xs[:, :spec.N], out=out[:, :spec.M], flags=0x20 | 0x1)
        torch.cuda.synchronize()
        assert float(out[:, spec.M:].min()) == 7.0 and float(out[:, spec.M:].max()) == 7.0
        _util.check_outputs(out[:, :spec.M].double().cpu().numpy(), None, ref, "bf16", False, "strided decode")
        # host buffers: the library copies in and out itself (default path for 3 tokens = decode)
        y_host = np.zeros((spec.B, spec.M), np.float32)
        binding.tsvd_forward_host(layer.handle, x_np.ctypes.data, y_host.ctypes.data, spec.B, binding.TSVD_BF16, 0x1)
        _util.check_outputs(y_host.astype(np.float64), None, ref, "bf16", False, "host decode")
    finally:
        layer.close()


def test_kernels_launched_early_still_see_inputs_written_just_before():
    """The kernels may start while the kernel before them in the stream still runs; they must not
    read their input before it has completed.  x is doubled in place between two forwards: every
    digit stays the same and only the per-token exponent moves, so y doubles exactly."""
    import torch
    from paper_2308_07641_b200 import TSVDLinear
    for B in (2, 40, 200):          # decode, small-batch and large-batch kernels
        spec = gen.scaled(C["cfg2"], name=f"pdl_B{B}", M=600, N=1500, K=520, B=B, seed=61)
        U, V, S = gen.make_weights(spec)
        x = _util.torch_x(gen.make_x(spec), "bf16").float()
        layer = TSVDLinear(U, S, V)
        try:
            y1 = layer.forward(x).clone()
            for _ in range(5):
                x.mul_(2.0)
                y = layer.forward(x)
                y1.mul_(2.0)
                assert torch.equal(y, y1)
            torch.cuda.synchronize()
        finally:
            layer.close()


def test_decode_falls_back_when_the_digits_do_not_fit_shared_memory():
    from paper_2308_07641_b200 import binding
    N = 13000                       # 2 tokens x 4 digits x 13056 columns fit 200 KiB; so do 4 and 8 tokens on a quarter each
    U = np.zeros((8, 8), np.int8); V = np.zeros((8, N), np.int8); S = np.ones(8, np.float32)
    h = binding.tsvd_pack(U, S, V)
    try:
        for B in (1, 2, 4, 8):
            assert binding.tsvd_plan(h, B, binding.TSVD_F32)["path"] == "decode"
    finally:
        binding.tsvd_destroy(h)
    N = 40000                       # 40064 padded columns x 4 digits: one token fits; two and four on a quarter each (cluster form); eight do not
    V = np.zeros((8, N), np.int8)
    h = binding.tsvd_pack(U, S, V)
    try:
        assert binding.tsvd_plan(h, 1, binding.TSVD_F32)["path"] == "decode"
        assert binding.tsvd_plan(h, 2, binding.TSVD_F32)["path"] == "decode"
        assert binding.tsvd_plan(h, 4, binding.TSVD_F32)["path"] == "decode"
        assert binding.tsvd_plan(h, 8, binding.TSVD_F32)["path"] == "tensor"
        with pytest.raises(binding.TSVDError) as ei:
            binding.tsvd_plan(h, 8, binding.TSVD_F32, 0x20)
        assert ei.value.status == binding.TSVD_E_TOOBIG
    finally:
        binding.tsvd_destroy(h)


def test_out_f32_flag_and_strides():
    """bf16 activations with fp32 output, and leading dimensions larger than the row length."""
    import torch
    from paper_2308_07641_b200 import TSVDLinear, TSVD_FLAG_OUT_F32
    spec = gen.scaled(C["cfg2"], name="strided", M=200, N=150, K=170, B=11, seed=21)
    U, V, S = gen.make_weights(spec)
    x = gen.make_x(spec)
    layer = TSVDLinear(U, S, V)
    try:
        xt = _util.torch_x(x, "bf16")
        xbig = torch.zeros((spec.B, spec.N + 10), dtype=torch.bfloat16, device="cuda")
        xbig[:, :spec.N] = xt
        ybig = torch.full((spec.B, spec.M + 24), 7.0, dtype=torch.float32, device="cuda")
        layer.forward(xbig[:, :spec.N], out=ybig[:, :spec.M], flags=TSVD_FLAG_OUT_F32)
        torch.cuda.synchronize()
        ref = oracle.forward(U, S, V, _util.oracle_x(x, "bf16"))
        y = ybig[:, :spec.M].double().cpu().numpy()
        assert np.abs(y - ref.y).max() <= 1e-5 * np.abs(ref.y).max()
        assert torch.all(ybig[:, spec.M:] == 7.0)          # padding untouched
    finally:
        layer.close()


def test_repeatable_and_handle_reuse():
    """Two calls on one handle with different batch sizes; int32 z identical run to run."""
    import torch
    from paper_2308_07641_b200 import TSVDLinear
    spec = gen.scaled(C["cfg5_d20"], name="reuse", M=200, N=300, K=260, B=50)
    U, V, S = gen.make_weights(spec)
    x = gen.make_x(spec)
    layer = TSVDLinear(U, S, V)
    try:
        y1, z1, _ = _util.run_gpu(layer, x[:7], "i8")
        y2, z2, _ = _util.run_gpu(layer, x, "i8")
        y3, z3, _ = _util.run_gpu(layer, x, "i8")
        assert np.array_equal(z2, z3) and np.array_equal(z1, z2[:7])
        ref = oracle.forward(U, S, V, x)
        _util.check_outputs(y2, z2, ref, "i8", False, "reuse")
        assert np.abs(y1 - y2[:7]).max() <= 1e-5 * np.abs(ref.y).max()
    finally:
        layer.close()


def test_host_buffer_entry_point():
    from paper_2308_07641_b200 import binding
    spec = gen.scaled(C["cfg1"], name="host", M=100, N=90, K=80, B=5, seed=31)
    U, V, S = gen.make_weights(spec)
    x = gen.make_x(spec)
    h = binding.tsvd_pack(U, S, V)
    try:
        y = np.zeros((spec.B, spec.M), np.float32)
        z = np.zeros((spec.B, spec.K), np.float32)
        binding.tsvd_forward_host(h, x.ctypes.data, y.ctypes.data, spec.B, binding.TSVD_F32, 0, z.ctypes.data)
        ref = oracle.forward(U, S, V, x.astype(np.float64))
        _util.check_outputs(y.astype(np.float64), z, ref, "f32", False, "host")
    finally:
        binding.tsvd_destroy(h)


def test_host_buffer_entry_point_pipelined_chunks():
    """768 tokens and more go through the host entry point in chunks on three streams; every token
    (and z) must come back as from one forward.  Pinned and pageable host buffers."""
    import torch
    from paper_2308_07641_b200 import binding
    spec = gen.scaled(C["cfg2"], name="host_chunks", M=300, N=200, K=150, B=1000, seed=33)
    U, V, S = gen.make_weights(spec)
    x = gen.make_x(spec)
    ref = oracle.forward(U, S, V, _util.oracle_x(x, "bf16"))
    h = binding.tsvd_pack(U, S, V)
    try:
        y = np.zeros((spec.B, spec.M), np.float32)
        z = np.zeros((spec.B, spec.K), np.float32)
        binding.tsvd_forward_host(h, x.ctypes.data, y.ctypes.data, spec.B, binding.TSVD_BF16, 0x1, z.ctypes.data)
        _util.check_outputs(y.astype(np.float64), z, ref, "bf16", False, "host, pageable")
        xp = torch.from_numpy(x.view(np.int16)).pin_memory()
        yp = torch.zeros((spec.B, spec.M), dtype=torch.int16).pin_memory()
        for _ in range(2):
            binding.tsvd_forward_host(h, xp.data_ptr(), yp.data_ptr(), spec.B, binding.TSVD_BF16, 0)
        y16 = yp.view(torch.bfloat16).float().double().numpy()
        _util.check_outputs(y16, None, ref, "bf16", True, "host, pinned")
        assert binding.tsvd_last_status(h) == binding.TSVD_OK
    finally:
        binding.tsvd_destroy(h)


# ---- full-size configurations: every token (None) where the checker needs seconds, else sampled token
#      columns (cfg4 is also compared on 130 tokens with the numeric edge cases) -------------------
FULL = [
    (C["cfg2"], None),
    (C["cfg3_b1"], None),
    (C["cfg3_b4"], None),
    (C["cfg3_b16"], None),
    (C["cfg4"], [0, 1023, 2047]),
    (C["cfg5_d05"], [0, 100, 255]),
    (C["cfg5_d20"], None),
    (C["cfg5_d50"], [0, 100, 255]),
]


@pytest.mark.parametrize("spec,sample", FULL, ids=lambda v: v.name if hasattr(v, "name") else None)
def test_full_size_sampled(spec, sample):
    _util.run_and_check(spec, sample_tokens=sample)


@pytest.mark.parametrize("B", [200, 20], ids=["tile_kernels", "cluster_kernels"])
def test_bounded_wait_gives_up_and_reports_timeout(B):
    """Failure detection without a fault: a forward whose digits are withheld (test hook: by the copy
    producer of the tile kernels, by the converting warps of the cluster kernels) must end by itself,
    report TSVD_E_TIMEOUT through the handle's status word, and leave the context and the handle usable
    for a correct forward right after."""
    import time
    import torch
    from paper_2308_07641_b200 import TSVDLinear, binding
    spec = gen.scaled(C["cfg2"], name="stall", M=256, N=256, K=256, B=B, seed=41)
    U, V, S = gen.make_weights(spec)
    x = gen.make_x(spec)
    layer = TSVDLinear(U, S, V)
    try:
        xt = _util.torch_x(x, "bf16")
        assert binding.tsvd_last_status(layer.handle) == binding.TSVD_OK
        t0 = time.perf_counter()
        layer.forward(xt, flags=binding.TSVD_FLAG_TEST_STALL)
        torch.cuda.synchronize()
        assert time.perf_counter() - t0 < 5.0                      # bounded, not the default 2 s per wait chain
        assert binding.tsvd_last_status(layer.handle) == binding.TSVD_E_TIMEOUT
        assert binding.tsvd_last_status(layer.handle) == binding.TSVD_OK   # reading resets the word
        y64, z, y_bf16 = _util.run_gpu(layer, x, "bf16")
        ref = oracle.forward(U, S, V, _util.oracle_x(x, "bf16"))
        _util.check_outputs(y64, z, ref, "bf16", y_bf16, "after a timed-out forward")
        assert binding.tsvd_last_status(layer.handle) == binding.TSVD_OK
    finally:
        layer.close()


@pytest.mark.parametrize("B", [63, 64, 65, 128])
def test_batch_sizes_around_the_small_batch_switch(B):
    """Up to 64 tokens the tile kernels run one (padded) token tile per row tile unless the split form is
    estimated faster (not here: short contractions); beyond 64 always the tile kernels."""
    spec = gen.scaled(C["cfg2"], name=f"switch_B{B}", M=300, N=520, K=390, B=B, seed=51)
    _util.run_and_check(spec)


def test_split_form_with_one_stage_unsplit():
    """Few row tiles on a long contraction: the split form (U-stage: 4 row tiles x 2 token tiles, 16 parts
    each); its V-stage has 128 output tiles, about one per SM, and is not split (every part is the last one)."""
    spec = gen.scaled(C["cfg5_d20"], name="unsplit", M=512, N=8192, K=8192, B=20, seed=52, density=0.05)
    _util.run_and_check(spec, sample_tokens=[0, 8, 16, 19])


@pytest.mark.parametrize("B", [385, 400, 448])
@pytest.mark.parametrize("x_dtype,base", [("bf16", "cfg2"), ("f32", "cfg1"), ("i8", "cfg5_d20")])
def test_u_stage_in_one_round_of_256_column_tiles(B, x_dtype, base):
    """20 row tiles x 9 or 10 token tiles of 48 are more tiles than SMs, 20 x 7 of 64 tokens are not: the
    U-stage then runs tiles of 256 columns on one accumulator buffer (ragged last tile at 385 and 400)."""
    spec = gen.scaled(C[base], name=f"wide_u_{x_dtype}_B{B}", M=2560 - 7, N=330, K=1300, B=B, seed=53)
    _util.run_and_check(spec, sample_tokens=[0, 1, 47, 48, 63, 64, 191, 192, B - 2, B - 1])


@pytest.mark.parametrize("B", [100, 128, 200, 256, 300])
def test_int8_v_stage_in_tiles_of_128_tokens(B):
    """int8 activations: 128-token tiles where they leave fewer padded tokens than 192-token ones (z bit-exact)."""
    spec = gen.scaled(C["cfg5_d20"], name=f"narrow_i8_B{B}", M=200, N=1500, K=700, B=B, seed=54)
    _util.run_and_check(spec)


@pytest.mark.parametrize("B", [65, 100, 192, 300, 512])
@pytest.mark.parametrize("x_dtype,base", [("bf16", "cfg2"), ("f32", "cfg1"), ("i8", "cfg5_d20")])
def test_split_form_beyond_64_tokens(B, x_dtype, base):
    """Two row tiles in each stage and a contraction of 20000 columns: the split form is preferred up to 512
    tokens (16-token tiles, up to sixteen parts per tile, integer atomics, last-arriver tail)."""
    spec = gen.scaled(C[base], name=f"split_{x_dtype}_B{B}", M=200, N=20000, K=250, B=B, seed=55, density=0.05)
    _util.run_and_check(spec, sample_tokens=[0, 15, 16, B // 2, B - 1])


@pytest.mark.parametrize("B", [385, 448])
@pytest.mark.parametrize("x_dtype,base,flags", [("f32", "cfg1", 0), ("bf16", "cfg2", 0x200)])
def test_four_digit_v_stage_in_one_round_of_256_column_tiles(B, x_dtype, base, flags):
    """fp32 activations (or bf16 with four digits): 20 row tiles of V x 9 or 10 token tiles of 48 are more
    tiles than SMs, 20 x 7 of 64 tokens are not: the V-stage, too, then runs tiles of 256 columns."""
    spec = gen.scaled(C[base], name=f"wide_v_{x_dtype}_B{B}", M=300, N=1300, K=2560 - 9, B=B, seed=56)
    _util.run_and_check(spec, flags=flags, sample_tokens=[0, 47, 48, 63, 64, 191, 192, B - 1])


@pytest.mark.parametrize("B,N", [(1, 60000), (2, 40000), (2, 65280)])
def test_decode_one_and_two_tokens_on_rows_too_long_for_one_cta(B, N):
    """fp32 activations, four digits: the digits of a whole row exceed a CTA's shared memory, a quarter fits:
    the cluster form serves one and two tokens as well."""
    from paper_2308_07641_b200 import binding
    spec = gen.scaled(C["cfg1"], name=f"long_row_B{B}_{N}", M=200, N=N, K=300, B=B, seed=57, density=0.02)
    res = _util.run_and_check(spec, flags=0x20)
    assert res["status"] in (0, 10)
