"""GPU parity at the numeric edges of the fixed-point arithmetic, element by element against the
CPU checker at the stated tolerances, on every kernel family:

  tensor  (B > 64: 192-column tiles)      small  (5..64 tokens: split contraction)
  decode  (1..16 tokens)                  index  (1..4 tokens, index lists)      simple (CUDA cores)

Cases: S with negative, zero and widely spread entries (S comes from a pseudo-inverse, Eq. 4);
tokens with outliers 2^8 .. 2^20 above their bulk; an all-zero token inside a batch; int8
activations containing -128; fp32 activations scaled by 2^-100 and 2^100; a bias.  Where the
documented range of the arithmetic is left (bf16 outliers from 2^12 up) the forward must say so
through TSVD_E_RANGE, and the wide form (TSVD_FLAG_WIDE_X) and the CUDA-core path must still
meet the tolerance.
"""
import numpy as np
import pytest

import gen
import oracle
from tests import _util

pytestmark = pytest.mark.gpu

C = gen.CONFIGS
OK, RANGE = 0, 10
SIMPLE, DECODE, TENSOR, INDEX, WIDE = 0x10, 0x20, 0x40, 0x80, 0x200

# (family name, forced path flag, batch, tsvd_pack flags)
# "small": 23 tokens on the cluster kernels of the tensor-core path; "split": 22 tokens on a contraction too long
# for them (8300 columns), i.e. the 16-token tiles with the contraction split over CTAs
FAMILIES = [("tensor", TENSOR, 150, 0), ("small", TENSOR, 23, 0), ("split", TENSOR, 22, 0), ("decode", DECODE, 3, 0),
            ("decode8", DECODE, 7, 0), ("decode16", DECODE, 13, 0), ("index", INDEX, 4, 1), ("simple", SIMPLE, 11, 0)]
# the outlier cases below are sized for contractions of about 1100 columns (the error of the sums grows with
# the square root of the nonzeros per row): not the split family's 8300
FAST = [f for f in FAMILIES if f[0] not in ("simple", "split")]


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2308_07641_b200 import build
    build.build()


def _spec(base, name, B, **kw):
    kw.setdefault("M", 520)
    kw.setdefault("N", 1100)
    kw.setdefault("K", 650)
    if B == 13:       # the decode16 family: nine to sixteen tokens need 1024+ columns in both stages
        kw["N"], kw["K"] = max(kw["N"], 1100), max(kw["K"], 1030)
    if B == 22:       # the split family: a contraction of more than 64 blocks of 128 columns
        kw["N"] = max(kw["N"], 8300)
    return gen.scaled(C[base], name=name, B=B, **kw)


def _signed_S(S, seed, lo_exp, hi_exp):
    """Unsorted S with both signs, exact zeros and magnitudes log-uniform over 10^lo .. 10^hi."""
    g = np.random.default_rng(seed)
    out = (10.0 ** g.uniform(lo_exp, hi_exp, S.size) * g.choice([-1.0, 1.0], S.size)).astype(np.float32)
    out[g.random(S.size) < 0.15] = 0.0
    return out


# ---- (a) S from a pseudo-inverse: any sign, zeros, unsorted, many decades -----------------------
@pytest.mark.parametrize("fam", FAMILIES, ids=lambda f: f[0])
@pytest.mark.parametrize("x_dtype,base", [("bf16", "cfg2"), ("f32", "cfg1"), ("i8", "cfg5_d20")])
def test_signed_zero_and_spread_S(fam, x_dtype, base):
    name, flag, B, pack = fam
    spec = _spec(base, f"S_signed_{name}_{x_dtype}", B, seed=301, density=0.2)
    U, V, S = gen.make_weights(spec)
    _util.run_and_check(spec, flags=flag, pack_flags=pack, weights=(U, V, _signed_S(S, 1, -1.5, 1.5)), expect_status=OK)


@pytest.mark.parametrize("fam", FAMILIES, ids=lambda f: f[0])
@pytest.mark.parametrize("x_dtype,base", [("bf16", "cfg2"), ("f32", "cfg1")])
def test_S_over_twelve_decades(fam, x_dtype, base):
    """|S| from 1e-6 to 1e6: the rank components below 2^-18 of a token's largest |t| are not resolved
    (the status word may say so); every output still meets the tolerance because every output row
    sees some of the large components."""
    name, flag, B, pack = fam
    spec = _spec(base, f"S_wide_{name}_{x_dtype}", B, seed=302, density=0.25)
    U, V, S = gen.make_weights(spec)
    _util.run_and_check(spec, flags=flag, pack_flags=pack, weights=(U, V, _signed_S(S, 2, -6, 6)), expect_status=(OK, RANGE))


# ---- (b) outliers ------------------------------------------------------------------------------
def _with_outliers(spec, p):
    """Every token gets 2^p at one column and every second token -2^p at another."""
    x = gen.make_x(spec)
    x = gen.set_entries(x, spec.x_dtype, np.arange(spec.B), [5], 2.0 ** p)
    return gen.set_entries(x, spec.x_dtype, np.arange(0, spec.B, 2), [77], -(2.0 ** p))


@pytest.mark.parametrize("fam", FAST, ids=lambda f: f[0])
@pytest.mark.parametrize("density", [0.2, 0.05])
def test_bf16_outliers_inside_the_documented_range(fam, density):
    """Outliers 2^8 above a unit-scale bulk: inside the range of three digits; status stays OK."""
    name, flag, B, pack = fam
    spec = _spec("cfg2", f"outlier8_{name}_{density}", B, seed=303, density=density)
    _util.run_and_check(spec, flags=flag, pack_flags=pack, x=_with_outliers(spec, 8), expect_status=OK)


@pytest.mark.parametrize("fam", FAST, ids=lambda f: f[0])
@pytest.mark.parametrize("p", [12, 16])
@pytest.mark.parametrize("density", [0.2, 0.05])
def test_bf16_outliers_beyond_three_digits_are_reported_and_the_wide_form_serves_them(fam, p, density):
    import torch
    from paper_2308_07641_b200 import TSVDLinear, binding
    name, flag, B, pack = fam
    spec = _spec("cfg2", f"outlier{p}_{name}_{density}", B, seed=304, density=density)
    U, V, S = gen.make_weights(spec)
    x = _with_outliers(spec, p)
    # three digits: the forward completes and says that the range was exceeded
    layer = TSVDLinear(U, S, V, pack)
    try:
        layer.forward(_util.torch_x(x, "bf16"), flags=flag)
        torch.cuda.synchronize()
        assert binding.tsvd_last_status(layer.handle) == binding.TSVD_E_RANGE
        assert binding.tsvd_last_status(layer.handle) == binding.TSVD_OK      # reading resets it
    finally:
        layer.close()
    # four digits: within tolerance, nothing to report
    _util.run_and_check(spec, flags=flag | WIDE, pack_flags=pack, weights=(U, V, S), x=x, expect_status=OK)


@pytest.mark.parametrize("p", [12, 20])
@pytest.mark.parametrize("density", [0.2, 0.05])
def test_bf16_outliers_on_the_cuda_core_path(p, density):
    """fp32 partial sums over the nonzeros only: no dynamic-range limit, nothing reported."""
    spec = _spec("cfg2", f"outlier{p}_simple_{density}", 11, seed=305, density=density)
    _util.run_and_check(spec, flags=SIMPLE, x=_with_outliers(spec, p), expect_status=OK)


@pytest.mark.parametrize("fam", FAST, ids=lambda f: f[0])
@pytest.mark.parametrize("p", [8, 12, 16, 20])
def test_f32_outliers(fam, p):
    """fp32 outputs are compared in the maximum norm, which the outliers set; 30 bits of the token's
    range are far inside it.  From 2^18 up the bulk keeps fewer than 12 bits and the status says so."""
    name, flag, B, pack = fam
    spec = _spec("cfg1", f"f32_outlier{p}_{name}", B, seed=306, density=0.05)
    _util.run_and_check(spec, flags=flag, pack_flags=pack, x=_with_outliers(spec, p),
                        expect_status=OK if p <= 16 else RANGE)


# ---- (c) an all-zero token inside a batch, (d) int8 -128, (e) extreme scales ----------------------
@pytest.mark.parametrize("fam", FAMILIES, ids=lambda f: f[0])
@pytest.mark.parametrize("x_dtype,base", [("bf16", "cfg2"), ("f32", "cfg1"), ("i8", "cfg5_d20")])
def test_all_zero_token_inside_a_batch(fam, x_dtype, base):
    name, flag, B, pack = fam
    spec = _spec(base, f"zero_token_{name}_{x_dtype}", B, seed=307, density=0.2)
    x = gen.make_x(spec)
    x = gen.set_entries(x, x_dtype, [1, B - 1], np.arange(spec.N), 0.0)
    res = _util.run_and_check(spec, flags=flag, pack_flags=pack, x=x, expect_status=OK)
    assert res is not None


@pytest.mark.parametrize("fam", FAMILIES, ids=lambda f: f[0])
def test_int8_minus_128(fam):
    name, flag, B, pack = fam
    spec = _spec("cfg5_d50", f"i8_min_{name}", B, seed=308, density=0.5)
    x = gen.make_x(spec)
    x = gen.set_entries(x, "i8", np.arange(B), np.arange(0, spec.N, 3), -128)
    x = gen.set_entries(x, "i8", [0], np.arange(spec.N), -128)          # one token of nothing but -128
    _util.run_and_check(spec, flags=flag, pack_flags=pack, x=x, expect_status=OK)


@pytest.mark.parametrize("fam", FAMILIES, ids=lambda f: f[0])
@pytest.mark.parametrize("e", [-100, 100])
def test_f32_extreme_scales(fam, e):
    """2^-100 lies below the floor of the scaling rule (2^-90): ten bits are lost, 20 remain."""
    name, flag, B, pack = fam
    spec = _spec("cfg1", f"f32_scale{e}_{name}", B, seed=309, density=0.2, s_dist="lognormal")
    x = np.ldexp(gen.make_x(spec), e).astype(np.float32)
    _util.run_and_check(spec, flags=flag, pack_flags=pack, x=x, expect_status=(OK, RANGE) if e < 0 else OK)


def test_mixed_token_scales_in_one_batch():
    """Per-token scaling: tokens 2^-40 .. 2^40 apart in one batch do not disturb one another."""
    spec = _spec("cfg2", "mixed_scales", 150, seed=310, density=0.2)
    x = _util.oracle_x(gen.make_x(spec), "bf16")
    x = x * np.ldexp(1.0, (np.arange(spec.B) % 9 - 4) * 10)[:, None]
    xb = gen.rng.f32_to_bf16_bits(x.astype(np.float32))     # exact: powers of two
    from paper_2308_07641_b200 import TSVD_FLAG_OUT_F32
    U, V, S = gen.make_weights(spec)
    # per-token comparison (the maximum norm of the whole batch would hide the small tokens)
    from paper_2308_07641_b200 import TSVDLinear
    layer = TSVDLinear(U, S, V)
    try:
        y64, _, _ = _util.run_gpu(layer, xb, "bf16", TSVD_FLAG_OUT_F32, want_z=False)
    finally:
        layer.close()
    ref = oracle.forward(U, S, V, _util.oracle_x(xb, "bf16")).y
    for b in range(spec.B):
        assert np.abs(y64[b] - ref[b]).max() <= 1e-5 * np.abs(ref[b]).max(), b


# ---- bias ----------------------------------------------------------------------------------------
@pytest.mark.parametrize("fam", FAMILIES, ids=lambda f: f[0])
@pytest.mark.parametrize("x_dtype,base", [("bf16", "cfg2"), ("f32", "cfg1"), ("i8", "cfg5_d20")])
def test_bias(fam, x_dtype, base):
    name, flag, B, pack = fam
    spec = _spec(base, f"bias_{name}_{x_dtype}", B, seed=311, density=0.2, M=300, N=333, K=200)
    scale = {"bf16": 50.0, "f32": 5.0, "i8": 2000.0}[x_dtype]        # comparable to |y|
    bias = (scale * gen.rng.normal(311, 9, spec.M)).astype(np.float32)
    _util.run_and_check(spec, flags=flag, pack_flags=pack, bias=bias, expect_status=OK)


def test_bias_can_be_replaced_and_removed():
    from paper_2308_07641_b200 import TSVDLinear
    spec = _spec("cfg1", "bias_swap", 9, seed=312, M=140, N=130, K=150)
    U, V, S = gen.make_weights(spec)
    x = gen.make_x(spec)
    b1 = gen.rng.normal(1, 9, spec.M).astype(np.float32)
    b2 = gen.rng.normal(2, 9, spec.M).astype(np.float32)
    layer = TSVDLinear(U, S, V)
    try:
        for bias in (b1, b2, None, b1):
            layer.set_bias(bias)
            y64, _, _ = _util.run_gpu(layer, x, "f32", want_z=False)
            ref = oracle.forward(U, S, V, x.astype(np.float64), bias)
            _util.check_outputs(y64, None, ref, "f32", False, "bias swap")
    finally:
        layer.close()


# ---- (f) the largest configuration on 128+ tokens ---------------------------------------------------
def test_cfg4_on_many_tokens_across_tile_boundaries():
    """cfg4 (16384 x 4096 x 4096, 2048 tokens): the V-stage works on 64-token tiles, the U-stage on
    48-token tiles whose last one is ragged (2048 = 42 * 48 + 32).  First and last token of tiles of
    both kinds, the ragged tail, and a spread of others: 136 tokens, every output of each."""
    edges = [0, 1, 47, 48, 63, 64, 95, 96, 127, 128, 191, 192, 1007, 1008, 1023, 1024,
             1967, 1968, 1983, 1984, 2015, 2016, 2017, 2046, 2047]
    g = np.random.default_rng(4)
    rest = sorted(set(int(v) for v in g.choice(2048, 140, replace=False)) - set(edges))[:136 - len(edges)]
    sample = sorted(edges + rest)
    assert len(sample) >= 128
    _util.run_and_check(C["cfg4"], sample_tokens=sample, expect_status=OK)


def test_reserve_sizes_the_scratch_once():
    """After tsvd_reserve no forward of at most that many tokens allocates: device memory in use
    stays flat over forwards of every batch regime and path."""
    import torch
    from paper_2308_07641_b200 import TSVDLinear
    spec = _spec("cfg2", "reserve", 300, seed=313)
    U, V, S = gen.make_weights(spec)
    x = _util.torch_x(gen.make_x(spec), "bf16")
    layer = TSVDLinear(U, S, V)
    try:
        layer.reserve(300, "bf16")
        y = torch.empty((300, spec.M), dtype=torch.bfloat16, device="cuda")
        # a first use of each kernel family lets the CUDA runtime load its code (lazy module loading,
        # which takes device memory of its own); the library's scratch is what is compared afterwards
        for B, flags in ((300, 0), (2, 0), (6, 0), (40, 0), (5, SIMPLE)):
            layer.forward(x[:B], out=y[:B], flags=flags)
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        for B in (300, 1, 4, 5, 64, 65, 200):
            for flags in (0, WIDE, SIMPLE, TENSOR):
                layer.forward(x[:B], out=y[:B], flags=flags)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert free1 == free0
    finally:
        layer.close()


def test_reserve_covers_both_forms_of_the_tensor_core_path():
    """Two row tiles per stage and a contraction of 20000 columns: batches of up to 512 tokens take the
    split-contraction form, whose scratch per token is the larger one; after tsvd_reserve(300) no batch up
    to 300 tokens allocates on either form."""
    import torch
    from paper_2308_07641_b200 import TSVDLinear
    spec = gen.scaled(C["cfg2"], name="reserve_split", M=200, N=20000, K=250, B=300, seed=314, density=0.05)
    U, V, S = gen.make_weights(spec)
    x = _util.torch_x(gen.make_x(spec), "bf16")
    layer = TSVDLinear(U, S, V)
    try:
        layer.reserve(300, "bf16")
        y = torch.empty((300, spec.M), dtype=torch.bfloat16, device="cuda")
        for B, flags in ((300, 0), (2, 0), (6, 0), (40, 0), (5, SIMPLE)):     # (lazy module loading, as above)
            layer.forward(x[:B], out=y[:B], flags=flags)
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        for B in (300, 192, 100, 65, 64, 20, 5, 1):
            for flags in (0, WIDE, TENSOR):
                layer.forward(x[:B], out=y[:B], flags=flags)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert free1 == free0
    finally:
        layer.close()
