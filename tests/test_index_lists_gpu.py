"""Index-list form for very sparse rows: the same map, U and V stored as lists of their nonzeros
(tsvd_pack with TSVD_PACK_INDEX_LISTS, forward with TSVD_FLAG_PATH_INDEX), against the CPU checker."""
from __future__ import annotations

import numpy as np
import pytest

import gen
from tests import _util

pytestmark = pytest.mark.gpu
C = gen.CONFIGS
INDEX, LISTS = 0x80, 0x1

CASES = [
    gen.scaled(C["cfg1"], name="idx_tiny_1x1x1", M=1, N=1, K=1, B=1, density=1.0),
    gen.scaled(C["cfg1"], name="idx_f32_b3", M=300, N=333, K=200, B=3, density=0.05, seed=71),
    gen.scaled(C["cfg1"], name="idx_f32_b1", M=131, N=1100, K=257, B=1, density=0.1, seed=72),
    gen.scaled(C["cfg3_b1"], name="idx_bf16_b1", M=512, N=640, K=384, density=0.05),
    gen.scaled(C["cfg3_b4"], name="idx_bf16_b2", M=520, N=2100, K=390, B=2, density=0.02, seed=73),
    gen.scaled(C["cfg3_b4"], name="idx_bf16_b4", M=1024, N=4096, K=1024, density=0.05),
    gen.scaled(C["cfg5_d05"], name="idx_i8_b4", M=256, N=384, K=512, B=4),
    gen.scaled(C["cfg5_d50"], name="idx_i8_b1_dense", M=129, N=257, K=255, B=1, density=1.0),
    gen.scaled(C["cfg2"], name="idx_all_zero", M=140, N=130, K=150, B=2, density=0.0),
    gen.scaled(C["cfg2"], name="idx_row_density_varies", M=260, N=300, K=280, B=4, density=0.1, row_density_spread=0.9),
]


@pytest.mark.parametrize("spec", CASES, ids=lambda s: s.name)
def test_index_list_cases_every_element(spec):
    _util.run_and_check(spec, flags=INDEX, pack_flags=LISTS)


def test_index_lists_are_on_request_only_and_sized_by_the_nonzeros():
    import torch
    from paper_2308_07641_b200 import binding
    rng = np.random.default_rng(7)
    U = (rng.integers(-1, 2, (40, 24)) * (rng.random((40, 24)) < 0.2)).astype(np.int8)
    V = (rng.integers(-1, 2, (24, 36)) * (rng.random((24, 36)) < 0.2)).astype(np.int8)
    S = np.ones(24, np.float32)
    plain = binding.tsvd_pack(U, S, V)
    lists = binding.tsvd_pack(U, S, V, LISTS)
    try:
        assert binding.tsvd_index_bytes(plain) == (0, 0)
        assert binding.tsvd_index_bytes(lists) == (4 * 25 + 2 * int(np.count_nonzero(V)), 4 * 41 + 2 * int(np.count_nonzero(U)))
        assert binding.tsvd_plan(lists, 2, binding.TSVD_BF16)["path"] == "decode"          # never the default
        assert binding.tsvd_plan(lists, 2, binding.TSVD_BF16, INDEX)["path"] == "index"
        for h, B in ((plain, 2), (lists, 5)):                                              # no lists / too many tokens
            with pytest.raises(binding.TSVDError) as ei:
                binding.tsvd_plan(h, B, binding.TSVD_BF16, INDEX)
            assert ei.value.status == binding.TSVD_E_TOOBIG
        x = torch.zeros(5 * 36, device="cuda"); y = torch.zeros(5 * 40, device="cuda")
        L = binding.lib()
        assert L.tsvd_forward_ex(plain, x.data_ptr(), 36, y.data_ptr(), 40, 2, 0, INDEX, None, None) == binding.TSVD_E_TOOBIG
        assert L.tsvd_forward_ex(lists, x.data_ptr(), 36, y.data_ptr(), 40, 2, 0, INDEX | 0x20, None, None) == binding.TSVD_E_DTYPE
        assert L.tsvd_forward_ex(lists, x.data_ptr(), 36, y.data_ptr(), 40, 2, 0, INDEX, None, None) == binding.TSVD_OK
        torch.cuda.synchronize()
    finally:
        binding.tsvd_destroy(plain)
        binding.tsvd_destroy(lists)


def test_index_lists_refuse_more_columns_than_an_entry_can_address():
    from paper_2308_07641_b200 import binding
    N = binding.TSVD_INDEX_MAX_COLUMNS + 1
    U = np.zeros((2, 2), np.int8); V = np.zeros((2, N), np.int8); S = np.ones(2, np.float32)
    with pytest.raises(binding.TSVDError) as ei:
        binding.tsvd_pack(U, S, V, LISTS)
    assert ei.value.status == binding.TSVD_E_TOOBIG
    with pytest.raises(binding.TSVDError) as ei:
        binding.tsvd_pack(U, S, V, 0x2)
    assert ei.value.status == binding.TSVD_E_DTYPE


def test_index_and_decode_paths_give_the_same_integers():
    """Both quantise the stage inputs by the same rule and add exact integers, so z (before any
    rounding to fp32 for int8 activations) is identical, and y agrees to the last rounding."""
    import torch
    from paper_2308_07641_b200 import TSVDLinear
    spec = gen.scaled(C["cfg5_d05"], name="idx_vs_decode", M=700, N=900, K=520, B=4, seed=74)
    U, V, S = gen.make_weights(spec)
    x = _util.torch_x(gen.make_x(spec), spec.x_dtype)
    layer = TSVDLinear(U, S, V, LISTS)
    try:
        z_idx = torch.zeros((spec.B, spec.K), dtype=torch.int32, device="cuda")
        z_dec = torch.zeros_like(z_idx)
        y_idx = layer.forward(x, flags=INDEX, z_out=z_idx).clone()
        y_dec = layer.forward(x, flags=0x20, z_out=z_dec).clone()
        torch.cuda.synchronize()
        assert torch.equal(z_idx, z_dec)
        scale = float(y_dec.abs().max())
        assert float((y_idx - y_dec).abs().max()) <= 1e-6 * scale
    finally:
        layer.close()


def test_index_lists_at_full_size():
    """The sparsest workload's layer (4096 x 4096, rank 8192, nonzero rate 0.05) at four int8 tokens:
    z bit-exact and y within the fp32 tolerance, every element."""
    spec = gen.scaled(C["cfg5_d05"], name="idx_full_size", B=4)
    _util.run_and_check(spec, flags=INDEX, pack_flags=LISTS)

