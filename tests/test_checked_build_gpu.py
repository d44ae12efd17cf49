"""The library compiled with -DTSVD_CHECK_BOUNDS (the contraction kernel checks its ring and tile
indices and reports through the status word): forwards of every tensor-path regime must give the same
results as the regular build, against the CPU checker, with the status word clean."""
import pytest

import gen
from tests import _util

pytestmark = pytest.mark.gpu
C = gen.CONFIGS


@pytest.fixture()
def checked_library():
    from paper_2308_07641_b200 import binding, build
    build.build()
    path = build.build_checked()
    binding.use_library(path)
    try:
        yield binding
    finally:
        binding.use_library(None)


CASES = [
    gen.scaled(C["cfg2"], name="chk_resident_panels", M=640, N=256, K=384, B=330, seed=401),      # K <= 1024: digit panels stay resident
    gen.scaled(C["cfg4"], name="chk_streamed_tiles", M=300, N=1500, K=1300, B=200, seed=402),       # longer contractions: tiles streamed
    gen.scaled(C["cfg2"], name="chk_small_batch_split", M=520, N=8300, K=390, B=40, seed=403),      # split contraction, last-arriver tail
    gen.scaled(C["cfg5_d20"], name="chk_int8", M=256, N=384, K=1200, B=100, seed=404),
    gen.scaled(C["cfg1"], name="chk_f32_ragged", M=129, N=130, K=127, B=65, seed=405),
    gen.scaled(C["cfg2"], name="chk_wide_u_tiles", M=2560, N=330, K=1300, B=400, seed=406),         # U-stage: one round of 256-column tiles
]


@pytest.mark.parametrize("spec", CASES, ids=lambda s: s.name)
def test_checked_build_runs_clean(checked_library, spec):
    assert checked_library.LIB_PATH.endswith("libtsvd_checked.so")
    res = _util.run_and_check(spec, flags=0x40, expect_status=0)
    assert res["status"] == 0
