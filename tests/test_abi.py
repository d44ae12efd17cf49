"""The C ABI without a GPU: the library loads, exports every declared symbol, and rejects bad
arguments on the host before touching a device."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2308_07641_b200 import build
    build.build()
    from paper_2308_07641_b200 import binding as b
    return b


def _declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(tsvd_[a-z0-9_]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol(binding):
    lib = binding.lib()
    declared = _declared_symbols()
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(lib, name), f"libtsvd.so does not export {name}"
    assert declared == set(binding.EXPORTS)


def test_constants_match_the_header(binding):
    import re
    hdr = open(os.path.join(ROOT, "include", "tsvd.h")).read()
    def define(name):
        return int(re.search(r"#define\s+" + name + r"\s+(0x[0-9a-fA-F]+|\d+)", hdr).group(1), 0)
    assert define("TSVD_DECODE_MAX_B") == binding.TSVD_DECODE_MAX_B
    assert define("TSVD_INDEX_MAX_B") == binding.TSVD_INDEX_MAX_B
    assert define("TSVD_FLAG_PATH_DECODE") == binding.TSVD_FLAG_PATH_DECODE
    assert define("TSVD_FLAG_PATH_SIMPLE") == binding.TSVD_FLAG_PATH_SIMPLE
    assert define("TSVD_FLAG_PATH_TENSOR") == binding.TSVD_FLAG_PATH_TENSOR
    assert define("TSVD_FLAG_OUT_F32") == binding.TSVD_FLAG_OUT_F32
    assert define("TSVD_FLAG_PATH_INDEX") == binding.TSVD_FLAG_PATH_INDEX
    assert define("TSVD_PACK_INDEX_LISTS") == binding.TSVD_PACK_INDEX_LISTS
    assert define("TSVD_INDEX_MAX_COLUMNS") == binding.TSVD_INDEX_MAX_COLUMNS
    assert define("TSVD_MAX_CONTRACTION") == binding.TSVD_MAX_CONTRACTION
    assert define("TSVD_TERNARIZE_MAX_LEN") == binding.TSVD_TERNARIZE_MAX_LEN
    assert define("TSVD_FLAG_WIDE_X") == binding.TSVD_FLAG_WIDE_X
    assert int(re.search(r"TSVD_E_RANGE\s*=\s*(\d+)", hdr).group(1)) == binding.TSVD_E_RANGE
    assert define("TSVD_FLAG_PATH_MASK") == (binding.TSVD_FLAG_PATH_SIMPLE | binding.TSVD_FLAG_PATH_DECODE |
                                            binding.TSVD_FLAG_PATH_TENSOR | binding.TSVD_FLAG_PATH_INDEX)


def test_strerror_covers_all_codes(binding):
    seen = {binding.tsvd_strerror(i) for i in range(0, 12)}
    assert len(seen) == 12 and "unknown status" not in seen
    assert binding.tsvd_strerror(99) == "unknown status"


def test_host_side_validation(binding):
    lib = binding.lib()
    h = ctypes.c_void_p()
    U = np.zeros((2, 2), np.int8); S = np.zeros(2, np.float32); V = np.zeros((2, 2), np.int8)
    assert lib.tsvd_pack(None, S.ctypes.data, V.ctypes.data, 2, 2, 2, 0, ctypes.byref(h)) == binding.TSVD_E_NULL
    assert lib.tsvd_pack(U.ctypes.data, S.ctypes.data, V.ctypes.data, 2, 2, 2, 0, None) == binding.TSVD_E_NULL
    assert lib.tsvd_pack(U.ctypes.data, S.ctypes.data, V.ctypes.data, 0, 2, 2, 0, ctypes.byref(h)) == binding.TSVD_E_SHAPE
    assert lib.tsvd_pack(U.ctypes.data, S.ctypes.data, V.ctypes.data, 2, 2, 2, 7, ctypes.byref(h)) == binding.TSVD_E_DTYPE
    assert h.value is None
    # The digit sums of a row are combined in 32-bit integers, |sum| <= 128 * 257 * columns: the
    # contraction length is bounded where that would leave 31 bits (checked before any device call).
    big = binding.TSVD_MAX_CONTRACTION + 1
    assert 128 * 257 * binding.TSVD_MAX_CONTRACTION < 2 ** 31 <= 128 * 257 * (binding.TSVD_MAX_CONTRACTION + 128)
    assert lib.tsvd_pack(U.ctypes.data, S.ctypes.data, V.ctypes.data, 2, 2, big, 0, ctypes.byref(h)) == binding.TSVD_E_TOOBIG
    assert lib.tsvd_pack(U.ctypes.data, S.ctypes.data, V.ctypes.data, 2, big, 2, 0, ctypes.byref(h)) == binding.TSVD_E_TOOBIG
    assert h.value is None
    assert lib.tsvd_reserve(None, 1, 0) == binding.TSVD_E_NULL
    one = ctypes.c_void_p(16)     # never dereferenced: the sizes are checked first
    assert lib.tsvd_ternarize(None, 1, 4, 4, 0.5, one, 4, None, None) == binding.TSVD_E_NULL
    assert lib.tsvd_ternarize(one, 1, 4, 3, 0.5, one, 4, None, None) == binding.TSVD_E_SHAPE
    assert lib.tsvd_ternarize(one, 1, 4, 4, 2.0, one, 4, None, None) == binding.TSVD_E_SHAPE
    assert lib.tsvd_ternarize(one, 1, binding.TSVD_TERNARIZE_MAX_LEN + 1, 1 << 20, 0.5, one, 1 << 20, None, None) == binding.TSVD_E_TOOBIG
    assert lib.tsvd_set_bias(None, None) == binding.TSVD_E_NULL
    assert lib.tsvd_forward_v(None, one, 4, one, 4, 1, 0, 0, None) == binding.TSVD_E_NULL
    assert lib.tsvd_forward_v_patches(None, one, 0, 1, 4, 4, 16, 1, 1, 1, 1, 0, 0, 1, 1, one, 4, 0, None) == binding.TSVD_E_NULL
    assert lib.tsvd_im2col(None, 0, 1, 4, 4, 1, 1, 1, 1, 1, 0, 0, 1, 1, one, 1, None) == binding.TSVD_E_NULL
    assert lib.tsvd_im2col(one, 0, 1, 2, 2, 1, 3, 3, 1, 1, 0, 0, 1, 1, one, 9, None) == binding.TSVD_E_SHAPE   # kernel larger than the image
    assert lib.tsvd_im2col(one, 0, 1, 4, 4, 2, 3, 3, 1, 1, 0, 0, 1, 1, one, 17, None) == binding.TSVD_E_SHAPE  # ld_out < k1*k2*C
    assert lib.tsvd_im2col(one, 7, 1, 4, 4, 2, 3, 3, 1, 1, 0, 0, 1, 1, one, 18, None) == binding.TSVD_E_DTYPE
    assert lib.tsvd_forward(None, None, None, 1, 0, None) == binding.TSVD_E_NULL
    assert lib.tsvd_info(None, None, None, None, None, None, None) == binding.TSVD_E_NULL
    assert lib.tsvd_last_status(None) == binding.TSVD_E_NULL
    lib.tsvd_destroy(None)  # no-op


def test_no_cpu_fallback_without_device(binding):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(binding.TSVDError) as e:
        binding.tsvd_pack(np.zeros((2, 2), np.int8), np.ones(2, np.float32), np.zeros((2, 2), np.int8))
    assert e.value.status == binding.TSVD_E_CUDA


def test_product_does_not_import_the_checker():
    pkg = os.path.join(ROOT, "paper_2308_07641_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert "oracle" not in text, f"{fn} mentions the checker"


def test_recorded_dram_traffic_is_well_formed():
    """profiles/dram_traffic.txt: per workload the hashed source files exist, and the lookup bench.py
    uses returns either the recorded bytes (sources unchanged since the capture) or None."""
    import importlib.util
    import json
    spec = importlib.util.spec_from_file_location("bench_for_test", os.path.join(ROOT, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    with open(os.path.join(ROOT, "profiles", "dram_traffic.txt")) as f:
        rec = json.load(f)["workloads"]
    assert rec
    for workload, w in rec.items():
        for name in w["sources"]:
            assert os.path.exists(os.path.join(ROOT, "paper_2308_07641_b200", "csrc", name))
        fresh = w["sha1"] == bench.kernel_source_sha1(w["sources"])
        for stage, byts in w["bytes_per_launch"].items():
            assert isinstance(byts, int) and byts > 0
            assert bench.recorded_traffic(workload, stage) == (byts if fresh else None)
    assert bench.recorded_traffic("no_such_workload", "v_stage") is None

