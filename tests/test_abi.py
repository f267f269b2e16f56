"""CPU-only checks of the C-ABI boundary: the library loads, exports every symbol the
header declares, and rejects bad arguments before touching any device."""
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def mg():
    from paper_2506_11728_b200 import build
    build.build_library()
    from paper_2506_11728_b200 import binding
    return binding


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "mipgemm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mipgemm_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(mg):
    names = declared_symbols()
    assert "mipgemm_s8s8s32" in names and "mipgemm_conv_u8s8s32" in names and len(names) >= 12
    for name in names:
        assert hasattr(mg._lib, name), name
        assert name in mg.SIGNATURES, name
        assert callable(getattr(mg, name)), name
    assert sorted(mg.SIGNATURES) == names


def test_version_and_status_strings(mg):
    assert mg.mipgemm_version() >= 100
    for st in range(7):
        assert mg.mipgemm_status_string(st) not in ("", "unknown status")
    assert mg.mipgemm_status_string(99) == "unknown status"


def test_argument_errors_are_synchronous(mg):
    s = 0  # stream handle is never dereferenced on these paths
    a = b = c = 256  # fake, aligned, non-NULL addresses; never dereferenced either
    assert mg.mipgemm_s8s8s32(-1, 4, 4, a, 4, b, 4, c, 4, 0, s, check=False) == mg.ERR_INVALID_ARG
    assert mg.mipgemm_s8s8s32(4, 4, 8, a, 7, b, 8, c, 4, 0, s, check=False) == mg.ERR_INVALID_ARG
    assert mg.mipgemm_s8s8s32(4, 4, 8, a, 8, b, 7, c, 4, 0, s, check=False) == mg.ERR_INVALID_ARG
    assert mg.mipgemm_s8s8s32(4, 4, 8, a, 8, b, 8, c, 3, 0, s, check=False) == mg.ERR_INVALID_ARG
    assert mg.mipgemm_s8s8s32(4, 4, 8, 0, 8, b, 8, c, 4, 0, s, check=False) == mg.ERR_INVALID_ARG
    assert mg.mipgemm_s8s8s32(4, 4, 8, a, 8, b, 8, 0, 4, 0, s, check=False) == mg.ERR_INVALID_ARG
    assert mg.mipgemm_s8s8s32(4, 4, 8, a, 8, b, 8, c + 2, 4, 0, s, check=False) == mg.ERR_INVALID_ARG
    assert mg.mipgemm_s8s8s32(4, 4, 131072, a, 131072, b, 131072, c, 4, 0, s, check=False) == mg.ERR_K_TOO_LARGE
    assert mg.mipgemm_u8s8s32(4, 4, 65794, a, 65794, b, 65794, c, 4, 0, s, check=False) == mg.ERR_K_TOO_LARGE
    # empty problems are fine and need no device
    assert mg.mipgemm_s8s8s32(0, 4, 8, a, 8, b, 8, c, 4, 0, s, check=False) == mg.OK
    assert mg.mipgemm_last_path() & mg.PATH_MASK == mg.PATH_TRIVIAL
    assert mg.mipgemm_u8s8s32(4, 0, 8, a, 8, b, 8, c, 0, 0, s, check=False) == mg.OK


def test_conv_argument_errors(mg):
    x = w = y = 256
    bad = mg.ERR_INVALID_ARG
    conv = mg.mipgemm_conv_u8s8s32
    assert conv(1, 8, 8, 4, 4, 3, 3, 0, 1, 1, 1, 1, 1, x, w, y, 0, 0, check=False) == bad      # stride 0
    assert conv(1, 2, 2, 4, 4, 5, 5, 1, 1, 0, 0, 1, 1, x, w, y, 0, 0, check=False) == bad      # filter > image
    assert conv(1, 8, 8, 4, 4, 3, 3, 1, 1, -1, 0, 1, 1, x, w, y, 0, 0, check=False) == bad     # negative pad
    assert conv(1, 8, 8, 4, 4, 3, 3, 1, 1, 1, 1, 1, 1, 0, w, y, 0, 0, check=False) == bad      # NULL X
    assert conv(1, 64, 64, 8192, 4, 3, 3, 1, 1, 1, 1, 1, 1, x, w, y, 0, 0, check=False) == mg.ERR_K_TOO_LARGE
    assert conv(0, 8, 8, 4, 4, 3, 3, 1, 1, 1, 1, 1, 1, x, w, y, 0, 0, check=False) == mg.OK


def test_workspace_queries(mg):
    q = mg.mipgemm_workspace_query_gemm
    assert q(1000, 3001, 768, 256, 768, 512, 768, 1024, 3001) == 0
    need = q(1000, 3001, 777, 256, 777, 512, 777, 1024, 3001)
    assert need >= (1000 + 3001) * 784 and need % 256 == 0
    assert q(1000, 3001, 768, 257, 768, 512, 768, 1024, 3001) >= 1000 * 768   # misaligned base of A only
    qc = mg.mipgemm_workspace_query_conv
    assert qc(32, 56, 56, 64, 64, 3, 3, 1, 1, 1, 1, 1, 1) == 0                  # TMA im2col
    assert qc(32, 56, 56, 64, 256, 1, 1, 1, 1, 0, 0, 1, 1) == 0                 # pointwise
    assert qc(32, 224, 224, 3, 64, 7, 7, 2, 2, 3, 3, 1, 1) == 64 * 7 * 32          # gathered: slot-padded weights only
    assert qc(2, 32, 32, 3, 64, 3, 3, 1, 1, 2, 2, 2, 2) >= 2 * 32 * 32 * 32        # dilated columns: explicit matrix


def test_tuning_validation(mg):
    with pytest.raises(mg.MipGemmError):
        mg.mipgemm_set_tuning(block_n=48)
    mg.mipgemm_set_tuning(block_n=128, stages=3)
    mg.mipgemm_set_tuning()


def test_constant_weight_ranges_are_bookkeeping_only(mg):
    """Registering and unregistering weight ranges touches no device."""
    assert mg.mipgemm_register_constant_weights(0, 16, check=False) == mg.ERR_INVALID_ARG
    assert mg.mipgemm_register_constant_weights(4096, 0, check=False) == mg.ERR_INVALID_ARG
    assert mg.mipgemm_register_constant_weights(4096, 1 << 20) == mg.OK
    assert mg.mipgemm_register_constant_weights(1 << 30, 1 << 20) == mg.OK
    assert mg.mipgemm_unregister_constant_weights(8192, check=False) == mg.ERR_INVALID_ARG   # not a base
    assert mg.mipgemm_unregister_constant_weights(4096) == mg.OK
    assert mg.mipgemm_unregister_constant_weights(4096, check=False) == mg.ERR_INVALID_ARG   # already gone
    assert mg.mipgemm_unregister_constant_weights(1 << 30) == mg.OK
