"""The C-ABI library loads, exports every symbol its header declares, and rejects bad
arguments on the host before anything is launched (runs without a GPU)."""
import ctypes as C
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    from paper_1805_11046_b200 import build
    build.build_library()
    return C.CDLL(str(build.LIB))


def declared_functions():
    text = (ROOT / "include" / "qbp.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qbp_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 17
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_entry_points():
    import torch  # noqa: F401  (the binding uses torch for device memory only)
    from paper_1805_11046_b200 import binding
    assert sorted(binding.EXPORTS) == declared_functions()


def test_struct_layouts_match_the_header():
    from paper_1805_11046_b200 import binding
    assert C.sizeof(binding.ConvDesc) == 36
    assert C.sizeof(binding.LayerDesc) == 36 + 4 + 3 * 8 + 4 + 4 + 8 + 4 + 4
    assert C.sizeof(binding.LayerCtx) == 15 * 8
    assert C.sizeof(binding.Epilogue) == 8 * 8 and C.sizeof(binding.Requant) == 4 * 8


def _err(lib):
    lib.qbp_last_error.restype = C.c_char_p
    return lib.qbp_last_error().decode()


def test_host_side_refusals(lib):
    i64 = C.c_int64
    null = C.c_void_p(0)
    fake = C.c_void_p(4096)            # never dereferenced: validation fails first
    # Range BN needs n >= 2: C(1) is infinite
    assert lib.qbp_rangebn_fwd(fake, i64(1), i64(8), null, null, 0, fake, fake, fake, fake, null, fake,
                               C.c_size_t(1 << 30), null) == -1
    assert "at least 2" in _err(lib)
    # reduction too long for an int32 accumulator of 8-bit codes
    assert lib.qbp_gemm_s8(0, 0, i64(128), i64(128), i64(33040), fake, fake, fake, fake, null, fake, null, fake,
                           C.c_size_t(1 << 30), null) == -3
    assert "33025" in _err(lib)
    # shapes the tensor-core path does not take
    assert lib.qbp_gemm_s8(0, 0, i64(100), i64(128), i64(128), fake, fake, fake, fake, null, fake, null, fake,
                           C.c_size_t(1 << 30), null) == -2
    # both outputs missing; NULL operand; misaligned operand; too small a workspace
    assert lib.qbp_gemm_s8(0, 0, i64(128), i64(128), i64(128), fake, fake, fake, fake, null, null, null, fake,
                           C.c_size_t(1 << 30), null) == -1
    assert lib.qbp_gemm_s8(0, 0, i64(128), i64(128), i64(128), null, fake, fake, fake, null, fake, null, fake,
                           C.c_size_t(1 << 30), null) == -1
    assert lib.qbp_gemm_s8(0, 0, i64(128), i64(128), i64(128), C.c_void_p(4100), fake, fake, fake, null, fake, null, fake,
                           C.c_size_t(1 << 30), null) == -1
    assert lib.qbp_gemm_s8(0, 0, i64(128), i64(128), i64(128), fake, fake, fake, fake, null, fake, null, fake,
                           C.c_size_t(16), null) == -4
    assert "workspace" in _err(lib)
    # quantiser enums
    assert lib.qbp_quantize_s8(fake, i64(4), i64(4), 7, 0, C.c_uint64(0), C.c_uint32(0), null, fake, fake, null, null,
                               fake, C.c_size_t(1 << 30), null) == -1
    assert lib.qbp_quantize_s16(fake, i64(4), i64(4), 0, 0, C.c_uint64(0), C.c_uint32(0), null, null, null, null, fake,
                                fake, C.c_size_t(1 << 30), null) == -1


def test_convolution_shapes_outside_the_implementation_are_refused(lib):
    from paper_1805_11046_b200.binding import ConvDesc
    fake = C.c_void_p(4096); null = C.c_void_p(0)
    for d in (ConvDesc(1, 8, 8, 64, 64, 3, 3, 2, 1),      # stride 2
              ConvDesc(1, 8, 8, 64, 64, 5, 5, 1, 2),      # 5x5
              ConvDesc(1, 8, 8, 24, 64, 3, 3, 1, 1)):     # channels not a multiple of 16
        assert lib.qbp_conv_s8_implicit(0, C.byref(d), fake, fake, fake, fake, null, fake, null, fake, C.c_size_t(1 << 30),
                                        null) == -2


def test_epilogue_statistics_need_all_three_buffers_the_output_and_few_columns(lib):
    from paper_1805_11046_b200.binding import Epilogue
    fake = C.c_void_p(4096); null = C.c_void_p(0); i64 = C.c_int64
    part = Epilogue(col_sum=4096, col_min=0, col_max=4096)
    assert lib.qbp_gemm_s8(0, 0, i64(128), i64(128), i64(128), fake, fake, fake, fake, null, fake, C.byref(part), fake,
                           C.c_size_t(1 << 30), null) == -1
    full = Epilogue(col_sum=4096, col_min=4096, col_max=4096)
    assert lib.qbp_gemm_s8(0, 0, i64(128), i64(128), i64(128), fake, fake, fake, fake, fake, null, C.byref(full), fake,
                           C.c_size_t(1 << 30), null) == -1              # no fp32 output to take them from
    assert lib.qbp_gemm_s8(0, 0, i64(128), i64(512), i64(128), fake, fake, fake, fake, null, fake, C.byref(full), fake,
                           C.c_size_t(1 << 30), null) == -2              # more than 256 columns
    both = Epilogue(col_sum=4096, col_min=4096, col_max=4096, relu=1)
    assert lib.qbp_gemm_s8(0, 0, i64(128), i64(128), i64(128), fake, fake, fake, fake, null, fake, C.byref(both), fake,
                           C.c_size_t(1 << 30), null) == -1              # statistics and the ReLU / requantisation tail exclude one another
    noparams = Epilogue(q_out=4096)
    assert lib.qbp_gemm_s8(0, 0, i64(128), i64(128), i64(128), fake, fake, fake, fake, null, fake, C.byref(noparams), fake,
                           C.c_size_t(1 << 30), null) == -1              # requantisation without clamping values


def test_workspace_queries_are_pure(lib):
    for name in ("qbp_quantize_workspace_bytes", "qbp_gemm_s8_workspace_bytes", "qbp_rangebn_workspace_bytes"):
        getattr(lib, name).restype = C.c_size_t
    assert lib.qbp_quantize_workspace_bytes(C.c_int64(10), C.c_int64(64), 0) > 0
    assert lib.qbp_quantize_workspace_bytes(C.c_int64(10), C.c_int64(64), 1) > lib.qbp_quantize_workspace_bytes(
        C.c_int64(10), C.c_int64(64), 0)
    assert lib.qbp_gemm_s8_workspace_bytes(C.c_int64(4096), C.c_int64(4096), C.c_int64(4096)) >= 4096 * 12
    assert lib.qbp_rangebn_workspace_bytes(C.c_int64(1000), C.c_int64(64)) > 0


def test_host_side_refusals_of_the_low_bit_entry_points(lib):
    i64 = C.c_int64
    null = C.c_void_p(0)
    fake = C.c_void_p(4096)            # never dereferenced: validation fails first
    big = C.c_size_t(1 << 30)
    assert lib.qbp_binarize_s8(null, i64(8), fake, null, null) == -1
    assert lib.qbp_stc_ternarize_s8(fake, i64(8), 0, C.c_uint64(0), 0, fake, fake, fake, big, null) == -1        # samples < 1
    assert lib.qbp_stc_ternarize_s8(fake, i64(8), 128, C.c_uint64(0), 0, fake, fake, fake, big, null) == -1      # samples > 127
    assert lib.qbp_stc_ternarize_s8(fake, i64(8), 1, C.c_uint64(0), 0, fake, fake, fake, C.c_size_t(16), null) == -4
    # Algorithm 1: what the weight-gradient product would refuse is refused before the ternariser runs
    assert lib.qbp_tbp_weight_gradient(null, i64(64), i64(24), i64(32), fake, fake, fake, 1, C.c_uint64(0), 0, fake, fake, fake,
                                       null, fake, fake, big, null) == -2
    assert lib.qbp_tbp_weight_gradient(null, i64(64), i64(32), i64(32), fake, fake, fake, 1, C.c_uint64(0), 0, fake, fake, fake,
                                       null, null, fake, big, null) == -1                                      # no output wanted
    assert lib.qbp_pack_bits(fake, i64(1), i64(0), 0, fake, null) == -1
    assert lib.qbp_xnor_gemm_bits(i64(0), i64(1), i64(1), fake, fake, fake, null) == -1
    assert lib.qbp_gated_xnor_gemm_bits(i64(1), i64(1), i64(1), fake, null, fake, fake, null) == -1
