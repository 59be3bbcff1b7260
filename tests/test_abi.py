"""The C ABI without a GPU: the library loads, exports every function that
include/pvt.h declares, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2405_14852_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "pvt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pvt_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_function_is_exported():
    names = declared_functions()
    assert {"pvt_vstep_select", "pvt_vstep_encode", "pvt_dequant", "pvt_workspace_bytes", "pvt_status"} <= set(names)
    L = ctypes.CDLL(B.library_path()) if os.path.exists(B.library_path()) else B.lib()
    for n in names:
        assert hasattr(L, n), f"{n} is declared in pvt.h but not exported"


def test_version_and_error_text():
    assert B.pvt_version() >= 100
    for code in (0, -1, -2, -3, -4):
        assert B.strerror(code)


def _layer(**kw):
    base = dict(rows=16, cols=64, group_dim=8, num_codebooks=1, codebook_size=256, codebook_dtype=B.PVT_F16,
                code_dtype=B.PVT_U8, beam=8, eta=1.0, reserved_=0, W=0x1000, g=0x1000, scale=0x1000,
                codebooks=0x1000, codes=0x1000)
    base.update(kw)
    return B.pvt_layer(**base)


def test_workspace_bytes_depends_on_shape_not_on_a_device():
    small = B.pvt_workspace_bytes(_layer(), 16)
    big = B.pvt_workspace_bytes(_layer(rows=4096, cols=4096, codebook_size=65536, code_dtype=B.PVT_U16), 20971)
    assert 0 < small < big
    assert big >= 4 * 4096 * 512  # one key per group


@pytest.mark.parametrize("kw,k,code", [
    (dict(), 0, B.PVT_EINVAL),                      # k = 0
    (dict(), 16 * 8 + 1, B.PVT_EINVAL),             # k > G
    (dict(cols=60), 1, B.PVT_EINVAL),               # cols % 8
    (dict(group_dim=12), 1, B.PVT_EUNSUPPORTED),
    (dict(group_dim=16, cols=72), 1, B.PVT_EINVAL),  # cols % 16
    (dict(eta=-1.0), 1, B.PVT_EINVAL),
    (dict(eta=float("nan")), 1, B.PVT_EINVAL),
    (dict(g=None), 1, B.PVT_EINVAL),
    (dict(g=0x1004), 1, B.PVT_EINVAL),              # misaligned
])
def test_select_rejects_bad_arguments_before_launch(kw, k, code):
    L = _layer(**kw)
    rc = B.lib().pvt_vstep_select(ctypes.byref(L), k, 0x2000, 0x4000, 1 << 30, None)
    assert rc == code


@pytest.mark.parametrize("kw,code", [
    (dict(num_codebooks=5), B.PVT_EUNSUPPORTED),
    (dict(group_dim=16, num_codebooks=2), B.PVT_EUNSUPPORTED),   # groups of 16: one codebook
    (dict(num_codebooks=3, beam=9), B.PVT_EUNSUPPORTED),
    (dict(num_codebooks=4, codebook_size=64, code_dtype=B.PVT_U16), B.PVT_EUNSUPPORTED),
    (dict(codebook_size=1), B.PVT_EUNSUPPORTED),
    (dict(codebook_size=70000, code_dtype=B.PVT_U16), B.PVT_EUNSUPPORTED),
    (dict(codebook_size=512), B.PVT_EINVAL),        # 512 codewords do not fit U8 codes
    (dict(num_codebooks=2, codebook_size=512, code_dtype=B.PVT_U16), B.PVT_EUNSUPPORTED),
    (dict(num_codebooks=2, beam=9), B.PVT_EUNSUPPORTED),
    (dict(codebook_dtype=7), B.PVT_EINVAL),
    (dict(W=None), B.PVT_EINVAL),
    (dict(num_codebooks=2, codes=0x1001), B.PVT_EINVAL),          # pairs of one-byte codes are read two bytes at a time
    (dict(codebook_size=1024, code_dtype=B.PVT_U16, codes=0x1001), B.PVT_EINVAL),
])
def test_encode_rejects_bad_arguments_before_launch(kw, code):
    L = _layer(**kw)
    rc = B.lib().pvt_vstep_encode(ctypes.byref(L), 0x2000, 4, None, 0x4000, 1 << 30, None)
    assert rc == code


def test_too_small_workspace_is_reported():
    L = _layer()
    assert B.lib().pvt_vstep_select(ctypes.byref(L), 4, 0x2000, 0x4000, 256, None) == B.PVT_EWORKSPACE
    assert B.lib().pvt_vstep_encode(ctypes.byref(L), 0x2000, 4, None, 0x4000, 256, None) == B.PVT_EWORKSPACE
    assert B.lib().pvt_vstep_select(ctypes.byref(L), 4, 0x2000, 0x4010, 1 << 30, None) == B.PVT_EINVAL  # alignment


def test_dequant_rejects_bad_arguments():
    L = _layer()
    assert B.lib().pvt_dequant(ctypes.byref(L), None, B.PVT_F32, None, None) == B.PVT_EINVAL
    assert B.lib().pvt_dequant(ctypes.byref(L), 0x2000, 5, None, None) == B.PVT_EINVAL


def test_misaligned_index_and_output_pointers_are_rejected():
    L = _layer()
    lib = B.lib()
    assert lib.pvt_vstep_select(ctypes.byref(L), 4, 0x2002, 0x4000, 1 << 30, None) == B.PVT_EINVAL
    assert lib.pvt_vstep_encode(ctypes.byref(L), 0x2002, 4, None, 0x4000, 1 << 30, None) == B.PVT_EINVAL
    assert lib.pvt_vstep_encode(ctypes.byref(L), 0x2000, 4, 0x3002, 0x4000, 1 << 30, None) == B.PVT_EINVAL
    assert lib.pvt_vstep_refine(ctypes.byref(L), 0x2000, 4, 1, None, 0x3001, None, None) == B.PVT_EINVAL
    assert lib.pvt_vstep_select_noalloc(ctypes.byref(L), 4, 0x2002, None, None) == B.PVT_EINVAL
    assert lib.pvt_dequant(ctypes.byref(_layer(num_codebooks=2, codes=0x1001)), 0x4000, B.PVT_F32, None, None) == B.PVT_EINVAL


def test_adam_bias_is_computed_in_the_library_and_equals_the_checkers():
    """Host arithmetic of the library (no GPU): 1 - beta^t for the betas of Appendix J over many steps, bit for
    bit what the CPU checker uses, plus the closed values of the first step."""
    from oracle import pvt_oracle as oracle
    for step in list(range(1, 200)) + [1000, 12345, 10 ** 6]:
        for b1, b2 in ((0.9, 0.95), (0.9, 0.999), (0.0, 0.5)):
            assert B.pvt_adam_bias(step, b1, b2) == oracle.adam_bias(step, b1, b2)
    one = ctypes.c_float
    assert B.pvt_adam_bias(1, 0.9, 0.95) == (one(1.0 - one(0.9).value).value, one(1.0 - one(0.95).value).value)
    b1, b2 = ctypes.c_float(), ctypes.c_float()
    assert B.lib().pvt_adam_bias(0, 0.9, 0.95, ctypes.byref(b1), ctypes.byref(b2)) == B.PVT_EINVAL
    assert B.lib().pvt_adam_bias(3, 1.0, 0.95, ctypes.byref(b1), ctypes.byref(b2)) == B.PVT_EINVAL
    assert B.lib().pvt_adam_bias(3, 0.9, 0.95, None, ctypes.byref(b2)) == B.PVT_EINVAL


def test_buffer_and_sampling_calls_reject_bad_arguments():
    L = _layer()
    lib = B.lib()
    big = 1 << 30
    assert lib.pvt_vstep_select_ste(ctypes.byref(L), None, 4, 0x2000, 0x4000, big, None) == B.PVT_EINVAL
    assert lib.pvt_vstep_select_ste(ctypes.byref(L), 0x3004, 4, 0x2000, 0x4000, big, None) == B.PVT_EINVAL  # alignment
    assert lib.pvt_vstep_select_ste(ctypes.byref(L), 0x1000, 4, 0x2000, 0x4000, big, None) == B.PVT_EINVAL  # buffer == g
    assert lib.pvt_vstep_select_ste(ctypes.byref(L), 0x3000, 0, 0x2000, 0x4000, big, None) == B.PVT_EINVAL
    assert lib.pvt_vstep_select_ste(ctypes.byref(L), 0x3000, 4, 0x2000, 0x4000, 256, None) == B.PVT_EWORKSPACE
    assert lib.pvt_vstep_sample(ctypes.byref(L), 4, 7, 1, 0x2000, 0x4000, big, None) == B.PVT_EINVAL  # unknown rule
    assert lib.pvt_vstep_sample(ctypes.byref(L), 0, B.PVT_SAMPLE_UNIFORM, 1, 0x2000, 0x4000, big, None) == B.PVT_EINVAL
    assert lib.pvt_vstep_sample(ctypes.byref(_layer(g=None)), 4, B.PVT_SAMPLE_PROPORTIONAL, 1, 0x2000, 0x4000, big,
                                None) == B.PVT_EINVAL
    assert lib.pvt_vstep_sample(ctypes.byref(L), 4, B.PVT_SAMPLE_UNIFORM, 1, 0x2000, 0x4000, 256, None) == B.PVT_EWORKSPACE


def test_block_call_validates_every_layer_before_launching():
    lib = B.lib()
    good, bad = _layer(), _layer(cols=60)
    n = 2
    arr = (B.pvt_layer * n)(good, bad)
    ks = (ctypes.c_uint64 * n)(4, 4)
    idx = (ctypes.c_void_p * n)(0x2000, 0x3000)
    assert lib.pvt_block_workspace_bytes(arr, ks, n) == 0
    assert lib.pvt_vstep_block(arr, ks, n, idx, None, B.PVT_F32, 0x4000, 1 << 30, None) == B.PVT_EINVAL
    arr = (B.pvt_layer * n)(good, _layer(rows=64, cols=256))
    need = lib.pvt_block_workspace_bytes(arr, ks, n)
    assert need == max(B.pvt_workspace_bytes(arr[0], 4), B.pvt_workspace_bytes(arr[1], 4))
    assert lib.pvt_vstep_block(arr, ks, n, idx, None, B.PVT_F32, 0x4000, need - 1, None) == B.PVT_EWORKSPACE
    ks_bad = (ctypes.c_uint64 * n)(4, 0)
    assert lib.pvt_vstep_block(arr, ks_bad, n, idx, None, B.PVT_F32, 0x4000, 1 << 30, None) == B.PVT_EINVAL
    idx_bad = (ctypes.c_void_p * n)(0x2000, None)
    assert lib.pvt_vstep_block(arr, ks, n, idx_bad, None, B.PVT_F32, 0x4000, 1 << 30, None) == B.PVT_EINVAL
    assert lib.pvt_vstep_block(arr, ks, 0, idx, None, B.PVT_F32, 0x4000, 1 << 30, None) == B.PVT_EINVAL
