"""CPU-side checks of the C ABI: the library loads, exports every declared symbol, and rejects bad
arguments on the host before any launch (these calls never reach a kernel)."""
import ctypes
import re
from pathlib import Path

import pytest

import paper_1909_05840_b200 as qb
from paper_1909_05840_b200 import build as qb_build

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    qb_build.build()
    return qb.lib()


def _declared_functions():
    text = (ROOT / "include" / "qbert.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qb_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert "qb_gemm" in names and "qb_quantize_act" in names and "qb_layer_linears" in names
    for name in names:
        assert hasattr(lib, name), f"{name} declared in qbert.h but not exported"
    assert set(qb.EXPORTS) <= set(names)


def test_version_and_status_strings(lib):
    assert qb.version() >= 100
    assert lib.qb_status_string(0) == b"QB_OK"
    assert lib.qb_status_string(-6) == b"QB_ERR_TIMEOUT"
    assert lib.qb_status_string(-5) == b"QB_ERR_NONFINITE"


def test_packed_words_and_workspace_sizes(lib):
    assert qb.packed_words(768, 768, 4) == 768 * 768 * 4 // 32
    assert qb.packed_words(768, 768, 3) == 768 * 768 * 3 // 32
    assert qb.packed_words(768, 768, 5) == 0
    assert qb.packed_words(0, 768, 4) == 0
    assert qb.workspace_bytes() >= 256
    assert qb.workspace_bytes(groups=768) >= 256 + 8 * 768
    assert qb.workspace_bytes(groups=768) % 256 == 0


def test_desc_struct_layout_matches_header():
    # 7 pointers, 3 int64, 2 int32, 1 pointer on a 64-bit ABI
    assert ctypes.sizeof(qb.LinearDescC) == 7 * 8 + 3 * 8 + 2 * 4 + 8


def test_argument_errors_are_returned_before_any_launch(lib):
    A = 0x1000  # fake, 16-byte aligned "device" addresses: validation never dereferences them
    ws_bytes = qb.workspace_bytes(groups=128)
    # null pointer
    assert lib.qb_quantize_act(None, 4, 128, A, A, A, A, ws_bytes, None) == qb.QB_ERR_INVALID
    # K not a multiple of 128
    assert lib.qb_quantize_act(A, 4, 100, A, A, A, A, ws_bytes, None) == qb.QB_ERR_ALIGN
    # misaligned pointer
    assert lib.qb_quantize_act(A + 4, 4, 128, A, A, A, A, ws_bytes, None) == qb.QB_ERR_ALIGN
    # workspace too small / null
    assert lib.qb_quantize_act(A, 4, 128, A, A, A, A, 8, None) == qb.QB_ERR_WORKSPACE
    assert lib.qb_quantize_act(A, 4, 128, A, A, A, None, ws_bytes, None) == qb.QB_ERR_WORKSPACE
    # weights: bad bit width, groups that do not divide N, one-sided range
    assert lib.qb_quantize_pack_weights(A, 12, 128, 5, 1, None, None, A, A, A, A, ws_bytes, None) == qb.QB_ERR_INVALID
    assert lib.qb_quantize_pack_weights(A, 12, 128, 4, 5, None, None, A, A, A, A, ws_bytes, None) == qb.QB_ERR_INVALID
    assert lib.qb_quantize_pack_weights(A, 12, 128, 4, 3, A, None, A, A, A, A, ws_bytes, None) == qb.QB_ERR_INVALID
    assert lib.qb_quantize_pack_weights(A, 1024, 128, 4, 1024, None, None, A, A, A, A, 256, None) == qb.QB_ERR_WORKSPACE
    # the batch forms validate every descriptor before anything is launched
    bad = (qb.WeightDescC * 2)()
    bad[0] = qb.WeightDescC(A, 12, 128, 4, 1, None, None, A, A, A)
    bad[1] = qb.WeightDescC(A, 12, 100, 4, 1, None, None, A, A, A)   # K not a multiple of 128
    assert lib.qb_quantize_pack_weights_batch(bad, 2, A, ws_bytes, None) == qb.QB_ERR_ALIGN
    assert lib.qb_fake_quantize_weights_batch(bad, 2, A, ws_bytes, None) == qb.QB_ERR_ALIGN
    assert lib.qb_fake_quantize_weights_batch(None, 0, A, ws_bytes, None) == qb.QB_ERR_INVALID
    assert lib.qb_fake_quantize_weights_batch(bad, 1, A, 8, None) == qb.QB_ERR_WORKSPACE
    # gemm
    assert lib.qb_gemm(A, A, A, A, A, A, None, 8, 12, 128, 4, 5, A, None, A, ws_bytes, None) == qb.QB_ERR_INVALID
    assert lib.qb_gemm(A, A, A, A, A, A, None, 8, 12, 192, 4, 3, A, None, A, ws_bytes, None) == qb.QB_ERR_ALIGN
    assert lib.qb_gemm(A, A, A, A, A, A, None, 8, 12, 128, 4, 3, None, None, A, ws_bytes, None) == qb.QB_ERR_INVALID
    assert lib.qb_gemm(A, A, A, A, A, A, None, 8, 12, 1 << 20, 4, 3, A, None, A, ws_bytes, None) == qb.QB_ERR_INVALID
    assert b"qb_gemm" in lib.qb_last_error()
    # narrow-output forms: same validation
    assert lib.qb_gemm_bf16(A, A, A, A, A, A, None, 8, 12, 128, 4, 5, A, A, ws_bytes, None) == qb.QB_ERR_INVALID
    assert lib.qb_gemm_bf16(A, A, A, A, A, A, None, 8, 12, 192, 4, 3, A, A, ws_bytes, None) == qb.QB_ERR_ALIGN
    assert lib.qb_gemm_bf16(A, A, A, A, A, A, None, 8, 12, 128, 4, 3, None, A, ws_bytes, None) == qb.QB_ERR_INVALID
    # re-quantized output and int8 row sums
    assert lib.qb_gemm_i8(A, A, A, A, A, A, None, 8, 12, 128, 4, 3, None, A, A, ws_bytes, None) == qb.QB_ERR_INVALID
    assert lib.qb_gemm_i8(A, A, A, A, A, A, None, 8, 12, 192, 4, 3, A, A, A, ws_bytes, None) == qb.QB_ERR_ALIGN
    assert lib.qb_layer_linears_i8(None, None, 2, A, ws_bytes, None) == qb.QB_ERR_INVALID
    assert lib.qb_rowsum_i8(A, 8, 100, A, None) == qb.QB_ERR_ALIGN
    assert lib.qb_rowsum_i8(None, 8, 128, A, None) == qb.QB_ERR_INVALID
    # fake quantization and its straight-through backward
    assert lib.qb_fake_quantize_weights(A, 12, 128, 5, 1, None, None, A, A, A, A, ws_bytes, None) == qb.QB_ERR_INVALID
    assert lib.qb_fake_quantize_weights(A, 12, 100, 4, 3, None, None, A, A, A, A, ws_bytes, None) == qb.QB_ERR_ALIGN
    assert lib.qb_fake_quantize_weights(A, 12, 128, 4, 3, None, None, A, A, A, None, ws_bytes, None) == qb.QB_ERR_WORKSPACE
    assert lib.qb_ste_backward(A, A, 12, 128, 5, None, None, A, None) == qb.QB_ERR_INVALID
    assert lib.qb_ste_backward(A, A, 12, 128, 3, A, None, A, None) == qb.QB_ERR_INVALID
    assert lib.qb_ste_backward(A, A + 4, 12, 128, 3, None, None, A, None) == qb.QB_ERR_ALIGN
    # embedding tables
    assert lib.qb_quantize_embedding(A, 100, 768, 4, 100, A, A, A, A, qb.workspace_bytes(groups=768), None) == qb.QB_ERR_INVALID
    assert lib.qb_quantize_embedding(A, 100, 800, 4, 100, A, A, A, A, qb.workspace_bytes(groups=800), None) == qb.QB_ERR_ALIGN
    assert lib.qb_quantize_embedding(A, 100, 768, 4, 128, A, A, A, A, 256, None) == qb.QB_ERR_WORKSPACE
    assert lib.qb_quantize_embedding(A, 100, 8192, 4, 128, A, A, A, A, ws_bytes, None) == qb.QB_ERR_INVALID
    assert lib.qb_embedding_lookup(None, 4, A, A, A, 100, 768, 4, 128, 0, A, A, ws_bytes, None) == qb.QB_ERR_INVALID
    assert lib.qb_embedding_lookup(A, 4, A, A, A, 100, 768, 4, 128, 0, A + 4, A, ws_bytes, None) == qb.QB_ERR_ALIGN
    # stack: every descriptor is validated before the first launch
    good = qb.LinearDescC(A, A, A, A, A, A, None, 8, 12, 128, 4, 3, A)
    bad = qb.LinearDescC(A, A, A, A, A, A, None, 8, 12, 128, 7, 3, A)
    arr = (qb.LinearDescC * 2)(good, bad)
    assert lib.qb_layer_linears(arr, 2, A, ws_bytes, None) == qb.QB_ERR_INVALID
    assert lib.qb_layer_linears(None, 2, A, ws_bytes, None) == qb.QB_ERR_INVALID
    assert lib.qb_layer_linears_bf16(arr, 2, A, ws_bytes, None) == qb.QB_ERR_INVALID
    assert b"qb_layer_linears_bf16" in lib.qb_last_error() or b"qb_gemm" in lib.qb_last_error()


def test_no_cpu_fallback_without_a_device(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    A = 0x1000
    st = lib.qb_quantize_act(A, 4, 128, A, A, A, A, qb.workspace_bytes(), None)
    assert st == qb.QB_ERR_CUDA  # valid arguments, but no sm_100 device: an error, never a CPU path


def test_weight_launch_count_is_host_arithmetic(lib):
    """qb_quantize_pack_weights_launch_count plans on the host: no device, no pointer is touched."""
    def arr_of(shapes):
        arr = (qb.WeightDescC * len(shapes))()
        for i, (N, K, bits, G, ranged) in enumerate(shapes):
            r = 0x1000 if ranged else None
            arr[i] = qb.WeightDescC(0x1000, N, K, bits, G, r, r, 0x1000, 0x1000, 0x1000)
        return arr
    base = [(2304, 768, 384), (768, 768, 128), (3072, 768, 128), (768, 3072, 128)]
    mixed = [(N, K, (2, 3, 4, 8)[l % 4], G, False) for l in range(12) for (N, K, G) in base]
    assert lib.qb_quantize_pack_weights_launch_count(arr_of(mixed), len(mixed)) == 1      # a mixed-precision stack: one launch
    assert lib.qb_quantize_pack_weights_launch_count(arr_of(mixed * 3), 3 * len(mixed)) == 2  # 144 matrices: 96 + 48
    assert lib.qb_quantize_pack_weights_launch_count(arr_of([(768, 768, 4, 1, False)]), 1) == 2  # one range per tensor: two passes
    both = [(768, 768, 4, 128, False), (768, 768, 4, 1, False)]
    assert lib.qb_quantize_pack_weights_launch_count(arr_of(both), 2) == 3
    clustered = [(768, 768, 4, 12, False), (3072, 768, 2, 12, False), (768, 768, 3, 128, False)]  # clusters of 2 and 6, and single CTAs
    assert lib.qb_quantize_pack_weights_launch_count(arr_of(clustered), 3) == 3
    assert lib.qb_quantize_pack_weights_launch_count(None, 0) == 0
    assert lib.qb_quantize_pack_weights_launch_count(arr_of([(768, 700, 4, 128, False)]), 1) == 0
    # the activation quantizer: one pair of launches per 64 tensors
    assert [lib.qb_quantize_act_launch_count(n) for n in (0, 1, 64, 65, 96)] == [0, 2, 2, 4, 4]
