"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, and its argument validation returns the documented status codes."""
import ctypes
import os
import re

import pytest
import torch

from paper_2505_00570_b200 import binding as fk

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built_library():
    if not os.path.exists(fk.LIB_PATH):
        from paper_2505_00570_b200 import build
        build.build()
    return fk.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "freqkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(freqkv_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = declared_functions()
    assert len(names) >= 15
    lib = fk.lib()
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(fk.EXPORTS) == names


def test_version_and_status_strings():
    assert fk.lib().freqkv_version() >= 100
    assert fk.status_string(fk.OK) == "FREQKV_OK"
    assert fk.status_string(fk.ERR_CAPACITY) == "FREQKV_ERR_CAPACITY"
    assert fk.status_string(99) == "FREQKV_ERR_UNKNOWN"


def test_layout_struct_matches_header_size():
    assert ctypes.sizeof(fk.Layout) == 6 * 4 + 4 * 8


def test_layout_contiguous():
    st, lay = fk.layout_contiguous(fk.BF16, 2, 3, 4, 100, 128)
    assert st == fk.OK
    assert (lay.stride_token, lay.stride_head, lay.stride_layer, lay.stride_batch) == (128, 12800, 51200, 153600)
    assert fk.layout_contiguous(fk.BF16, 1, 1, 1, 16, 100)[0] == fk.ERR_UNSUPPORTED   # head_dim % 8
    assert fk.layout_contiguous(fk.BF16, 1, 1, 1, 16, 512)[0] == fk.ERR_UNSUPPORTED   # head_dim > 256
    assert fk.layout_contiguous(fk.BF16, 0, 1, 1, 16, 128)[0] == fk.ERR_INVALID_ARG
    assert fk.layout_contiguous(7, 1, 1, 1, 16, 128)[0] == fk.ERR_UNSUPPORTED


K, V = 0x10000000, 0x20000000  # fake, never dereferenced by the host-only checks


def lay(cap=4096, hd=128, B=1, Ly=2, H=2, dtype=fk.BF16):
    st, out = fk.layout_contiguous(dtype, B, Ly, H, cap, hd)
    assert st == fk.OK
    return out


def test_check_compress_lengths():
    L = lay()
    assert fk.check_compress(L, K, V, 4096, 2046, 4) == fk.OK
    assert fk.check_compress(L, K, V, 4096, 4092, 4) == fk.OK          # identity
    assert fk.check_compress(L, K, V, 4, 0, 4) == fk.OK                # only sinks
    assert fk.check_compress(L, K, V, 4096, 4093, 4) == fk.ERR_INVALID_ARG  # kept > len - sink
    assert fk.check_compress(L, K, V, 4097, 10, 4) == fk.ERR_INVALID_ARG    # len > capacity
    assert fk.check_compress(L, K, V, 3, 0, 4) == fk.ERR_INVALID_ARG        # sink > len
    assert fk.check_compress(L, K, V, 100, -1, 4) == fk.ERR_INVALID_ARG
    assert fk.check_compress(L, K, V, 100, 10, -1) == fk.ERR_INVALID_ARG


def test_check_compress_pointers():
    L = lay()
    assert fk.check_compress(L, 0, V, 100, 10, 4) == fk.ERR_INVALID_ARG
    assert fk.check_compress(L, K, 0, 100, 10, 4) == fk.ERR_INVALID_ARG
    assert fk.check_compress(L, K + 8, V, 100, 10, 4) == fk.ERR_UNSUPPORTED   # not 16-byte aligned
    assert fk.check_compress(L, K, K, 100, 10, 4) == fk.ERR_INVALID_ARG       # K and V alias
    assert fk.check_compress(L, K, K + 4096, 100, 10, 4) == fk.ERR_INVALID_ARG  # K and V overlap
    assert fk.lib().freqkv_check_compress(None, K, V, 100, 10, 4) == fk.ERR_INVALID_ARG


def test_check_layout_strides():
    L = lay()
    L.stride_token = 136                      # padded rows: fine
    L.stride_head = 136 * 4096
    L.stride_layer = 2 * L.stride_head
    L.stride_batch = 2 * L.stride_layer
    assert fk.check_compress(L, K, V, 100, 10, 4) == fk.OK
    L.stride_token = 132                      # rows not 16-byte aligned
    assert fk.check_compress(L, K, V, 100, 10, 4) == fk.ERR_UNSUPPORTED
    L = lay()
    L.stride_token = 64                       # rows overlap
    assert fk.check_compress(L, K, V, 100, 10, 4) == fk.ERR_UNSUPPORTED
    L = lay()
    L.stride_head = 128 * 100                 # heads overlap inside the capacity
    assert fk.check_compress(L, K, V, 100, 10, 4) == fk.ERR_UNSUPPORTED
    L = lay()
    L.stride_layer, L.stride_head = L.stride_head, L.stride_layer   # permuted axes are fine
    assert fk.check_compress(L, K, V, 100, 10, 4) == fk.OK
    L = lay()
    L.stride_batch = -8
    assert fk.check_compress(L, K, V, 100, 10, 4) == fk.ERR_INVALID_ARG


def test_check_append():
    L = lay(cap=64, B=2)
    NK, NV = 0x30000000, 0x40000000
    assert fk.check_append(L, K, V, NK, NV, 1, [10, 63]) == fk.OK
    assert fk.check_append(L, K, V, NK, NV, 2, [10, 63]) == fk.ERR_CAPACITY    # the lazy trigger
    assert fk.check_append(L, K, V, NK, NV, 1, [10, 64]) == fk.ERR_CAPACITY
    assert fk.check_append(L, K, V, NK, NV, 1, [10, 65]) == fk.ERR_INVALID_ARG
    assert fk.check_append(L, K, V, NK, NV, 1, [-1, 3]) == fk.ERR_INVALID_ARG
    assert fk.check_append(L, K, V, 0, NV, 1, [0, 0]) == fk.ERR_INVALID_ARG
    assert fk.check_append(L, K, V, NK + 4, NV, 1, [0, 0]) == fk.ERR_UNSUPPORTED
    assert fk.check_append(L, K, V, 0, 0, 0, [0, 0]) == fk.OK                  # nothing to append
    assert fk.check_append(L, K, V, NK, NV, -1, [0, 0]) == fk.ERR_INVALID_ARG


def test_check_attend():
    L = lay(cap=64, B=2)
    Q, O = 0x30000000, 0x40000000
    assert fk.check_attend(L, K, V, 0, Q, O, 1, [1, 64]) == fk.OK
    assert fk.check_attend(L, K, V, 0, Q, O, 4, [10, 20]) == fk.OK
    assert fk.check_attend(L, K, V, 0, Q, O, 3, [10, 20]) == fk.ERR_UNSUPPORTED      # group size not 1, 2, 4, 8
    assert fk.check_attend(L, K, V, 0, Q, O, 0, [10, 20]) == fk.ERR_INVALID_ARG
    assert fk.check_attend(L, K, V, 0, Q, O, 1, [0, 20]) == fk.ERR_INVALID_ARG       # an empty cache has nothing to attend to
    assert fk.check_attend(L, K, V, 0, Q, O, 1, [10, 65]) == fk.ERR_INVALID_ARG
    assert fk.check_attend(L, K, V, L.layers, Q, O, 1, [10, 20]) == fk.ERR_INVALID_ARG
    assert fk.check_attend(L, K, V, -1, Q, O, 1, [10, 20]) == fk.ERR_INVALID_ARG
    assert fk.check_attend(L, K, V, 0, Q, Q, 1, [10, 20]) == fk.ERR_INVALID_ARG
    assert fk.check_attend(L, K, V, 0, 0, O, 1, [10, 20]) == fk.ERR_INVALID_ARG
    assert fk.check_attend(L, K, V, 0, Q + 2, O, 1, [10, 20]) == fk.ERR_UNSUPPORTED
    assert fk.check_attend(lay(hd=64), K, V, 0, Q, O, 1, [10]) == fk.ERR_UNSUPPORTED


def test_check_attend_prefill():
    L = lay(cap=64, B=2)
    Q, O = 0x30000000, 0x40000000
    assert fk.check_attend_prefill(L, K, V, 0, Q, O, 1, 10, [10, 64]) == fk.OK
    assert fk.check_attend_prefill(L, K, V, 0, Q, O, 3, 1, [1, 20]) == fk.OK                 # any group size
    assert fk.check_attend_prefill(L, K, V, 0, Q, O, 1, 0, [10, 20]) == fk.ERR_INVALID_ARG   # an empty chunk
    assert fk.check_attend_prefill(L, K, V, 0, Q, O, 1, 11, [10, 20]) == fk.ERR_INVALID_ARG  # chunk longer than a cache length
    assert fk.check_attend_prefill(L, K, V, 0, Q, O, 1, 5, [10, 65]) == fk.ERR_INVALID_ARG
    assert fk.check_attend_prefill(L, K, V, 0, Q, O, 0, 5, [10, 20]) == fk.ERR_INVALID_ARG
    assert fk.check_attend_prefill(L, K, V, L.layers, Q, O, 1, 5, [10, 20]) == fk.ERR_INVALID_ARG
    assert fk.check_attend_prefill(L, K, V, 0, Q, Q, 1, 5, [10, 20]) == fk.ERR_INVALID_ARG
    assert fk.check_attend_prefill(L, K, V, 0, 0, O, 1, 5, [10, 20]) == fk.ERR_INVALID_ARG
    assert fk.check_attend_prefill(L, K, V, 0, Q + 2, O, 1, 5, [10, 20]) == fk.ERR_UNSUPPORTED
    assert fk.check_attend_prefill(lay(hd=64), K, V, 0, Q, O, 1, 5, [10]) == fk.ERR_UNSUPPORTED
    assert fk.check_attend_prefill(lay(dtype=fk.F32), K, V, 0, Q, O, 1, 5, [10]) == fk.ERR_UNSUPPORTED  # bf16 caches only


def test_null_context_is_rejected():
    L = lay()
    lib = fk.lib()
    assert lib.freqkv_compress(None, ctypes.byref(L), K, V, 100, 10, 4, None) == fk.ERR_INVALID_ARG
    assert lib.freqkv_destroy(None) == fk.ERR_INVALID_ARG
    assert lib.freqkv_set_variant(None, 0) == fk.ERR_INVALID_ARG
    assert lib.freqkv_create(None, 0) == fk.ERR_INVALID_ARG


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_create_fails_loudly_without_gpu():
    with pytest.raises(fk.FreqKVError):
        fk.Context(0)


def test_fold_level_rule():
    """Host-only rule of how often variant GEMM folds: twice where the lengths halve twice and that saves
    64-row slices over tiles of 256 rows, not at all for at most 256 kept rows, else once."""
    from paper_2505_00570_b200 import binding as fk

    assert fk.gemm_fold_levels(4092, 2046) == 2 and fk.gemm_fold_levels(4096, 2048) == 2 and fk.gemm_fold_levels(8188, 4094) == 2
    assert fk.gemm_fold_levels(4092, 2046, 2046) == 1      # another band of components: one level
    assert fk.gemm_fold_levels(4092, 2045) == 1 and fk.gemm_fold_levels(4094, 2047) == 1 and fk.gemm_fold_levels(2046, 1022) == 1
    assert fk.gemm_fold_levels(3000, 1500) == 1            # 375 twice-folded rows fill two tiles as badly as 750 fill three
    assert fk.gemm_fold_levels(4092, 40) == 0 and fk.gemm_fold_levels(4092, 256) == 0
    assert fk.gemm_fold_levels(0, 0) == -1 and fk.gemm_fold_levels(10, 11) == -1 and fk.gemm_fold_levels(10, 5, -1) == -1
