"""CPU-only checks of the boundary: the library builds for sm_100a, loads, and exports every
symbol ``include/slope.h`` declares; pure host logic (sizes, argument checks) behaves."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2608_24070_b200 import build, binding

    build.build()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "slope.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(slope_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    from paper_2608_24070_b200 import binding

    names = declared_symbols()
    assert len(names) >= 14
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTS) == names


def test_size_helpers(lib):
    assert lib.slope_values_bytes(4096, 4096) == 4096 * 4096
    assert lib.slope_meta_bytes(4096, 11008) == 4096 * 11008 // 8
    assert lib.slope_mask_bytes(512, 512) == 512 * 512 // 8
    assert lib.slope_adapter_workspace_bytes(16384, 4096, 4096, 64) > 0
    assert lib.slope_adapter_workspace_bytes(16384, 4096, 4096, 0) == 0


def test_host_side_argument_checks_need_no_gpu(lib):
    null = None
    assert lib.slope_prune_24(null, 128, 128, null, null, null, null) == 1            # invalid arg
    buf = ctypes.create_string_buffer(64)
    p = ctypes.cast(buf, ctypes.c_void_p)
    assert lib.slope_prune_24(p, 100, 128, p, p, null, null) == 2                      # shape
    assert lib.slope_linear_fwd(p, 0, p, p, 128, 128, null, null, 0, p, null) == 2     # no tokens
    assert lib.slope_linear_fwd(p, 16, p, p, 128, 128, null, null, 24, p, null) == 1   # rank without factors
    assert lib.slope_adapter_fwd_bwd(7, p, p, p, p, 16, 128, 128, 16, p, p, p, p, p, 0, null) == 1
    assert lib.slope_status_string(6) == b"device-side wait timed out"
    # one of every kind of refusal, all before any CUDA call
    a = (ctypes.addressof(buf) + 15) & ~15                                            # 16-byte aligned host address
    assert lib.slope_linear_fwd(a, 16, a, a, 128, 128, a, a, 24, a, null) == 2         # rank not a multiple of 16
    assert lib.slope_linear_fwd(a + 2, 16, a, a, 128, 128, null, null, 0, a, null) == 3  # misaligned pointer
    assert lib.slope_linear_fwd(a, 16, a, a, 128, 100, null, null, 0, a, null) == 2    # d_in not a multiple of 128
    assert lib.slope_adapter_fwd_bwd(1, a, a, a, a, 16, 128, 128, 16, a, a, a, a, a, 0, null) == 1   # workspace too small
    assert lib.slope_adapter_fwd_bwd(0, a, a, a, a, 16, 128, 128, 0, a, a, a, a, a, 0, null) == 2    # adapter call without a rank
    assert lib.slope_linear_bwd_dw_masked(a, a, 16, 128, 128, null, a, null) == 1      # mask is not optional
    assert lib.slope_prune_nm(a, 128, 128, 2, 3, a, null, null) == 2                   # group size not 2, 4, 8, 16
    assert lib.slope_prune_nm(a, 128, 128, 4, 4, a, null, null) == 2                   # n must be below m
    assert lib.slope_sparse_add(a, a, 1.0, 1.0, 128, 100, a, null) == 2
    assert lib.slope_update_sparse_matrix(a, a, a, 128, 128, null, null) == 1
    assert lib.slope_update_sparse_matrix(a, a, a, 262144, 131072, a, null) == 2       # 2^35 elements: beyond its 32-bit unit indices
    # the one-launch set-up and the weight gradient with the adapter gradients riding along
    assert lib.slope_prune_24_double(a, 128, 128, a, a, null, a, null, null, null) == 1          # a compressed copy missing
    assert lib.slope_prune_24_double(a, 128, 192, a, a, null, a, a, null, null) == 2             # d_in not a multiple of 128
    assert lib.slope_prune_24_double(a, 128, 128, a, a, a + 8, a, a, null, null) == 3            # misaligned mask
    assert lib.slope_bwd_dw_adapter_workspace_bytes(16384, 4096, 4096, 64) >= lib.slope_adapter_workspace_bytes(16384, 4096, 4096, 64)
    assert lib.slope_bwd_dw_adapter_workspace_bytes(16384, 4096, 4096, 0) == 0
    assert lib.slope_linear_bwd_dw_adapter(a, a, a, a, 16, 128, 128, 16, a, a, a, a, a, 0, null) == 1   # workspace too small
    assert lib.slope_linear_bwd_dw_adapter(a, a, a, a, 16, 128, 128, 24, a, a, a, a, a, 1 << 30, null) == 2   # rank
    assert lib.slope_linear_bwd_dw_adapter(a, a, a, null, 16, 128, 128, 16, a, a, a, a, a, 1 << 30, null) == 1   # dT missing
    assert lib.slope_adapter_fwd_bwd(2, null, a, null, a, 16, 128, 128, 16, null, null, null, null, null, 0, null) == 1  # phase 2 needs dT


def test_binding_refuses_to_run_without_the_library(monkeypatch, tmp_path):
    from paper_2608_24070_b200 import binding

    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", tmp_path / "libslope.so")
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        binding.lib()


def test_format_sizes_against_the_papers_memory_accounting(lib):
    """The size functions of the compressed format, per group of four weights, next to the bit counts the
    paper prints: its sparse model holds 2 x (2 x 16 + 3) weight bits, 4 x 8 mask bits, 2 x 16 gradient bits
    and 2 x 2 x 32 optimizer bits per group (ratio 0.68 of dense); inference 35 of 64 bits (0.54)."""
    import math
    import os

    golden = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "memory_accounting.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if len(line) == 2:
                golden[line[0]] = float(line[1])
    # the paper's own arithmetic reproduces its printed ratios
    assert golden["index_bits_per_group"] == math.ceil(math.log2(math.comb(4, 2)))
    paper_sparse = 2 * (2 * 16 + 3) + 4 * 8 + 2 * 16 + 2 * 2 * 32
    assert golden["dense_training_bits"] == 4 * 16 + 4 * 16 + 2 * 4 * 32
    assert abs(paper_sparse / golden["dense_training_bits"] - golden["sparse_training_ratio"]) < 5e-3
    assert golden["sparse_inference_bits"] == 2 * 16 + 3
    assert abs(golden["sparse_inference_bits"] / golden["dense_inference_bits"] - golden["sparse_inference_ratio"]) < 1e-2
    # this library's format: 4-bit codes (2 bits per kept value, what the tensor cores read) and 1-bit masks
    rows, cols = 4096, 11008
    groups = rows * cols // 4
    copy_bits = 8 * (lib.slope_values_bytes(rows, cols) + lib.slope_meta_bytes(rows, cols)) / groups
    mask_bits = 8 * lib.slope_mask_bytes(rows, cols) / groups
    assert copy_bits == 2 * 16 + 4 and mask_bits == 4
    ours_training = 2 * copy_bits + mask_bits + 2 * 16 + 2 * 2 * 32
    assert ours_training == 236 and ours_training < paper_sparse
    assert abs(copy_bits / golden["dense_inference_bits"] - 0.5625) < 1e-12          # one bit per group above the paper's count
