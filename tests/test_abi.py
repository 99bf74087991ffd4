"""CPU-only checks of the C ABI: the library loads without a GPU, exports every symbol the
header declares, and rejects bad arguments on the host before anything could be launched."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2601_16515_b200 import build
    build.build()
    from paper_2601_16515_b200 import salad
    return salad


def declared_functions():
    text = open(os.path.join(ROOT, "include", "salad.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(salad_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = declared_functions()
    assert set(names) == set(lib.EXPORTS)
    raw = ctypes.CDLL(lib.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), n


def test_status_strings(lib):
    assert lib.status_string(0) == "SALAD_OK"
    for code, name in [(-1, "INVALID_ARG"), (-2, "UNSUPPORTED"), (-3, "WORKSPACE"), (-4, "CAPACITY"),
                       (-5, "CUDA"), (-6, "TIMEOUT"), (-7, "BAD_MASK")]:
        assert lib.status_string(code) == "SALAD_ERR_" + name
    assert lib.status_string(-99) == "SALAD_ERR_UNKNOWN"


def test_workspace_bytes(lib):
    assert lib.salad_workspace_bytes(1, 12, 32760, 128, 128, 64) > 12 * 128 * 128 * 2
    assert lib.salad_workspace_bytes(1, 12, 32760, 128, 128, 64) % 256 == 0
    assert lib.salad_workspace_bytes(1, 2, 1024, 64, 64, 64) > 0
    assert lib.salad_workspace_bytes(1, 2, 1024, 96, 64, 64) == 0       # head dim
    assert lib.salad_workspace_bytes(1, 2, 1024, 64, 32, 64) == 0       # Bq
    assert lib.salad_workspace_bytes(1, 2, 1024, 64, 64, 128) == 0      # Bk
    assert lib.salad_workspace_bytes(0, 2, 1024, 64, 64, 64) == 0
    # independent of N and of the block size, grows with batch*heads
    assert lib.salad_workspace_bytes(2, 1000, 64, 64, 64, 64) > lib.salad_workspace_bytes(2, 12, 64, 64, 64, 64)


def test_host_side_argument_checks(lib):
    L = lib._lib
    P = ctypes.c_void_p
    fake = P(0x1000)            # never dereferenced: validation fails first
    ws_bytes = lib.salad_workspace_bytes(1, 2, 1024, 64, 64, 64)
    rc = L.salad_sparse_attn_fwd(None, fake, fake, fake, None, 1, 2, 1024, 64, 64, 64, fake, fake, 1, 0.0,
                                 fake, ws_bytes, None, None)
    assert rc == lib.SALAD_ERR_INVALID_ARG
    rc = L.salad_sparse_attn_fwd(fake, fake, fake, fake, None, 1, 2, 1024, 96, 64, 64, fake, fake, 1, 0.0,
                                 fake, ws_bytes, None, None)
    assert rc == lib.SALAD_ERR_UNSUPPORTED
    rc = L.salad_sparse_attn_fwd(fake, fake, fake, fake, None, 1, 2, 1024, 64, 64, 64, fake, fake, 3, 0.0,
                                 fake, ws_bytes, None, None)
    assert rc == lib.SALAD_ERR_INVALID_ARG                                  # Hm not in {1, H}
    rc = L.salad_sparse_attn_fwd(fake, fake, fake, fake, None, 1, 2, 1024, 64, 64, 64, fake, fake, 1, -1.0,
                                 fake, ws_bytes, None, None)
    assert rc == lib.SALAD_ERR_INVALID_ARG                                  # negative scale
    rc = L.salad_sparse_attn_fwd(fake, fake, fake, fake, None, 1, 2, 1024, 64, 64, 64, fake, fake, 1, 0.0,
                                 fake, ws_bytes - 1, None, None)
    assert rc == lib.SALAD_ERR_WORKSPACE
    rc = L.salad_sparse_attn_fwd(fake, fake, fake, fake, None, 1, 2, 1024, 64, 64, 64, fake, fake, 1, 0.0,
                                 P(0x1010), ws_bytes, None, None)
    assert rc == lib.SALAD_ERR_WORKSPACE                                    # misaligned workspace
    rc = L.salad_sparse_attn_fwd(P(0x1004), fake, fake, fake, None, 1, 2, 1024, 64, 64, 64, fake, fake, 1, 0.0,
                                 fake, ws_bytes, None, None)
    assert rc == lib.SALAD_ERR_INVALID_ARG                                  # misaligned tensor
    rc = L.salad_fused_fwd(fake, fake, fake, fake, 1, 2, 1024, 64, 64, 64, fake, fake, 1, None, fake, 0.0, 1e-6,
                           fake, ws_bytes, None, None)
    assert rc == lib.SALAD_ERR_INVALID_ARG                                  # missing scale
    rc = L.salad_linear_attn_fwd(fake, fake, fake, fake, None, None, 1, 2, 1024, 64, -1.0, fake, ws_bytes,
                                 None, None)
    assert rc == lib.SALAD_ERR_INVALID_ARG                                  # negative eps
    win = (ctypes.c_int32 * 3)(1, 1, 1)
    assert L.salad_mask_build(0, 4, 4, 64, 64, 1, win, fake, None, 0, None, None) == lib.SALAD_ERR_INVALID_ARG
    assert L.salad_mask_build(4, 4, 4, 64, 64, 1, None, fake, None, 0, None, None) == lib.SALAD_ERR_INVALID_ARG
    assert L.salad_mask_build(4, 4, 4, 64, 64, 1, win, fake, None, 5, None, None) == lib.SALAD_ERR_INVALID_ARG
    assert L.salad_mask_build(4, 4, 4, 64, 64, 1000, win, fake, None, 0, None, None) == lib.SALAD_ERR_UNSUPPORTED
    neg = (ctypes.c_int32 * 3)(1, -1, 1)
    assert L.salad_mask_build(4, 4, 4, 64, 64, 1, neg, fake, None, 0, None, None) == lib.SALAD_ERR_INVALID_ARG


def test_mask_validator_argument_checks(lib):
    L = lib._lib
    P = ctypes.c_void_p
    fake = P(0x1000)
    assert L.salad_csr_validate(None, fake, 10, 4, 8, fake, None) == lib.SALAD_ERR_INVALID_ARG     # no row_ptr
    assert L.salad_csr_validate(fake, fake, 10, 4, 8, None, None) == lib.SALAD_ERR_INVALID_ARG     # no status word
    assert L.salad_csr_validate(fake, None, 10, 4, 8, fake, None) == lib.SALAD_ERR_INVALID_ARG     # capacity without a list
    assert L.salad_csr_validate(fake, fake, -1, 4, 8, fake, None) == lib.SALAD_ERR_INVALID_ARG
    assert L.salad_csr_validate(fake, fake, 10, 0, 8, fake, None) == lib.SALAD_ERR_INVALID_ARG
    assert L.salad_csr_validate(fake, fake, 10, 4, 0, fake, None) == lib.SALAD_ERR_INVALID_ARG
    assert L.salad_set_mask_validation(-5) == lib.SALAD_ERR_INVALID_ARG
    assert L.salad_set_mask_validation(100) == lib.SALAD_OK
    assert L.salad_set_mask_validation(0) == lib.SALAD_OK


def test_no_gpu_means_error_not_fallback(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    L = lib._lib
    fake = ctypes.c_void_p(0x1000)
    ws_bytes = lib.salad_workspace_bytes(1, 2, 1024, 64, 64, 64)
    rc = L.salad_sparse_attn_fwd(fake, fake, fake, fake, None, 1, 2, 1024, 64, 64, 64, fake, fake, 1, 0.0,
                                 fake, ws_bytes, None, None)
    assert rc == lib.SALAD_ERR_CUDA
