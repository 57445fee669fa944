"""The C-ABI library builds, loads and exports every symbol the header declares
(no compute without a GPU), and its host-side checks answer with error codes."""
import ctypes as C
import os
import re

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    import paper_2502_14477_b200 as esa
    esa.build_library()
    return esa.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "esa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(esa_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2502_14477_b200.binding import EXPORTED_SYMBOLS
    names = declared_symbols()
    assert len(names) >= 16
    for n in names:
        assert hasattr(lib, n), f"{n} declared in esa.h but not exported"
    assert set(names) == set(EXPORTED_SYMBOLS)


def test_status_strings(lib):
    assert lib.esa_status_string(0) == b"ESA_OK"
    assert lib.esa_status_string(3) == b"ESA_ERR_CAPACITY"
    assert lib.esa_status_string(99) == b"ESA_ERR_UNKNOWN"


def test_workspace_bytes_and_config_validation(lib):
    import paper_2502_14477_b200 as esa
    good = esa.EsaConfig(32, 8, 128, 128, 128, 2048, 4096, 3, 512, 8, 131072 + 256).to_c()
    n = lib.esa_workspace_bytes(C.byref(good))
    # two fp32-sized score buffers per cached token and sequence dominate
    assert n > 2 * 4 * 8 * (131072 + 256) and n < (1 << 30)
    for bad in (esa.EsaConfig(32, 5, 128, 128, 128, 2048, 4096, 3, 512, 8, 1024),      # H % H_G
                esa.EsaConfig(32, 8, 96, 128, 128, 2048, 4096, 3, 512, 8, 1024),       # head_dim
                esa.EsaConfig(32, 8, 128, 100, 128, 2048, 4096, 3, 512, 8, 1024),      # d_c
                esa.EsaConfig(32, 8, 128, 128, 128, 2048, 0, 3, 512, 8, 1024),         # top_k
                esa.EsaConfig(32, 8, 128, 128, 128, 2048, 4096, 3, 512, 65, 1024),     # max_batch
                esa.EsaConfig(32, 8, 128, 128, 128, 2048, 4096, 3, 512, 8, 1 << 31)):  # max_tokens
        assert lib.esa_workspace_bytes(C.byref(bad.to_c())) == 0
    assert lib.esa_workspace_bytes(None) == 0


def test_null_handles_are_rejected(lib):
    assert lib.esa_destroy(None) == 1
    assert lib.esa_launch_count(None) == -1
    assert lib.esa_last_device_status(None, None) == 1
    assert lib.esa_set_compressors(None, None, None, None, None) == 1
    assert lib.esa_select(None, 1, None, 1, None, None, None, None) == 1
    h = C.c_void_p()
    assert lib.esa_create(None, C.byref(h)) == 1
    import paper_2502_14477_b200 as esa
    bad = esa.EsaConfig(32, 5, 128, 128, 128, 2048, 4096, 3, 512, 8, 1024).to_c()
    assert lib.esa_create(C.byref(bad), C.byref(h)) == 2 and not h.value


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device error path")
def test_create_without_a_device_reports_cuda_error(lib):
    import paper_2502_14477_b200 as esa
    with pytest.raises(esa.EsaError) as e:
        esa.Esa(esa.EsaConfig(8, 2, 64, 32, 4, 512, 256, 3, 128, 1, 4096))
    assert e.value.status == 4


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2502_14477_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        binding.load_library()
