"""The C-ABI library builds, loads and exports what include/kmq.h declares;
host-side argument validation returns status codes (no GPU needed: every call
here is rejected before anything is launched)."""
import os
import re

import pytest

from paper_2602_15563_b200 import build as kb
from paper_2602_15563_b200 import kmq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    kb.build()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "kmq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kmq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    names = declared_functions()
    assert {"kmq_pack", "kmq_linear", "kmq_dequant_to_bf16", "kmq_unpack"} <= set(names)
    handle = kmq.lib()
    for name in names:
        assert getattr(handle, name) is not None
        assert name in kmq.SIGNATURES, f"{name} is declared in kmq.h but not bound"
        assert hasattr(kmq, name) or name == "kmq_status_string"
    assert sorted(kmq.SIGNATURES) == names


def test_sizes_and_strings():
    assert kmq.kmq_version() >= 100
    assert kmq.kmq_packed_bytes(4096, 4096, 1) == 4096 * 4096 // 8
    assert kmq.kmq_packed_bytes(8192, 28672, 4) == 8192 * 28672 // 2
    assert kmq.kmq_packed_bytes(3, 16, 2) == 3 * 4
    assert kmq.kmq_packed_bytes(3, 8, 2) == 0          # K not a multiple of 16
    assert kmq.kmq_packed_bytes(3, 32, 3) == 0
    assert kmq.kmq_packed_bytes(3, 32, 1, layout=9) == 0
    assert kmq.status_string(0) == "ok"
    assert "bits" in kmq.status_string(kmq.KMQ_ERR_BITS)
    assert kmq.status_string(1234) == "unknown status"
    assert kmq.kmq_linear_num_launches(4096, 4096, 4, 1) in (1, 2)
    assert kmq.kmq_linear_num_launches(4096, 4095, 4, 1) == 0
    assert isinstance(kmq.kmq_linear_variant(4096, 4096, 2, 1), str)
    assert kmq.kmq_workspace_bytes(4096, 4096, 3, 1) == 0
    T = kmq.KMQ_LAYOUT_TUNED
    assert kmq.kmq_packed_bytes(4096, 4096, 2, layout=T) == 4096 * 4096 // 4      # whole tiles and steps: no padding
    assert kmq.kmq_packed_bytes(17, 32, 1, layout=T) == 2 * 1 * 1024               # 2 tiles x 1 step x 1 KB
    assert kmq.kmq_packed_bytes(16, 8 * 17, 4, layout=T) == 1 * 2 * 1024            # 17 words per row -> 2 steps
    assert kmq.kmq_linear_num_launches(4096, 4096, 2, 17) == 3                    # canonical: passes of 8 batch rows
    assert kmq.kmq_linear_num_launches(4096, 4096, 2, 17, layout=T) == 1          # tuned: one multi-tile launch
    assert kmq.kmq_linear_num_launches(4096, 4096, 1, 64, layout=T) == 2          # b = 1: 32 batch rows per launch
    assert kmq.kmq_linear_variant(4096, 4096, 2, 1, layout=7) == "invalid"
    assert kmq.kmq_linear_variant(4096, 4096, 2, 1, layout=T) != kmq.kmq_linear_variant(4096, 4096, 2, 1)


def test_block_sample_count():
    assert kmq.kmq_block_sample_count(4, 128, 100) == 100          # stride 5: 103 positions, the first 100
    assert kmq.kmq_block_sample_count(4, 128, 10 ** 6) == 512
    assert kmq.kmq_block_sample_count(4, 128, 512) == 512
    assert kmq.kmq_block_sample_count(4, 128, 300) == 300          # stride 1
    assert kmq.kmq_block_sample_count(4, 100, 10) == 0             # K not a multiple of 64


A = 0x1000  # a non-NULL, 16-byte aligned fake address; never dereferenced: validation fails first


@pytest.mark.parametrize("call,expected", [
    (lambda: kmq.kmq_pack(0, 4, 32, 1, A, stream=0, check=False), kmq.KMQ_ERR_NULL),
    (lambda: kmq.kmq_pack(A, 4, 32, 1, 0, stream=0, check=False), kmq.KMQ_ERR_NULL),
    (lambda: kmq.kmq_pack(A, 4, 32, 3, A, stream=0, check=False), kmq.KMQ_ERR_BITS),
    (lambda: kmq.kmq_pack(A, 0, 32, 1, A, stream=0, check=False), kmq.KMQ_ERR_SHAPE),
    (lambda: kmq.kmq_pack(A, 4, 20, 4, A + 64, stream=0, check=False), kmq.KMQ_ERR_SHAPE),
    (lambda: kmq.kmq_pack(A, 4, 31, 1, A, stream=0, check=False), kmq.KMQ_ERR_SHAPE),
    (lambda: kmq.kmq_pack(A, 4, 32, 1, A, layout=5, stream=0, check=False), kmq.KMQ_ERR_LAYOUT),
    (lambda: kmq.kmq_pack(A + 4, 4, 32, 1, A, stream=0, check=False), kmq.KMQ_ERR_ALIGN),
    (lambda: kmq.kmq_unpack(A, 4, 32, 1, 0, stream=0, check=False), kmq.KMQ_ERR_NULL),
    (lambda: kmq.kmq_unpack(A, 4, 8, 2, A, stream=0, check=False), kmq.KMQ_ERR_SHAPE),
    (lambda: kmq.kmq_linear(A, A, A, 0, 4, 32, 1, 1, stream=0, check=False), kmq.KMQ_ERR_NULL),
    (lambda: kmq.kmq_linear(A, A, A, A, 4, 32, 8, 1, stream=0, check=False), kmq.KMQ_ERR_BITS),
    (lambda: kmq.kmq_linear(A, A, A, A, 4, 32, 1, 0, stream=0, check=False), kmq.KMQ_ERR_SHAPE),
    (lambda: kmq.kmq_linear(A, A, A, A, 4, 0, 1, 1, stream=0, check=False), kmq.KMQ_ERR_SHAPE),
    (lambda: kmq.kmq_linear(A, A, A, A, 4, 32, 1, 1, layout=9, stream=0, check=False), kmq.KMQ_ERR_LAYOUT),
    (lambda: kmq.kmq_linear(A, A + 2, A, A, 4, 32, 1, 1, stream=0, check=False), kmq.KMQ_ERR_ALIGN),
    (lambda: kmq.kmq_linear_host(A, A, 0, A, 4, 32, 1, 1, A, A, stream=0, check=False), kmq.KMQ_ERR_NULL),
    (lambda: kmq.kmq_linear_host(A, A, A, A, 4, 32, 5, 1, A, A, stream=0, check=False), kmq.KMQ_ERR_BITS),
    (lambda: kmq.kmq_dequant_to_bf16(A, 0, A, 4, 32, 1, stream=0, check=False), kmq.KMQ_ERR_NULL),
    (lambda: kmq.kmq_dequant_to_bf16(A, A, A, 4, 12, 4, stream=0, check=False), kmq.KMQ_ERR_SHAPE),
    (lambda: kmq.kmq_dequant_to_bf16(A, A, A + 8, 4, 32, 1, stream=0, check=False), kmq.KMQ_ERR_ALIGN),
    (lambda: kmq.kmq_block_table_pack(A, 0, 4, 128, 1, A, stream=0, check=False), kmq.KMQ_ERR_NULL),
    (lambda: kmq.kmq_block_table_pack(A, A, 4, 128, 8, A, stream=0, check=False), kmq.KMQ_ERR_BITS),
    (lambda: kmq.kmq_block_table_pack(A, A, 4, 96, 2, A, stream=0, check=False), kmq.KMQ_ERR_SHAPE),
    (lambda: kmq.kmq_block_table_unpack(A, 4, 128, 2, A, A + 2, stream=0, check=False), kmq.KMQ_ERR_ALIGN),
    (lambda: kmq.kmq_block_table_linear(A, A, A, 0, 4, 128, 1, 1, stream=0, check=False), kmq.KMQ_ERR_NULL),
    (lambda: kmq.kmq_block_table_linear(A, A, A, A, 4, 128, 3, 1, stream=0, check=False), kmq.KMQ_ERR_BITS),
    (lambda: kmq.kmq_block_table_linear(A, A, A, A, 4, 128, 1, 0, stream=0, check=False), kmq.KMQ_ERR_SHAPE),
    (lambda: kmq.kmq_block_table_linear(A, A + 8, A, A, 4, 128, 1, 1, stream=0, check=False), kmq.KMQ_ERR_ALIGN),
    (lambda: kmq.kmq_kmeans_rows(0, 4, 64, 2, 20, A, stream=0, check=False), kmq.KMQ_ERR_NULL),
    (lambda: kmq.kmq_kmeans_rows(A, 4, 64, 3, 20, A, stream=0, check=False), kmq.KMQ_ERR_BITS),
    (lambda: kmq.kmq_kmeans_rows(A, 4, 32769, 2, 20, A, stream=0, check=False), kmq.KMQ_ERR_SHAPE),
    (lambda: kmq.kmq_kmeans_rows(A, 4, 8, 4, 20, A, stream=0, check=False), kmq.KMQ_ERR_SHAPE),
    (lambda: kmq.kmq_kmeans_rows(A, 4, 64, 2, -1, A, stream=0, check=False), kmq.KMQ_ERR_SHAPE),
    (lambda: kmq.kmq_kmeans_rows(A, 4, 64, 2, 20, A, A + 8, stream=0, check=False), kmq.KMQ_ERR_ALIGN),
    (lambda: kmq.kmq_assign_pack(A, 0, 4, 32, 1, 0, A, stream=0, check=False), kmq.KMQ_ERR_NULL),
    (lambda: kmq.kmq_assign_pack(A, A, 4, 32, 8, 0, A, stream=0, check=False), kmq.KMQ_ERR_BITS),
    (lambda: kmq.kmq_assign_pack(A, A, 4, 24, 2, 0, A, stream=0, check=False), kmq.KMQ_ERR_SHAPE),
    (lambda: kmq.kmq_assign_pack(A, A, 4, 32, 1, 5, A, stream=0, check=False), kmq.KMQ_ERR_LAYOUT),
    (lambda: kmq.kmq_assign_pack(A + 4, A, 4, 32, 1, 0, A, stream=0, check=False), kmq.KMQ_ERR_ALIGN),
    (lambda: kmq.kmq_quantize_rows(A, 4, 65536, 1, 20, 0, A, A, stream=0, check=False), kmq.KMQ_ERR_SHAPE),
    (lambda: kmq.kmq_quantize_rows(A, 4, 64, 1, 20, 0, A, 0, stream=0, check=False), kmq.KMQ_ERR_NULL),
    (lambda: kmq.kmq_block_scales(A, 4, 96, 0, A, stream=0, check=False), kmq.KMQ_ERR_SHAPE),
    (lambda: kmq.kmq_block_scales(A, 4, 128, 2, A, stream=0, check=False), kmq.KMQ_ERR_LAYOUT),
    (lambda: kmq.kmq_block_scales(A, 4, 128, 0, 0, stream=0, check=False), kmq.KMQ_ERR_NULL),
    (lambda: kmq.kmq_block_sample(A, A, 4, 128, 0, A, stream=0, check=False), kmq.KMQ_ERR_SHAPE),
    (lambda: kmq.kmq_block_assign_pack(A, A, A, 4, 128, 3, A, stream=0, check=False), kmq.KMQ_ERR_BITS),
    (lambda: kmq.kmq_block_assign_pack(A, A, A + 2, 4, 128, 4, A, stream=0, check=False), kmq.KMQ_ERR_ALIGN),
    (lambda: kmq.kmq_block_quantize(A, 4, 128, 4, 0, 20, 8, A, A, A, A, stream=0, check=False), kmq.KMQ_ERR_SHAPE),
    (lambda: kmq.kmq_block_quantize(A, 4, 128, 4, 0, 20, 40000, A, A, A, 0, stream=0, check=False), kmq.KMQ_ERR_NULL),
    (lambda: kmq.kmq_block_quantize(A, 4096, 4096, 4, 0, 20, 40000, A, A, A, A, stream=0, check=False), kmq.KMQ_ERR_SHAPE),
])
def test_validation_status_codes(call, expected):
    assert call() == expected


def test_check_raises_with_message():
    with pytest.raises(kmq.KmqError) as e:
        kmq.kmq_pack(A, 4, 32, 7, A, stream=0)
    assert e.value.status == kmq.KMQ_ERR_BITS and "bits" in str(e.value)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(kmq, "_lib", None)
    monkeypatch.setattr(kmq, "_LIB_PATH", str(tmp_path / "libkmq.so"))
    with pytest.raises(ImportError, match="no CPU fallback"):
        kmq.kmq_version()


def test_product_code_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_2602_15563_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle\b|#include\s+[\"<].*oracle", src, flags=re.M), f
                assert "import_module(\"oracle" not in src and "oracle/" not in src, f
