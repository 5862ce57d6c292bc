"""CPU-side checks of the C ABI: the library builds for sm_100a, loads, exports every declared entry point,
the ctypes structs have the C sizes, and without a GPU the product path fails loudly instead of falling back."""
import ctypes
import os
import re
import subprocess
import tempfile

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_26219_b200 import build, binding
    build.build()
    return binding.lib()


def declared_symbols():
    text = ""
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if f.endswith(".h"):
            text += open(os.path.join(inc, f)).read()
    return sorted(set(re.findall(r"PATCHKV_API\s+[\w\s\*]+?\b(patchkv_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"patchkv_select_repair", "patchkv_restore", "patchkv_restore_from_host", "patchkv_create",
            "patchkv_destroy", "patchkv_query_status", "patchkv_last_error", "patchkv_record_bytes"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_ctypes_structs_match_the_header():
    from paper_2609_26219_b200 import binding as pk
    src = r'''
#include "patchkv.h"
#include <stdio.h>
int main(void) {
  printf("%zu %zu %zu %zu %zu %zu %zu\n", sizeof(patchkv_config), sizeof(patchkv_geom), sizeof(patchkv_pool),
         sizeof(patchkv_session), sizeof(patchkv_session_host), sizeof(patchkv_select_args), sizeof(patchkv_restore_stats));
  printf("%zu %zu %zu\n", offsetof(patchkv_select_args, attn), offsetof(patchkv_session, block_table), offsetof(patchkv_pool, k_base));
  return 0; }
'''
    with tempfile.TemporaryDirectory() as d:
        c = os.path.join(d, "s.c")
        open(c, "w").write(src)
        exe = os.path.join(d, "s")
        subprocess.check_call(["gcc", "-std=c11", "-I", os.path.join(ROOT, "include"), c, "-o", exe])
        out = subprocess.check_output([exe]).decode().split()
    sizes = [int(x) for x in out]
    want = [ctypes.sizeof(x) for x in (pk.Config, pk.Geom, pk.Pool, pk.Session, pk.Session, pk.SelectArgs, pk.RestoreStats)]
    assert sizes[:7] == want
    assert sizes[7:] == [pk.SelectArgs.attn.offset, pk.Session.block_table.offset, pk.Pool.k_base.offset]


def test_record_bytes_needs_no_gpu(lib):
    from paper_2609_26219_b200 import binding as pk
    assert pk.record_bytes(pk.TAG_BF16, 16, 8, 128, 32) == 65536
    assert pk.record_bytes(pk.TAG_INT8, 16, 8, 128, 32) == 34816
    assert pk.record_bytes(pk.TAG_INT4, 16, 8, 128, 32) == 26624
    assert pk.record_bytes(7, 16, 8, 128, 32) == 0


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_no_gpu_means_a_loud_failure_not_a_fallback(lib):
    from paper_2609_26219_b200 import binding as pk
    with pytest.raises(pk.PatchKVError):
        pk.Context(device=0)


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2609_26219_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f
