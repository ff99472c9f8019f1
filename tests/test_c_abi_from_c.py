"""The boundary is a C ABI: the header must compile as plain C99 (and as C++), and a C program
with no Python and no torch in it must be able to link the library and call it. Host-only: the
calls made here are refused or answered on the host, nothing is launched."""
import os
import shutil
import subprocess

import pytest

import __graft_entry__ as entry
from paper_2607_28633_b200 import binding as tk

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
INCLUDE = os.path.join(ROOT, "include")

PROGRAM = r"""
#include <stdio.h>
#include <string.h>
#include "topkv.h"

int main(void) {
  topkv_layout lo;
  topkv_batch b;
  topkv_endpoint s, t;
  int bad = 0;
  memset(&lo, 0, sizeof lo);
  lo.struct_size = sizeof lo;
  lo.kind = TOPKV_KIND_GQA;
  lo.num_layers = 80; lo.kv_factor = 2; lo.num_kv_heads = 8; lo.head_dim = 128;
  lo.elem_bytes = 2; lo.page_tokens = 16; lo.num_pool_pages = 4096;
  bad += topkv_layout_default_strides(&lo) != TOPKV_OK;
  bad += topkv_kv_bytes(&lo, 4096) != 1342177280LL;              /* Table 1: 1.3 GB */
  bad += topkv_wire_layer_bytes(&lo, 32768) != 134217728LL;
  memset(&b, 0, sizeof b);
  b.struct_size = sizeof b;
  b.num_requests = 8; b.max_pages_per_req = 256; b.total_tokens = 32768;
  /* NULL tables: refused on the host, nothing is launched */
  bad += topkv_pack_layer(0, (const void*)0x1000, &lo, &b, (void*)0x2000, 1 << 30, 0) != TOPKV_ERR_INVALID_ARG;
  bad += topkv_pack_layer(80, (const void*)0x1000, &lo, &b, (void*)0x2000, 1 << 30, 0) >= 0;
  bad += topkv_kernel_launch_count() != 0;
  memset(&s, 0, sizeof s); memset(&t, 0, sizeof t);
  s.struct_size = t.struct_size = sizeof s;
  s.has_nvlink = t.has_nvlink = 1;
  s.nvlink_domain = t.nvlink_domain = "node-a";
  s.node_ip = t.node_ip = "10.0.0.1";
  bad += topkv_select_transport(&s, &t, 0, 1) != TOPKV_TRANSPORT_NVLINK;  /* Alg. 1, first branch */
  bad += topkv_planning_rate(TOPKV_TRANSPORT_PCIE) != 50e9;              /* planning rate of 3.3 */
  printf("version %d, %s, bad %d\n", topkv_version(), topkv_strerror(TOPKV_ERR_CAPACITY), bad);
  return bad;
}
"""


@pytest.fixture(scope="module")
def built():
    entry.build()
    return tk.LIB_PATH


@pytest.mark.parametrize("compiler,flags", [("gcc", ["-std=c99", "-x", "c"]), ("g++", ["-std=c++17", "-x", "c++"])])
def test_header_compiles_on_its_own(compiler, flags, tmp_path):
    if shutil.which(compiler) is None:
        pytest.skip(f"{compiler} is not installed")
    src = tmp_path / "only_header.c"
    src.write_text('#include "topkv.h"\nint main(void) { return 0; }\n')
    subprocess.run([compiler, *flags, "-Wall", "-Wextra", "-pedantic", "-Werror", "-I", INCLUDE, "-fsyntax-only",
                    str(src)], check=True)


def test_a_plain_c_program_links_and_calls_the_library(built, tmp_path):
    if shutil.which("gcc") is None:
        pytest.skip("gcc is not installed")
    src, exe = tmp_path / "caller.c", tmp_path / "caller"
    src.write_text(PROGRAM)
    libdir = os.path.dirname(built)
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-I", INCLUDE, str(src), "-o", str(exe),
                    "-L", libdir, "-ltopkv", f"-Wl,-rpath,{libdir}"], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0, out.stdout + out.stderr
    assert "bad 0" in out.stdout and f"version {tk.topkv_version()}" in out.stdout


@pytest.mark.gpu
def test_a_c_program_runs_pack_and_unpack_on_the_gpu(built, tmp_path):
    """tests/c_caller/roundtrip.c (plain C, gcc): CUDA runtime + the library + the oracle, nothing else. Packs
    and unpacks three layers of a ragged batch and compares wire and destination pool with the
    oracle byte for byte (its exit status says so)."""
    import oracle
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    if shutil.which("gcc") is None or not os.path.exists(os.path.join(cuda, "include", "cuda_runtime.h")):
        pytest.skip("gcc or the CUDA runtime headers are not installed")
    exe = tmp_path / "roundtrip"
    libdir = os.path.dirname(built)
    oracle_so = oracle.build()
    odir = os.path.dirname(oracle_so)
    subprocess.run(["gcc", "-std=c99", "-O1", "-Wall", "-Wextra", os.path.join(ROOT, "tests", "c_caller", "roundtrip.c"),
                    "-o", str(exe), "-I", INCLUDE, "-I", odir, "-I", os.path.join(cuda, "include"),
                    "-L", libdir, "-ltopkv", oracle_so, "-L", os.path.join(cuda, "lib64"), "-lcudart",
                    f"-Wl,-rpath,{libdir}", f"-Wl,-rpath,{odir}", f"-Wl,-rpath,{os.path.join(cuda, 'lib64')}"],
                   check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0, out.stdout + out.stderr
    assert "wire identical, destination pool identical" in out.stdout
