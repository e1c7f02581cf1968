"""The C-ABI library loads without a GPU, exports every symbol the header declares, and rejects bad
arguments on the host before any launch."""
import ctypes
import os
import re

import paper_2607_28150_b200.binding as sg

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    import glob
    names = set()
    for path in sorted(glob.glob(os.path.join(ROOT, "include", "*.h"))):      # every header, the testing hooks too
        text = re.sub(r"/\*.*?\*/", "", open(path).read(), flags=re.S)
        names |= set(re.findall(r"\b(sg_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported():
    lib = ctypes.CDLL(sg.LIB_PATH)
    names = declared_symbols()
    assert set(sg.EXPORTED) <= set(names) and len(names) >= 7
    for n in names:
        assert hasattr(lib, n), n
        assert hasattr(sg, n), "binding lacks %s" % n


def test_strerror_covers_every_status():
    msgs = [sg.sg_strerror(i) for i in range(7)]
    assert msgs[0] == "ok" and len(set(msgs)) == 7


def test_host_side_argument_checks_need_no_gpu():
    lib = ctypes.CDLL(sg.LIB_PATH)
    lib.sg_pack_kv.restype = ctypes.c_int
    # null shape
    assert lib.sg_pack_kv(None, None, None, None, None, 0, None, None, None, None) == sg.SG_ERR_INVALID
    fake = ctypes.c_void_p(0x1000)
    s = sg.Shape(1, 1, 8, 2, 96, 4, 16, 16, 0x1000, 16 * 2 * 96, 2 * 96, 96)
    assert lib.sg_pack_kv(ctypes.byref(s), fake, fake, fake, fake, 4, fake, fake, None, None) == sg.SG_ERR_UNSUPPORTED
    s = sg.Shape(1, 1, 8, 3, 128, 4, 16, 16, 0x1000, 16 * 3 * 128, 3 * 128, 128)
    assert lib.sg_pack_kv(ctypes.byref(s), fake, fake, fake, fake, 4, fake, fake, None, None) == sg.SG_ERR_UNSUPPORTED
    s = sg.Shape(1, 1, 8, 2, 128, 4, 16, 16, 0x1000, 16 * 256, 256, 128)
    bad = ctypes.c_void_p(0x1004)        # misaligned
    assert lib.sg_pack_kv(ctypes.byref(s), bad, fake, fake, fake, 4, fake, fake, None, None) == sg.SG_ERR_INVALID
    assert lib.sg_pack_kv(ctypes.byref(s), fake, fake, fake, fake, -1, fake, fake, None, None) == sg.SG_ERR_INVALID
    # decode: split-KV partials are merged on chip (cluster mode), no workspace is ever needed
    s = sg.Shape(1, 1, 8, 2, 128, 4, 16384, 16384, 0x1000, 16384 * 256, 256, 128)
    assert sg.sg_workspace_bytes(sg.SG_OP_SPARSE_DECODE_ATTN, s, 8192, 4096) == 0
    assert sg.sg_workspace_bytes(sg.SG_OP_PACK_KV, s, 4, 4) == 0
    lib.sg_sparse_decode_attn.restype = ctypes.c_int
    lib.sg_sparse_decode_attn.argtypes = sg._lib.sg_sparse_decode_attn.argtypes
    s2 = sg.Shape(2, 1, 8, 2, 128, 4, 16384, 16384, 0x1000, 16384 * 256, 256, 128)     # decode takes one layer per call
    rc = lib.sg_sparse_decode_attn(ctypes.byref(s2), fake, fake, fake, fake, 64, fake, fake, fake, fake, 64, 0.0,
                                   fake, None, None, 0, None, None)
    assert rc == sg.SG_ERR_INVALID
    # score: workspace too small is reported before any launch
    lib.sg_score.restype = ctypes.c_int
    lib.sg_score.argtypes = sg._lib.sg_score.argtypes
    assert sg.sg_workspace_bytes(sg.SG_OP_SCORE, s) > 16
    assert lib.sg_score(ctypes.byref(s), fake, fake, fake, fake, 16, None, None) == sg.SG_ERR_WORKSPACE
    # score: more rows per KV head than the shared-memory Q buffer holds is refused, not truncated
    big = sg.Shape(1, 1, 64, 2, 128, 64, 16384, 16384, 0x1000, 16384 * 256, 256, 128)      # G*W = 2048
    assert lib.sg_score(ctypes.byref(big), fake, fake, fake, fake, 1 << 30, None, None) == sg.SG_ERR_UNSUPPORTED


def test_header_is_plain_c_and_a_c_program_links_against_the_library(tmp_path):
    """The boundary is usable from C: the header compiles as C99 (and C++11) with warnings on, and a C program that
    only uses host-side calls links against the shared library and runs without a GPU."""
    import shutil
    import subprocess
    hdr = os.path.join(ROOT, "include", "smartgen.h")
    if shutil.which("gcc") is None:
        return
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only", "-x", "c", hdr], check=True)
    if shutil.which("g++"):
        subprocess.run(["g++", "-std=c++11", "-Wall", "-Werror", "-fsyntax-only", "-x", "c++", hdr], check=True)
    src = tmp_path / "caller.c"
    src.write_text(r'''
#include <stdio.h>
#include <string.h>
#include "smartgen.h"
int main(void) {
  sg_shape s;
  memset(&s, 0, sizeof s);
  /* a null cu_seqlens is rejected on the host, before anything touches a device */
  s.num_layers = 1; s.batch = 1; s.num_q_heads = 8; s.num_kv_heads = 2; s.head_dim = 128; s.window = 4;
  s.total_tokens = 16; s.max_seqlen = 16; s.cache_layer_stride = 16 * 256; s.cache_token_stride = 256; s.cache_head_stride = 128;
  if (sg_pack_kv(&s, 0, 0, 0, 0, 4, 0, 0, 0, 0) != SG_ERR_INVALID) return 1;
  if (sg_transfer_budget(32, 1024, 0.5, 1.0) != 15872) return 2;              /* Eq. 2: M (L-1) T_p / T_t */
  if (sg_transfer_budget(32, 1024, 1e-9, 1.0) != 2048) return 3;              /* clipped to 2M */
  if (sg_speculative_delivered(32, 1024, 2048, 0.10, 10) != 32768) return 4;  /* 10 % per iteration */
  if (strcmp(sg_strerror(SG_OK), "ok") != 0) return 5;
  printf("c caller ok\n");
  return 0;
}
''')
    exe = tmp_path / "caller"
    libdir = os.path.dirname(sg.LIB_PATH)
    subprocess.run(["gcc", "-std=c99", "-Wall", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe),
                    "-L", libdir, "-lsmartgen", "-Wl,-rpath," + libdir], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout
    assert "c caller ok" in out


def test_debug_and_profiling_builds_of_the_scoring_kernel_compile(tmp_path):
    """The library has two optional builds of csrc/score.cu (SG_NVCC_FLAGS of the build script): -DSG_CHECKS adds
    device-side checks of shared-memory carve-up, TMA coordinates and TMEM addresses that report through the status
    word and never trap; -DSG_SCORE_PROFILE adds per-role wait counters.  Both must keep compiling for sm_100a."""
    import shutil
    import subprocess
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        return
    src = os.path.join(ROOT, "paper_2607_28150_b200", "csrc", "score.cu")
    for flag in ("-DSG_CHECKS", "-DSG_SCORE_PROFILE"):
        subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O1", "-std=c++17", "--use_fast_math", flag,
                        "-I", os.path.join(ROOT, "include"), "-I", os.path.dirname(src), "-c", src,
                        "-o", str(tmp_path / "score_dbg.o")], check=True, capture_output=True)
