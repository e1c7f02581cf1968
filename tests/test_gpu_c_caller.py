"""GPU: the library driven from a plain C program (no Python, no torch): device memory from the CUDA runtime,
sg_select_topk -> sg_pack_kv on a small ragged batch, results checked inside the C program against loops written there."""
import os
import shutil
import subprocess

import pytest

import paper_2607_28150_b200.binding as sg

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

C_SOURCE = r'''
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <cuda_runtime.h>
#include "smartgen.h"

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("cuda error %d at line %d\n", (int)e_, __LINE__); return 10; } } while (0)

int main(void) {
  enum { B = 2, HKV = 2, HQ = 4, D = 64, L = 2 };
  const int lens[B] = {300, 77}, ks[B] = {40, 9};
  int cu[B + 1] = {0, 300, 377}, cuk[B + 1] = {0, 40, 49};
  const int T = 377, KT = 49;
  size_t n_imp = (size_t)L * HKV * T, n_cache = (size_t)L * T * HKV * D, n_sel = (size_t)L * HKV * KT, n_pk = (size_t)L * KT * HKV * D;
  float* imp = (float*)malloc(n_imp * sizeof(float));
  unsigned short* k = (unsigned short*)malloc(n_cache * 2);
  unsigned short* v = (unsigned short*)malloc(n_cache * 2);
  unsigned seed = 12345u;
  size_t i;
  for (i = 0; i < n_imp; ++i) { seed = seed * 1664525u + 1013904223u; imp[i] = (float)(seed >> 8) / 16777216.0f; }
  for (i = 0; i < n_cache; ++i) { seed = seed * 1664525u + 1013904223u; k[i] = (unsigned short)(seed >> 16); v[i] = (unsigned short)(seed >> 7); }

  int *d_cu, *d_cuk, *d_sel, *d_status; float* d_imp; unsigned short *d_k, *d_v, *d_pk, *d_pv;
  CK(cudaMalloc((void**)&d_cu, 64)); CK(cudaMalloc((void**)&d_cuk, 64)); CK(cudaMalloc((void**)&d_status, 16));
  CK(cudaMalloc((void**)&d_imp, n_imp * 4)); CK(cudaMalloc((void**)&d_sel, n_sel * 4));
  CK(cudaMalloc((void**)&d_k, n_cache * 2)); CK(cudaMalloc((void**)&d_v, n_cache * 2));
  CK(cudaMalloc((void**)&d_pk, n_pk * 2)); CK(cudaMalloc((void**)&d_pv, n_pk * 2));
  CK(cudaMemcpy(d_cu, cu, sizeof cu, cudaMemcpyHostToDevice)); CK(cudaMemcpy(d_cuk, cuk, sizeof cuk, cudaMemcpyHostToDevice));
  CK(cudaMemcpy(d_imp, imp, n_imp * 4, cudaMemcpyHostToDevice));
  CK(cudaMemcpy(d_k, k, n_cache * 2, cudaMemcpyHostToDevice)); CK(cudaMemcpy(d_v, v, n_cache * 2, cudaMemcpyHostToDevice));
  CK(cudaMemset(d_status, 0, 16));

  sg_shape s;
  memset(&s, 0, sizeof s);
  s.num_layers = L; s.batch = B; s.num_q_heads = HQ; s.num_kv_heads = HKV; s.head_dim = D; s.window = 4;
  s.total_tokens = T; s.max_seqlen = 300; s.cu_seqlens = d_cu;
  s.cache_layer_stride = (long long)T * HKV * D; s.cache_token_stride = HKV * D; s.cache_head_stride = D;
  if (sg_select_topk(&s, d_imp, d_cuk, KT, d_sel, NULL, 0, d_status, NULL) != SG_OK) return 20;
  if (sg_pack_kv(&s, d_k, d_v, d_sel, d_cuk, KT, d_pk, d_pv, d_status, NULL) != SG_OK) return 21;
  CK(cudaDeviceSynchronize());

  int* sel = (int*)malloc(n_sel * 4); int status[4];
  unsigned short* pk = (unsigned short*)malloc(n_pk * 2); unsigned short* pv = (unsigned short*)malloc(n_pk * 2);
  CK(cudaMemcpy(sel, d_sel, n_sel * 4, cudaMemcpyDeviceToHost)); CK(cudaMemcpy(status, d_status, 16, cudaMemcpyDeviceToHost));
  CK(cudaMemcpy(pk, d_pk, n_pk * 2, cudaMemcpyDeviceToHost)); CK(cudaMemcpy(pv, d_pv, n_pk * 2, cudaMemcpyDeviceToHost));
  if (status[0] != 0) return 22;
  {
    int l, b, g, j, t;
    for (l = 0; l < L; ++l) for (g = 0; g < HKV; ++g) for (b = 0; b < B; ++b) {
      const float* x = imp + ((size_t)l * HKV + g) * T + cu[b];
      const int* row = sel + ((size_t)l * HKV + g) * KT + cuk[b];
      /* the k_b selected positions are ascending, in range, and no unselected score exceeds a selected one */
      float lowest = 2.0f;
      for (j = 0; j < ks[b]; ++j) {
        if (row[j] < 0 || row[j] >= lens[b] || (j > 0 && row[j] <= row[j - 1])) return 30;
        if (x[row[j]] < lowest) lowest = x[row[j]];
      }
      for (t = 0, j = 0; t < lens[b]; ++t) {
        if (j < ks[b] && row[j] == t) { ++j; continue; }
        if (x[t] > lowest) return 31;
      }
      /* packed rows are the selected cache rows, byte for byte */
      for (j = 0; j < ks[b]; ++j) {
        const size_t src = ((size_t)l * T + cu[b] + row[j]) * HKV * D + (size_t)g * D;
        const size_t dst = (((size_t)l * KT + cuk[b]) * HKV + (size_t)g * ks[b] + j) * D;
        if (memcmp(pk + dst, k + src, D * 2) != 0 || memcmp(pv + dst, v + src, D * 2) != 0) return 32;
      }
    }
  }
  {
    /* the one-call form writes what the two calls wrote */
    int* d_sel2; unsigned short *d_pk2, *d_pv2;
    int* sel2 = (int*)malloc(n_sel * 4);
    unsigned short* pk2 = (unsigned short*)malloc(n_pk * 2); unsigned short* pv2 = (unsigned short*)malloc(n_pk * 2);
    CK(cudaMalloc((void**)&d_sel2, n_sel * 4)); CK(cudaMalloc((void**)&d_pk2, n_pk * 2)); CK(cudaMalloc((void**)&d_pv2, n_pk * 2));
    if (sg_select_pack_kv(&s, d_imp, d_cuk, KT, d_k, d_v, d_sel2, d_pk2, d_pv2, d_status, NULL) != SG_OK) return 40;
    CK(cudaDeviceSynchronize());
    CK(cudaMemcpy(sel2, d_sel2, n_sel * 4, cudaMemcpyDeviceToHost)); CK(cudaMemcpy(status, d_status, 16, cudaMemcpyDeviceToHost));
    CK(cudaMemcpy(pk2, d_pk2, n_pk * 2, cudaMemcpyDeviceToHost)); CK(cudaMemcpy(pv2, d_pv2, n_pk * 2, cudaMemcpyDeviceToHost));
    if (status[0] != 0) return 41;
    if (memcmp(sel2, sel, n_sel * 4) != 0 || memcmp(pk2, pk, n_pk * 2) != 0 || memcmp(pv2, pv, n_pk * 2) != 0) return 42;
  }
  printf("c caller on the gpu ok\n");
  return 0;
}
'''


def test_c_program_drives_select_and_pack(tmp_path):
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    if shutil.which("gcc") is None or not os.path.exists(os.path.join(cuda, "include", "cuda_runtime.h")):
        pytest.skip("no C toolchain / CUDA headers on this box")
    src = tmp_path / "gpu_caller.c"
    src.write_text(C_SOURCE)
    exe = tmp_path / "gpu_caller"
    libdir = os.path.dirname(sg.LIB_PATH)
    subprocess.run(["gcc", "-std=c99", "-Wall", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
                    str(src), "-o", str(exe), "-L", libdir, "-lsmartgen", "-L", os.path.join(cuda, "lib64"), "-lcudart",
                    "-Wl,-rpath," + libdir, "-Wl,-rpath," + os.path.join(cuda, "lib64")], check=True)
    res = subprocess.run([str(exe)], capture_output=True, text=True)
    assert res.returncode == 0 and "c caller on the gpu ok" in res.stdout, (res.returncode, res.stdout, res.stderr)
