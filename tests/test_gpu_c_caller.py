"""GPU: the library driven from a plain C program (no Python, no torch): device memory from the CUDA runtime,
sg_select_topk -> sg_pack_kv on a small ragged batch, then sg_score (with sg_workspace_bytes) and sg_sparse_decode_attn on a
small prompt; every result is checked inside the C program against loops written there."""
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
#include <math.h>
#include <cuda_runtime.h>
#include "smartgen.h"

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("cuda error %d at line %d\n", (int)e_, __LINE__); return 10; } } while (0)

/* bf16 helpers: the test data are multiples of 1/8 of small magnitude, exactly representable in bf16 */
static unsigned short to_bf16(float x) { unsigned int u; memcpy(&u, &x, 4); return (unsigned short)(u >> 16); }
static double from_bf16(unsigned short b) { unsigned int u = (unsigned int)b << 16; float f; memcpy(&f, &u, 4); return (double)f; }

/* sg_score (with sg_workspace_bytes) and sg_sparse_decode_attn from plain C, checked against loops written here */
static int score_and_decode(void) {
  enum { N = 300, HKV = 2, HQ = 4, G = 2, D = 64, W = 4, KSEL = 40, NLOC = 25 };
  static unsigned short q[W * HQ * D], k[N * HKV * D], v[N * HKV * D], qd[HQ * D], pk[KSEL * HKV * D], pv[KSEL * HKV * D], out[HQ * D];
  static float imp[HKV * N], lse[HQ];
  static int loc[HKV * NLOC];
  int cu[2] = {0, N}, cuk[2] = {0, KSEL}, cul[2] = {0, NLOC};
  unsigned seed = 777u;
  int i, g, h, t, c, j;
  for (i = 0; i < W * HQ * D; ++i) { seed = seed * 1664525u + 1013904223u; q[i] = to_bf16((float)((int)(seed >> 27) - 16) / 8.0f); }
  for (i = 0; i < HQ * D; ++i) { seed = seed * 1664525u + 1013904223u; qd[i] = to_bf16((float)((int)(seed >> 27) - 16) / 8.0f); }
  for (i = 0; i < N * HKV * D; ++i) {
    seed = seed * 1664525u + 1013904223u; k[i] = to_bf16((float)((int)(seed >> 27) - 16) / 8.0f);
    seed = seed * 1664525u + 1013904223u; v[i] = to_bf16((float)((int)(seed >> 27) - 16) / 8.0f);
  }
  /* decode list of head g: packed rows = tokens 3, 10, 17, ... (copied here), local rows = tokens 5 + 11*j */
  for (g = 0; g < HKV; ++g) {
    for (j = 0; j < KSEL; ++j) {
      memcpy(pk + ((size_t)g * KSEL + j) * D, k + ((size_t)(3 + 7 * j) * HKV + g) * D, D * 2);
      memcpy(pv + ((size_t)g * KSEL + j) * D, v + ((size_t)(3 + 7 * j) * HKV + g) * D, D * 2);
    }
    for (j = 0; j < NLOC; ++j) loc[g * NLOC + j] = 5 + 11 * j + g;
  }
  unsigned short *d_q, *d_k, *d_v, *d_qd, *d_pk, *d_pv, *d_out; float *d_imp, *d_lse; int *d_cu, *d_cuk, *d_cul, *d_loc, *d_status; void* d_ws;
  CK(cudaMalloc((void**)&d_q, sizeof q)); CK(cudaMalloc((void**)&d_k, sizeof k)); CK(cudaMalloc((void**)&d_v, sizeof v));
  CK(cudaMalloc((void**)&d_qd, sizeof qd)); CK(cudaMalloc((void**)&d_pk, sizeof pk)); CK(cudaMalloc((void**)&d_pv, sizeof pv));
  CK(cudaMalloc((void**)&d_out, sizeof out)); CK(cudaMalloc((void**)&d_imp, sizeof imp)); CK(cudaMalloc((void**)&d_lse, sizeof lse));
  CK(cudaMalloc((void**)&d_cu, 64)); CK(cudaMalloc((void**)&d_cuk, 64)); CK(cudaMalloc((void**)&d_cul, 64)); CK(cudaMalloc((void**)&d_loc, sizeof loc));
  CK(cudaMalloc((void**)&d_status, 16)); CK(cudaMemset(d_status, 0, 16));
  CK(cudaMemcpy(d_q, q, sizeof q, cudaMemcpyHostToDevice)); CK(cudaMemcpy(d_k, k, sizeof k, cudaMemcpyHostToDevice));
  CK(cudaMemcpy(d_v, v, sizeof v, cudaMemcpyHostToDevice)); CK(cudaMemcpy(d_qd, qd, sizeof qd, cudaMemcpyHostToDevice));
  CK(cudaMemcpy(d_pk, pk, sizeof pk, cudaMemcpyHostToDevice)); CK(cudaMemcpy(d_pv, pv, sizeof pv, cudaMemcpyHostToDevice));
  CK(cudaMemcpy(d_cu, cu, sizeof cu, cudaMemcpyHostToDevice)); CK(cudaMemcpy(d_cuk, cuk, sizeof cuk, cudaMemcpyHostToDevice));
  CK(cudaMemcpy(d_cul, cul, sizeof cul, cudaMemcpyHostToDevice)); CK(cudaMemcpy(d_loc, loc, sizeof loc, cudaMemcpyHostToDevice));
  sg_shape s;
  memset(&s, 0, sizeof s);
  s.num_layers = 1; s.batch = 1; s.num_q_heads = HQ; s.num_kv_heads = HKV; s.head_dim = D; s.window = W;
  s.total_tokens = N; s.max_seqlen = N; s.cu_seqlens = d_cu;
  s.cache_layer_stride = (long long)N * HKV * D; s.cache_token_stride = HKV * D; s.cache_head_stride = D;
  {
    size_t need = sg_workspace_bytes(SG_OP_SCORE, &s, 0, 0);
    if (need == 0) return 50;
    CK(cudaMalloc(&d_ws, need));
    if (sg_score(&s, d_q, d_k, d_imp, d_ws, need - 1, d_status, NULL) != SG_ERR_WORKSPACE) return 51;   /* too small: refused */
    if (sg_score(&s, d_q, d_k, d_imp, d_ws, need, d_status, NULL) != SG_OK) return 52;
  }
  if (sg_sparse_decode_attn(&s, d_qd, d_pk, d_pv, d_cuk, KSEL, d_k, d_v, d_loc, d_cul, NLOC, 0.0f, d_out, d_lse, NULL, 0, d_status, NULL) != SG_OK) return 53;
  CK(cudaDeviceSynchronize());
  { int status[4]; CK(cudaMemcpy(status, d_status, 16, cudaMemcpyDeviceToHost)); if (status[0] != 0) return 54; }
  CK(cudaMemcpy(imp, d_imp, sizeof imp, cudaMemcpyDeviceToHost)); CK(cudaMemcpy(out, d_out, sizeof out, cudaMemcpyDeviceToHost));
  CK(cudaMemcpy(lse, d_lse, sizeof lse, cudaMemcpyDeviceToHost));
  /* importance[g][t] = sum over the G heads of g and the W window rows of softmax_t(q . k / sqrt(d)) over keys t <= N - W + i */
  for (g = 0; g < HKV; ++g) {
    static double acc[N], sc[N];
    for (t = 0; t < N; ++t) acc[t] = 0.0;
    for (h = g * G; h < (g + 1) * G; ++h) for (i = 0; i < W; ++i) {
      const int last = N - W + i; double mx = -1e300, sum = 0.0;
      for (t = 0; t <= last; ++t) {
        double dot = 0.0;
        for (c = 0; c < D; ++c) dot += from_bf16(q[((size_t)i * HQ + h) * D + c]) * from_bf16(k[((size_t)t * HKV + g) * D + c]);
        sc[t] = dot / 8.0; if (sc[t] > mx) mx = sc[t];            /* sqrt(64) = 8 */
      }
      for (t = 0; t <= last; ++t) { sc[t] = exp(sc[t] - mx); sum += sc[t]; }
      for (t = 0; t <= last; ++t) acc[t] += sc[t] / sum;
    }
    for (t = 0; t < N; ++t) if (fabs((double)imp[g * N + t] - acc[t]) > 1e-4 * acc[t] + 1e-30) return 60;
  }
  /* decode: attention of every query head over [packed rows of its KV head] ++ [local rows by index] */
  for (h = 0; h < HQ; ++h) {
    static double sc[KSEL + NLOC]; double mx = -1e300, sum = 0.0, o[D];
    g = h / G;
    for (j = 0; j < KSEL + NLOC; ++j) {
      const int tok = j < KSEL ? 3 + 7 * j : loc[g * NLOC + (j - KSEL)]; double dot = 0.0;
      for (c = 0; c < D; ++c) dot += from_bf16(qd[h * D + c]) * from_bf16(k[((size_t)tok * HKV + g) * D + c]);
      sc[j] = dot / 8.0; if (sc[j] > mx) mx = sc[j];
    }
    for (c = 0; c < D; ++c) o[c] = 0.0;
    for (j = 0; j < KSEL + NLOC; ++j) {
      const int tok = j < KSEL ? 3 + 7 * j : loc[g * NLOC + (j - KSEL)]; const double pj = exp(sc[j] - mx);
      sum += pj;
      for (c = 0; c < D; ++c) o[c] += pj * from_bf16(v[((size_t)tok * HKV + g) * D + c]);
    }
    for (c = 0; c < D; ++c) if (fabs(from_bf16(out[h * D + c]) - o[c] / sum) > 2e-2) return 61;
    if (fabs((double)lse[h] - (mx + log(sum))) > 1e-3) return 62;
  }
  return 0;
}

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
  {
    int rc = score_and_decode();
    if (rc != 0) return rc;
  }
  printf("c caller on the gpu ok\n");
  return 0;
}
'''


def test_c_program_drives_the_four_calls(tmp_path):
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    if shutil.which("gcc") is None or not os.path.exists(os.path.join(cuda, "include", "cuda_runtime.h")):
        pytest.skip("no C toolchain / CUDA headers on this box")
    src = tmp_path / "gpu_caller.c"
    src.write_text(C_SOURCE)
    exe = tmp_path / "gpu_caller"
    libdir = os.path.dirname(sg.LIB_PATH)
    subprocess.run(["gcc", "-std=c99", "-Wall", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
                    str(src), "-o", str(exe), "-L", libdir, "-lsmartgen", "-L", os.path.join(cuda, "lib64"), "-lcudart", "-lm",
                    "-Wl,-rpath," + libdir, "-Wl,-rpath," + os.path.join(cuda, "lib64")], check=True)
    res = subprocess.run([str(exe)], capture_output=True, text=True)
    assert res.returncode == 0 and "c caller on the gpu ok" in res.stdout, (res.returncode, res.stdout, res.stderr)
