"""The boundary used the way a C program would: no Python binding, no torch -- device memory
from cudaMalloc, plain pointers into the shared library, results copied back and written to a
file that this test compares with the fp64 oracle.
"""
import os
import shutil
import subprocess

import numpy as np
import pytest

from oracle import abs_oracle as orc
from tests.util import assert_sum_close, assert_vec_close, margin_ok, oracle_adamw

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
PKG = os.path.join(ROOT, "paper_2412_21124_b200")
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")

C_SOURCE = r"""
#include <stdio.h>
#include <stdlib.h>
#include <stdint.h>
#include <cuda_runtime_api.h>
#include "abs_normtest.h"

#define CHECK(x) do { if (!(x)) { fprintf(stderr, "failed: %s (line %d)\n", #x, __LINE__); return 1; } } while (0)

int main(int argc, char** argv) {
  CHECK(argc == 3);
  FILE* in = fopen(argv[1], "rb");
  CHECK(in);
  int64_t hdr[2];
  CHECK(fread(hdr, sizeof hdr, 1, in) == 1);
  const int K = (int)hdr[0];
  const int64_t d = hdr[1];
  const size_t vec = (size_t)d * sizeof(float);
  float* host = (float*)malloc(vec * (size_t)(K + 3));
  CHECK(host && fread(host, vec, (size_t)(K + 3), in) == (size_t)(K + 3));
  fclose(in);

  const void* grads[64];
  float *gbar, *p, *m, *v;
  void* stats;
  int64_t* b_next;
  for (int k = 0; k < K; ++k) {
    void* g;
    CHECK(cudaMalloc(&g, vec) == cudaSuccess);
    CHECK(cudaMemcpy(g, host + (size_t)k * d, vec, cudaMemcpyHostToDevice) == cudaSuccess);
    grads[k] = g;
  }
  CHECK(cudaMalloc((void**)&gbar, vec) == cudaSuccess);
  CHECK(cudaMalloc((void**)&p, vec) == cudaSuccess);
  CHECK(cudaMalloc((void**)&m, vec) == cudaSuccess);
  CHECK(cudaMalloc((void**)&v, vec) == cudaSuccess);
  CHECK(cudaMemcpy(p, host + (size_t)K * d, vec, cudaMemcpyHostToDevice) == cudaSuccess);
  CHECK(cudaMemcpy(m, host + (size_t)(K + 1) * d, vec, cudaMemcpyHostToDevice) == cudaSuccess);
  CHECK(cudaMemcpy(v, host + (size_t)(K + 2) * d, vec, cudaMemcpyHostToDevice) == cudaSuccess);
  const int64_t offs[3] = {0, d / 3, d};
  const size_t sbytes = abs_stats_bytes(d, 2);
  CHECK(sbytes > 0);
  CHECK(cudaMalloc(&stats, sbytes) == cudaSuccess);
  CHECK(cudaMalloc((void**)&b_next, sizeof(int64_t)) == cudaSuccess);

  cudaStream_t stream;
  CHECK(cudaStreamCreate(&stream) == cudaSuccess);
  FILE* out = fopen(argv[2], "wb");
  CHECK(out);
  double head[ABS_STATS_HEADER + 2 * ABS_SHARD_STRIDE];
  int64_t bn;

  /* the test alone, two shards */
  int rc = abs_norm_test(grads, K, d, ABS_F32, offs, 2, 0.1, 16, stats, gbar, b_next, stream);
  if (rc != ABS_OK) fprintf(stderr, "abs_norm_test: %s (cuda error %d)\n", abs_status_string(rc),
                            abs_last_cuda_error());
  CHECK(rc == ABS_OK);
  CHECK(cudaStreamSynchronize(stream) == cudaSuccess);
  CHECK(cudaMemcpy(head, stats, sizeof head, cudaMemcpyDeviceToHost) == cudaSuccess);
  CHECK(cudaMemcpy(&bn, b_next, sizeof bn, cudaMemcpyDeviceToHost) == cudaSuccess);
  CHECK(cudaMemcpy(host, gbar, vec, cudaMemcpyDeviceToHost) == cudaSuccess);
  fwrite(head, sizeof head, 1, out);
  fwrite(&bn, sizeof bn, 1, out);
  fwrite(host, vec, 1, out);

  /* the fused step, one shard, gbar not wanted */
  abs_adamw_hparams hp = {1e-3f, 0.9f, 0.999f, 1e-8f, 0.1f};
  rc = abs_normtest_adamw(grads, K, d, ABS_F32, NULL, 1, 0.1, 16, stats, NULL, b_next, p, m, v, &hp,
                          3, stream);
  CHECK(rc == ABS_OK);
  CHECK(cudaStreamSynchronize(stream) == cudaSuccess);
  CHECK(cudaMemcpy(head, stats, sizeof head, cudaMemcpyDeviceToHost) == cudaSuccess);
  CHECK(cudaMemcpy(&bn, b_next, sizeof bn, cudaMemcpyDeviceToHost) == cudaSuccess);
  fwrite(head, sizeof head, 1, out);
  fwrite(&bn, sizeof bn, 1, out);
  float* state[3] = {p, m, v};
  for (int i = 0; i < 3; ++i) {
    CHECK(cudaMemcpy(host, state[i], vec, cudaMemcpyDeviceToHost) == cudaSuccess);
    fwrite(host, vec, 1, out);
  }
  fclose(out);
  /* a rejected call launches nothing and says why */
  CHECK(abs_norm_test(grads, 0, d, ABS_F32, NULL, 1, 0.1, 16, stats, gbar, b_next, stream) == ABS_ERR_RANGE);
  CHECK(abs_norm_test(grads, K, d, ABS_F32, NULL, 1, 0.1, 16, stats, (float*)grads[0], b_next, stream) == ABS_ERR_ALIAS);
  printf("ok\n");
  return 0;
}
"""


@pytest.mark.skipif(shutil.which("gcc") is None, reason="needs gcc")
def test_c_program_drives_the_library(tmp_path):
    if not os.path.exists(os.path.join(CUDA, "include", "cuda_runtime_api.h")):
        pytest.skip("CUDA runtime headers not found")
    K, d, eta, b_cur, step = 5, 70_001, 0.1, 16, 3
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)
    rng = np.random.default_rng(17)
    while True:
        mu = rng.standard_normal(d) * 0.01
        grads = [(mu + 0.05 * rng.standard_normal(d)).astype(np.float32) for _ in range(K)]
        offs = [0, d // 3, d]
        ref2 = orc.norm_test(grads, eta, b_cur, shard_offsets=offs)
        if margin_ok(ref2["T"], b_cur):
            break
    p0 = (rng.standard_normal(d) * 0.02).astype(np.float32)
    m0 = (rng.standard_normal(d) * 0.001).astype(np.float32)
    v0 = (rng.random(d) * 1e-4).astype(np.float32)
    inp = tmp_path / "in.bin"
    with open(inp, "wb") as f:
        np.array([K, d], dtype=np.int64).tofile(f)
        for a in grads + [p0, m0, v0]:
            a.tofile(f)
    src = tmp_path / "drive.c"
    src.write_text(C_SOURCE)
    exe = tmp_path / "drive"
    libdir = os.path.join(CUDA, "lib64")
    subprocess.check_call(["gcc", "-std=c99", "-O1", "-I", os.path.join(ROOT, "include"),
                           "-I", os.path.join(CUDA, "include"), str(src), "-o", str(exe),
                           "-L", PKG, "-labs_normtest", "-L", libdir, "-lcudart",
                           "-Wl,-rpath," + PKG, "-Wl,-rpath," + libdir])
    outp = tmp_path / "out.bin"
    run = subprocess.run([str(exe), str(inp), str(outp)], stdout=subprocess.PIPE,
                         stderr=subprocess.PIPE, timeout=300)
    assert run.returncode == 0, run.stderr.decode()[-2000:]
    assert run.stdout.decode().strip() == "ok"

    nh = 8 + 2 * 4
    with open(outp, "rb") as f:
        head1 = np.fromfile(f, dtype=np.float64, count=nh)
        bn1 = int(np.fromfile(f, dtype=np.int64, count=1)[0])
        gbar = np.fromfile(f, dtype=np.float32, count=d)
        head2 = np.fromfile(f, dtype=np.float64, count=nh)
        bn2 = int(np.fromfile(f, dtype=np.int64, count=1)[0])
        p1, m1, v1 = (np.fromfile(f, dtype=np.float32, count=d) for _ in range(3))
    # the test alone: totals, both shard records, decision, gbar
    assert_sum_close(head1[0], ref2["n2"], "n2")
    assert_sum_close(head1[1], ref2["S"], "S")
    for s in range(2):
        assert_sum_close(head1[8 + 4 * s], ref2["shards"][s][0], "n2 of shard %d" % s)
        assert_sum_close(head1[8 + 4 * s + 1], ref2["shards"][s][1], "S of shard %d" % s)
    assert bn1 == ref2["b_next"] and int(head1[4]) == ref2["flags"] and head1[5] == K
    assert_vec_close(gbar.astype(np.float64), ref2["gbar"], "gbar")
    # the fused step
    ref1 = orc.norm_test(grads, eta, b_cur)
    assert_sum_close(head2[1], ref1["S"], "S (fused)")
    assert bn2 == ref1["b_next"]
    w_ref, m_ref, v_ref = oracle_adamw(orc, p0, m0, v0, ref1["gbar"], hp, step)
    assert_vec_close(p1.astype(np.float64), w_ref, "params")
    assert_vec_close(m1.astype(np.float64), m_ref, "m")
    assert_vec_close(v1.astype(np.float64), v_ref, "v")
