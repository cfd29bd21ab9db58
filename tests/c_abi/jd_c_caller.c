/* A plain C99 caller of the library's C ABI: no C++, no Python, no torch. It reads one problem
 * from a binary file, registers the head on the device, runs jd_verify_host and writes the
 * outputs to a second file. The GPU test builds it with gcc, feeds it a seeded workload and
 * compares what it wrote with the CPU checker.
 *
 * File layout (little endian): int32 B, M, d, V, mode; float tau, b_judge; uint64 seed;
 * then bf16 W[V*d], bf16 w_judge[d], bf16 H[B*(M+1)*d], int32 tokens[B*M], float draft[B*M*V].
 * Output: int32 device_status, variant, launches; int32 accept_len[B], next_token[B];
 * float judge[B*M], p[B*M], q[B*M]; uint8 masks[B*M]; float row_max[R], row_lse[R]. */
#include <cuda_runtime_api.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "jd.h"

#define CHECK(cond, msg) do { if (!(cond)) { fprintf(stderr, "jd_c_caller: %s\n", msg); return 1; } } while (0)

static void* slurp(FILE* f, size_t bytes) {
  void* p = malloc(bytes ? bytes : 1);
  if (p && fread(p, 1, bytes, f) != bytes) { free(p); return NULL; }
  return p;
}

int main(int argc, char** argv) {
  CHECK(argc == 3, "usage: jd_c_caller <problem file> <result file>");
  FILE* f = fopen(argv[1], "rb");
  CHECK(f, "cannot open the problem file");
  int32_t hdr[5];
  float tau, b_judge;
  uint64_t seed;
  CHECK(fread(hdr, 4, 5, f) == 5 && fread(&tau, 4, 1, f) == 1 && fread(&b_judge, 4, 1, f) == 1 &&
        fread(&seed, 8, 1, f) == 1, "short header");
  const int32_t B = hdr[0], M = hdr[1], d = hdr[2], V = hdr[3], mode = hdr[4];
  const size_t R = (size_t)B * (M + 1), BM = (size_t)B * M;
  uint16_t* W = slurp(f, (size_t)V * d * 2);
  uint16_t* wj = slurp(f, (size_t)d * 2);
  uint16_t* H = slurp(f, R * d * 2);
  int32_t* x = slurp(f, BM * 4);
  float* dl = slurp(f, BM * (size_t)V * 4);
  fclose(f);
  CHECK(W && wj && H && x && dl, "short problem file");

  void *dW = NULL, *dwj = NULL;
  CHECK(cudaMalloc(&dW, (size_t)V * d * 2) == cudaSuccess && cudaMalloc(&dwj, (size_t)d * 2) == cudaSuccess, "cudaMalloc");
  CHECK(cudaMemcpy(dW, W, (size_t)V * d * 2, cudaMemcpyHostToDevice) == cudaSuccess &&
        cudaMemcpy(dwj, wj, (size_t)d * 2, cudaMemcpyHostToDevice) == cudaSuccess, "cudaMemcpy");

  jd_config_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.max_B = B; cfg.max_M = M; cfg.d = d; cfg.V = V; cfg.dtype = JD_DTYPE_BF16; cfg.device = 0;
  jd_handle_t h = NULL;
  jd_status_t s = jd_create(&h, &cfg);
  if (s != JD_OK) { fprintf(stderr, "jd_create: %s\n", jd_status_string(s)); return 2; }
  s = jd_set_head(h, dW, dwj, b_judge);
  if (s != JD_OK) { fprintf(stderr, "jd_set_head: %s\n", jd_status_string(s)); return 2; }

  int32_t* accept = calloc(B, 4);
  int32_t* next = calloc(B, 4);
  float* judge = calloc(BM, 4);
  float* p = calloc(BM, 4);
  float* q = calloc(BM, 4);
  uint8_t* masks = calloc(BM, 1);
  float* row_max = calloc(R, 4);
  float* row_lse = calloc(R, 4);
  CHECK(accept && next && judge && p && q && masks && row_max && row_lse, "calloc");

  jd_verify_args_t a;
  memset(&a, 0, sizeof a);
  a.B = B; a.M = M; a.H = H; a.draft_tokens = x; a.draft_logits = dl;
  a.tau = tau; a.seed = seed; a.mode = (jd_mode_t)mode;
  a.resample = JD_RESAMPLE_RESIDUAL; a.variant = JD_VARIANT_AUTO; a.rule = JD_RULE_SAMPLING; a.top_k = 1;
  a.norm = JD_NORM_NONE; a.rms_eps = 0.f;
  a.accept_len = accept; a.next_token = next; a.judge_scores = judge; a.p_draft = p; a.q_draft = q;
  a.masks = masks; a.row_max = row_max; a.row_lse = row_lse; a.logits_debug = NULL;
  s = jd_verify_host(h, &a, NULL);
  if (s != JD_OK) { fprintf(stderr, "jd_verify_host: %s\n", jd_status_string(s)); return 3; }
  int dev_status = -1, variant = 0, launches = 0;
  CHECK(jd_last_device_status(h, &dev_status) == JD_OK && jd_last_launch_info(h, &variant, &launches) == JD_OK, "status");

  FILE* o = fopen(argv[2], "wb");
  CHECK(o, "cannot open the result file");
  const int32_t head[3] = {dev_status, variant, launches};
  fwrite(head, 4, 3, o);
  fwrite(accept, 4, B, o); fwrite(next, 4, B, o);
  fwrite(judge, 4, BM, o); fwrite(p, 4, BM, o); fwrite(q, 4, BM, o);
  fwrite(masks, 1, BM, o);
  fwrite(row_max, 4, R, o); fwrite(row_lse, 4, R, o);
  fclose(o);

  jd_destroy(h);
  cudaFree(dW); cudaFree(dwj);
  free(W); free(wj); free(H); free(x); free(dl);
  free(accept); free(next); free(judge); free(p); free(q); free(masks); free(row_max); free(row_lse);
  return 0;
}
