/* A plain C caller of the PSA library: no Python, no C++, only psa.h and the CUDA runtime for
 * device memory.  With q = 0 and v = 1 every attended row must come out as exactly 1.0 and
 * lse = ln(number of attended keys); rows without any attended key block as 0 and -inf.
 * Then the joint video + text call with v = 1 on the text tokens only (every row comes out as the
 * share of text keys among its attended keys), and the search entry points (an all-covering candidate
 * has loss exactly 0; the selection follows the hand-worked cases).
 * Prints "OK" and exits 0 on success. */
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "psa.h"

#define CHECK(x) do { int rc_ = (x); if (rc_ != 0) { fprintf(stderr, "%s -> %d\n", #x, rc_); return 1; } } while (0)

int main(void) {
  const int T = 4, H = 16, W = 16, L = T * H * W, D = 128, heads = 2;
  /* head 0: |dt - 1| <= 1, i.e. each query block attends itself and the next two temporal blocks;
   * head 1: only the next one (the last block attends nothing) */
  psa_head_params hp[2] = {{2, 1, 0, 1, 0, 0}, {1, 1, 0, 1, 0, 0}};
  psa_problem prob;
  memset(&prob, 0, sizeof(prob));
  prob.n_heads = heads; prob.head_dim = D; prob.tile.bt = 1; prob.tile.bh = 16; prob.tile.bw = 16;
  prob.scale = 0.088388f; prob.stride_head = (int64_t)L * D; prob.stride_token = D;

  int64_t nb = 0, nnz = 0;
  CHECK(psa_mask_sizes(hp, &prob, T, H, W, &nb, &nnz));
  if (nb != 4 || nnz != 9 + 3) { fprintf(stderr, "sizes nb=%lld nnz=%lld\n", (long long)nb, (long long)nnz); return 1; }

  const size_t n = (size_t)heads * L * D;
  uint16_t* h_buf = (uint16_t*)malloc(n * 2);
  uint16_t *d_q, *d_k, *d_v, *d_o; float* d_lse; uint8_t* d_mask; int32_t *d_rp, *d_col;
  CHECK(cudaMalloc((void**)&d_q, n * 2)); CHECK(cudaMalloc((void**)&d_k, n * 2));
  CHECK(cudaMalloc((void**)&d_v, n * 2)); CHECK(cudaMalloc((void**)&d_o, n * 2));
  CHECK(cudaMalloc((void**)&d_lse, sizeof(float) * heads * L));
  CHECK(cudaMalloc((void**)&d_mask, heads * nb * nb)); CHECK(cudaMalloc((void**)&d_rp, sizeof(int32_t) * (heads * nb + 1)));
  CHECK(cudaMalloc((void**)&d_col, sizeof(int32_t) * nnz));
  CHECK(cudaMemset(d_q, 0, n * 2));                                   /* q = 0 */
  for (size_t i = 0; i < n; ++i) h_buf[i] = (uint16_t)(0x3F80 ^ ((i * 2654435761u >> 7) & 0x7F));  /* k: arbitrary values near 1 */
  CHECK(cudaMemcpy(d_k, h_buf, n * 2, cudaMemcpyHostToDevice));
  for (size_t i = 0; i < n; ++i) h_buf[i] = 0x3F80;                   /* v = 1.0 */
  CHECK(cudaMemcpy(d_v, h_buf, n * 2, cudaMemcpyHostToDevice));

  CHECK(psa_mask_build(hp, &prob, T, H, W, d_mask, d_rp, d_col, nnz, NULL));
  CHECK(psa_attn_fwd(d_q, d_k, d_v, d_o, d_lse, hp, &prob, T, H, W, NULL));
  int32_t detail = 0;
  CHECK(psa_last_device_status(&detail));

  int32_t rp[9]; uint8_t mask[32];
  CHECK(cudaMemcpy(rp, d_rp, sizeof(rp), cudaMemcpyDeviceToHost));
  CHECK(cudaMemcpy(mask, d_mask, sizeof(mask), cudaMemcpyDeviceToHost));
  const int32_t want_rp[9] = {0, 3, 6, 8, 9, 10, 11, 12, 12};
  const uint8_t want_mask[32] = {1,1,1,0, 0,1,1,1, 0,0,1,1, 0,0,0,1,   0,1,0,0, 0,0,1,0, 0,0,0,1, 0,0,0,0};
  if (memcmp(rp, want_rp, sizeof(rp)) || memcmp(mask, want_mask, sizeof(mask))) { fprintf(stderr, "mask/row_ptr mismatch\n"); return 1; }

  float* lse = (float*)malloc(sizeof(float) * heads * L);
  CHECK(cudaMemcpy(h_buf, d_o, n * 2, cudaMemcpyDeviceToHost));
  CHECK(cudaMemcpy(lse, d_lse, sizeof(float) * heads * L, cudaMemcpyDeviceToHost));
  for (int hd = 0; hd < heads; ++hd)
    for (int i = 0; i < L; ++i) {
      const int t = i / (H * W);
      const int nblk = hd == 0 ? (T - t < 3 ? T - t : 3) : (t < T - 1 ? 1 : 0);
      const int keys = 256 * nblk;
      const float l = lse[hd * L + i];
      for (int c = 0; c < D; ++c) {
        const uint16_t o = h_buf[((size_t)hd * L + i) * D + c];
        if (o != (keys ? 0x3F80 : 0)) { fprintf(stderr, "out[%d][%d][%d] = 0x%04x\n", hd, i, c, o); return 1; }
      }
      if (keys ? fabsf(l - logf((float)keys)) > 1e-3f : !(isinf(l) && l < 0)) { fprintf(stderr, "lse[%d][%d] = %f\n", hd, i, l); return 1; }
    }
  {
    /* joint sequence: 77 text tokens after the L video tokens of each head; q = 0, v = 0 on video and
     * 1 on text tokens: out = n_text / (attended video keys + n_text), lse = ln(that denominator) */
    const int NT = 77, LT = L + NT;
    const size_t nj = (size_t)heads * LT * D;
    uint16_t* hj = (uint16_t*)malloc(nj * 2);
    float* lj = (float*)malloc(sizeof(float) * heads * LT);
    uint16_t *jq, *jk, *jv, *jo; float* jl;
    CHECK(cudaMalloc((void**)&jq, nj * 2)); CHECK(cudaMalloc((void**)&jk, nj * 2));
    CHECK(cudaMalloc((void**)&jv, nj * 2)); CHECK(cudaMalloc((void**)&jo, nj * 2));
    CHECK(cudaMalloc((void**)&jl, sizeof(float) * heads * LT));
    CHECK(cudaMemset(jq, 0, nj * 2));
    CHECK(cudaMemset(jk, 0, nj * 2));
    for (int hd = 0; hd < heads; ++hd)
      for (int i = 0; i < LT; ++i)
        for (int c = 0; c < D; ++c) hj[((size_t)hd * LT + i) * D + c] = i < L ? 0 : 0x3F80;
    CHECK(cudaMemcpy(jv, hj, nj * 2, cudaMemcpyHostToDevice));
    psa_problem pj = prob;
    pj.stride_head = (int64_t)LT * D;
    CHECK(psa_attn_fwd_joint(jq, jk, jv, jo, jl, hp, &pj, NT, T, H, W, NULL));
    CHECK(psa_last_device_status(&detail));
    CHECK(cudaMemcpy(hj, jo, nj * 2, cudaMemcpyDeviceToHost));
    CHECK(cudaMemcpy(lj, jl, sizeof(float) * heads * LT, cudaMemcpyDeviceToHost));
    for (int hd = 0; hd < heads; ++hd)
      for (int i = 0; i < LT; ++i) {
        int keys = L;                       /* a text query attends every video key */
        if (i < L) {
          const int t = i / (H * W);
          keys = 256 * (hd == 0 ? (T - t < 3 ? T - t : 3) : (t < T - 1 ? 1 : 0));
        }
        const float want = (float)NT / (float)(keys + NT);
        uint32_t bits = (uint32_t)hj[((size_t)hd * LT + i) * D + (i % D)] << 16;
        float got;
        memcpy(&got, &bits, 4);
        if (fabsf(got - want) > 0.01f * want) { fprintf(stderr, "joint out[%d][%d] = %f, want %f\n", hd, i, got, want); return 1; }
        if (fabsf(lj[hd * LT + i] - logf((float)(keys + NT))) > 1e-3f) { fprintf(stderr, "joint lse[%d][%d] = %f\n", hd, i, lj[hd * LT + i]); return 1; }
      }
  }
  {
    /* search: candidate 0 covers everything (loss exactly 0), candidate 1 is head 0's mask (loss > 0 for
     * arbitrary inputs); selection on hand-worked numbers */
    const psa_head_params cand[2] = {{4, 0, 0, 1, 0, 0}, {2, 1, 0, 1, 0, 0}};
    const int64_t sb = psa_search_scratch_bytes(2, T, H, W);
    if (sb <= 0) { fprintf(stderr, "scratch bytes %lld\n", (long long)sb); return 1; }
    void* scratch; float* d_loss; float loss[2];
    CHECK(cudaMalloc(&scratch, (size_t)sb)); CHECK(cudaMalloc((void**)&d_loss, 8));
    CHECK(cudaMemcpy(d_q, d_k, (size_t)L * D * 2, cudaMemcpyDeviceToDevice));   /* q = k: arbitrary, peaked rows */
    psa_problem ps = prob;
    ps.n_heads = 1;
    CHECK(psa_search_losses(d_q, d_k, d_k, cand, 2, &ps, T, H, W, scratch, d_loss, NULL));
    CHECK(psa_last_device_status(&detail));
    CHECK(cudaMemcpy(loss, d_loss, 8, cudaMemcpyDeviceToHost));
    if (loss[0] != 0.0f || !(loss[1] > 0.0f)) { fprintf(stderr, "losses %g %g\n", loss[0], loss[1]); return 1; }
    const float ls[4] = {0.020f, 0.001f, 0.008f, 0.004f}, sp[4] = {0.90f, 0.10f, 0.75f, 0.50f};
    if (psa_search_select(ls, sp, 4, 0.0005f) != 1 || psa_search_select(ls, sp, 4, 0.005f) != 3 ||
        psa_search_select(ls, sp, 4, 0.01f) != 2 || psa_search_select(ls, sp, 4, 0.05f) != 0 ||
        psa_search_select_at_sparsity(ls, sp, 4, 0.5f) != 3 || psa_search_select_at_sparsity(ls, sp, 4, 0.95f) != PSA_ERR_CAPACITY) {
      fprintf(stderr, "selection mismatch\n");
      return 1;
    }
  }
  CHECK(psa_shutdown());
  printf("OK %lld kernel launches\n", (long long)psa_launch_count());
  return 0;
}
