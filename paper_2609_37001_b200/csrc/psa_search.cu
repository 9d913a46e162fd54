// PSA-Search for one head (Algorithm 3): loss of every candidate mask against full attention.
// The attention outputs come from the stripe attention kernel (all candidates in one launch, reading
// the same q, k, v); this file holds the reduction  loss[c] = mean((out_c - out_full)^2),
// which is bound by reading the candidate outputs from HBM once (the reference stays in L2).
#include <cuda_bf16.h>

#include "psa_common.cuh"

namespace psa {

constexpr int kLossSlices = 64;    // blocks per candidate
constexpr int kLossThreads = 256;

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// partial[c][slice] = sum over the slice's elements of (out_c - ref)^2, accumulated in double across
// threads in a fixed order (deterministic).
__global__ void __launch_bounds__(kLossThreads)
search_loss_partial_kernel(const uint4* __restrict__ outs, const uint4* __restrict__ ref, long long vec_per_cand,
                           double* __restrict__ partial) {
  const int c = blockIdx.y, slice = blockIdx.x;
  const uint4* oc = outs + (long long)c * vec_per_cand;
  const long long per = (vec_per_cand + kLossSlices - 1) / kLossSlices;
  const long long lo = (long long)slice * per;
  const long long hi = lo + per < vec_per_cand ? lo + per : vec_per_cand;
  float acc = 0.f;
  for (long long i = lo + threadIdx.x; i < hi; i += kLossThreads) {
    const uint4 a = oc[i], b = ref[i];
    const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float d0 = bf16_lo(aw[j]) - bf16_lo(bw[j]), d1 = bf16_hi(aw[j]) - bf16_hi(bw[j]);
      acc = fmaf(d0, d0, acc);
      acc = fmaf(d1, d1, acc);
    }
  }
  __shared__ double red[kLossThreads];
  red[threadIdx.x] = (double)acc;
  __syncthreads();
  for (int off = kLossThreads / 2; off > 0; off >>= 1) {
    if (threadIdx.x < off) red[threadIdx.x] += red[threadIdx.x + off];
    __syncthreads();
  }
  if (threadIdx.x == 0) partial[(long long)c * kLossSlices + slice] = red[0];
}

__global__ void search_loss_final_kernel(const double* __restrict__ partial, int n_cand, double inv_count,
                                         float* __restrict__ losses) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= n_cand) return;
  double s = 0.0;
  for (int i = 0; i < kLossSlices; ++i) s += partial[(long long)c * kLossSlices + i];
  losses[c] = (float)(s * inv_count);
}

size_t search_partial_bytes(int n_cand) { return sizeof(double) * (size_t)n_cand * kLossSlices; }

cudaError_t launch_search_losses(const void* outs, const void* ref, long long elems_per_cand, int n_cand, double* partial,
                                 float* losses, cudaStream_t stream, int* launches) {
  const long long vec = elems_per_cand / 8;  // 8 bf16 per 16-byte vector; L * 128 is always a multiple
  dim3 grid(kLossSlices, n_cand);
  search_loss_partial_kernel<<<grid, kLossThreads, 0, stream>>>(static_cast<const uint4*>(outs), static_cast<const uint4*>(ref),
                                                               vec, partial);
  search_loss_final_kernel<<<(n_cand + 127) / 128, 128, 0, stream>>>(partial, n_cand, 1.0 / (double)elems_per_cand, losses);
  *launches += 2;
  return cudaGetLastError();
}

}  // namespace psa
