// psa_mask_build: block mask and GetKVBlocks index lists from the stripe parameters
// (Algorithm 1 evaluated on block coordinates; Algorithm 2, producer side).
// Integer work only, bound by the HBM writes of the mask bytes and the column ids.
#include "psa_common.cuh"

namespace psa {

// Row counts and their exclusive prefix sum.  The block mask of a head is the Kronecker
// product of its temporal and spatial axis masks, so the count of row (t', s') is
// cntT(t') * cntS(s').  One block; rows are scanned in chunks of blockDim.x.
__global__ void __launch_bounds__(1024)
mask_rowptr_kernel(const HeadParamsArray hp, const Geom g, int head0, int n_heads_here,
                   int* __restrict__ row_ptr, int row_base, int ptr_base) {
  extern __shared__ int sm[];  // [n_heads_here][Tp + Sp] axis row counts, then 1024 scan words
  const int per_head = g.Tp + g.Sp;
  int* cnt = sm;
  int* scan = sm + n_heads_here * per_head;
  for (int idx = threadIdx.x; idx < n_heads_here * per_head; idx += blockDim.x) {
    const int h = idx / per_head, a = idx % per_head;
    const psa_head_params p = hp.p[head0 + h];
    int c = 0;
    if (a < g.Tp) {
      for (int k = 0; k < g.Tp; ++k) c += axis_attends(k - a, p.Tw, p.To, p.Ts);
    } else {
      const int s = a - g.Tp;
      for (int k = 0; k < g.Sp; ++k) c += axis_attends(k - s, p.Sw, p.So, p.Ss);
    }
    cnt[idx] = c;
  }
  __syncthreads();
  const int rows = n_heads_here * g.NB;
  int carry = ptr_base;
  for (int base = 0; base < rows; base += blockDim.x) {
    const int r = base + threadIdx.x;
    int c = 0;
    if (r < rows) {
      const int h = r / g.NB, qb = r % g.NB;
      c = cnt[h * per_head + qb / g.Sp] * cnt[h * per_head + g.Tp + qb % g.Sp];
    }
    // inclusive scan over the block (Hillis-Steele in shared memory)
    scan[threadIdx.x] = c;
    __syncthreads();
    for (int off = 1; off < blockDim.x; off <<= 1) {
      int v = threadIdx.x >= off ? scan[threadIdx.x - off] : 0;
      __syncthreads();
      scan[threadIdx.x] += v;
      __syncthreads();
    }
    if (r < rows) row_ptr[row_base + r] = carry + scan[threadIdx.x] - c;
    const int total = scan[blockDim.x - 1];
    __syncthreads();
    carry += total;
  }
  if (threadIdx.x == 0) row_ptr[row_base + rows] = carry;
}

// Mask bytes and column lists.  Work units are interleaved over the grid:
//   units [0, n_chunks): 16 consecutive mask bytes each (flat over [head][qb][kb]);
//   units [n_chunks, n_chunks + rows): one warp-wide pass over a row's key blocks, writing
//   the attended ids in ascending order at row_ptr[row].
__global__ void __launch_bounds__(256)
mask_fill_kernel(const HeadParamsArray hp, const Geom g, int head0, int n_heads_here,
                 uint8_t* __restrict__ block_mask, const int* __restrict__ row_ptr,
                 int* __restrict__ col_idx, int row_base) {
  const long long nb2 = (long long)g.NB * g.NB;
  const long long total_bytes = nb2 * n_heads_here;
  const long long n_chunks = block_mask ? (total_bytes + 15) / 16 : 0;
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long nthreads = (long long)gridDim.x * blockDim.x;

  for (long long c = tid; c < n_chunks; c += nthreads) {
    const long long b0 = c * 16;
    int h = (int)(b0 / nb2);
    long long rem = b0 - (long long)h * nb2;
    int qb = (int)(rem / g.NB), kb = (int)(rem % g.NB);
    psa_head_params p = hp.p[head0 + h];
    int tq = qb / g.Sp, sq = qb % g.Sp;
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    const int n = (int)((total_bytes - b0) < 16 ? (total_bytes - b0) : 16);
    for (int i = 0; i < n; ++i) {
      const int tk = kb / g.Sp, sk = kb % g.Sp;
      const uint32_t bit = axis_attends(tk - tq, p.Tw, p.To, p.Ts) && axis_attends(sk - sq, p.Sw, p.So, p.Ss);
      w[i >> 2] |= bit << (8 * (i & 3));
      if (++kb == g.NB) {
        kb = 0;
        if (++qb == g.NB) {
          qb = 0;
          ++h;
          if (h < n_heads_here) p = hp.p[head0 + h];
        }
        tq = qb / g.Sp;
        sq = qb % g.Sp;
      }
    }
    uint8_t* dst = block_mask + (long long)head0 * nb2 + b0;
    if (n == 16) {
      *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
    } else {
      for (int i = 0; i < n; ++i) dst[i] = (uint8_t)(w[i >> 2] >> (8 * (i & 3)));
    }
  }

  if (col_idx == nullptr) return;
  const int lane = threadIdx.x & 31;
  const long long warp = tid >> 5, nwarps = nthreads >> 5;
  const int rows = n_heads_here * g.NB;
  for (long long r = warp; r < rows; r += nwarps) {
    const int h = (int)(r / g.NB), qb = (int)(r % g.NB);
    const psa_head_params p = hp.p[head0 + h];
    const int tq = qb / g.Sp, sq = qb % g.Sp;
    int pos = row_ptr[row_base + r];
    for (int base = 0; base < g.NB; base += 32) {
      const int kb = base + lane;
      bool att = false;
      if (kb < g.NB) {
        const int tk = kb / g.Sp, sk = kb % g.Sp;
        att = axis_attends(tk - tq, p.Tw, p.To, p.Ts) && axis_attends(sk - sq, p.Sw, p.So, p.Ss);
      }
      const unsigned m = __ballot_sync(0xffffffffu, att);
      if (att) col_idx[pos + __popc(m & ((1u << lane) - 1u))] = kb;
      pos += __popc(m);
    }
  }
}

cudaError_t launch_mask_build(const HeadParamsArray& hp, const Geom& g, int head0, int n_heads_here,
                              uint8_t* block_mask, int* row_ptr, int* col_idx, int ptr_base,
                              int n_sms, cudaStream_t stream, int* launches) {
  const int row_base = head0 * g.NB;
  if (row_ptr) {
    const size_t smem = sizeof(int) * ((size_t)n_heads_here * (g.Tp + g.Sp) + 1024);
    if (smem > 48 * 1024) {
      cudaError_t e = cudaFuncSetAttribute(mask_rowptr_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    mask_rowptr_kernel<<<1, 1024, smem, stream>>>(hp, g, head0, n_heads_here, row_ptr, row_base, ptr_base);
    ++*launches;
  }
  if (block_mask || col_idx) {
    mask_fill_kernel<<<n_sms * 8, 256, 0, stream>>>(hp, g, head0, n_heads_here, block_mask, row_ptr, col_idx, row_base);
    ++*launches;
  }
  return cudaGetLastError();
}

}  // namespace psa
