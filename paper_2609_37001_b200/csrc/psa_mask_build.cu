// psa_mask_build: block mask and GetKVBlocks index lists from the stripe parameters
// (Algorithm 1 evaluated on block coordinates; Algorithm 2, producer side).
// Integer work only, bound by the HBM writes of the mask bytes and the column ids.
//
// The two conditions of Algorithm 1 depend only on coordinate differences, so each block of
// threads first tabulates, for its head, "does difference d attend" for every temporal and
// every spatial difference (one modulo per table entry instead of two per mask byte).  Row
// counts are window sums of those tables, and the block mask of a head is the Kronecker
// product of its two axis masks, so the count of row (t', s') is cntT(t') * cntS(s') and
// its offset in the column list has a closed form.
#include "psa_common.cuh"

namespace psa {

struct HeadBases {
  int base[kMaxHeads];  // number of attended block pairs of all earlier heads
};

// Shared-memory tables of one head.  attT[d + Tp-1], attS[d + Sp-1] for differences d;
// cntT[t], cntS[s] row counts per axis; preT[t], preS[s] their exclusive prefix sums.
struct Tables {
  uint8_t* attT;
  uint8_t* attS;
  int* cntT;
  int* cntS;
  int* preT;
  int* preS;
};

__host__ __device__ inline size_t tables_bytes(const Geom& g) {
  const size_t bytes = (size_t)(2 * g.Tp - 1) + (size_t)(2 * g.Sp - 1);
  return ((bytes + 15) & ~size_t(15)) + sizeof(int) * 2 * (size_t)(g.Tp + g.Sp);
}

__device__ __forceinline__ Tables carve_tables(uint8_t* smem, const Geom& g) {
  Tables t;
  t.attT = smem;
  t.attS = smem + (2 * g.Tp - 1);
  const size_t bytes = (size_t)(2 * g.Tp - 1) + (size_t)(2 * g.Sp - 1);
  int* ints = reinterpret_cast<int*>(smem + ((bytes + 15) & ~size_t(15)));
  t.cntT = ints;
  t.cntS = ints + g.Tp;
  t.preT = t.cntS + g.Sp;
  t.preS = t.preT + g.Tp;
  return t;
}

// Builds the tables of one head cooperatively (whole block), ends with a barrier.
__device__ void build_tables(const Tables& t, const psa_head_params& p, const Geom& g) {
  for (int i = threadIdx.x; i < 2 * g.Tp - 1; i += blockDim.x) t.attT[i] = axis_attends(i - (g.Tp - 1), p.Tw, p.To, p.Ts);
  for (int i = threadIdx.x; i < 2 * g.Sp - 1; i += blockDim.x) t.attS[i] = axis_attends(i - (g.Sp - 1), p.Sw, p.So, p.Ss);
  __syncthreads();
  // cnt[x] = number of key coordinates k in [0, n) with att[k - x + n-1]: a window of n entries
  for (int x = threadIdx.x; x < g.Tp; x += blockDim.x) {
    int c = 0;
    for (int k = 0; k < g.Tp; ++k) c += t.attT[k - x + g.Tp - 1];
    t.cntT[x] = c;
  }
  // the spatial axis can be long: one warp per 32 coordinates, lanes stride over the window
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  for (int x = warp; x < g.Sp; x += nwarps) {
    int c = 0;
    for (int k = lane; k < g.Sp; k += 32) c += t.attS[k - x + g.Sp - 1];
    for (int off = 16; off > 0; off >>= 1) c += __shfl_xor_sync(0xffffffffu, c, off);
    if (lane == 0) t.cntS[x] = c;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int acc = 0;
    for (int x = 0; x < g.Tp; ++x) { t.preT[x] = acc; acc += t.cntT[x]; }
  }
  if (threadIdx.x == 32 || (blockDim.x <= 32 && threadIdx.x == 0)) {
    int acc = 0;
    for (int x = 0; x < g.Sp; ++x) { t.preS[x] = acc; acc += t.cntS[x]; }
  }
  __syncthreads();
}

// Offset of row (tq, sq) inside its head's column list, and its length.
__device__ __forceinline__ void row_extent(const Tables& t, const Geom& g, int tq, int sq, int& offset, int& count) {
  const int sumS = t.preS[g.Sp - 1] + t.cntS[g.Sp - 1];
  offset = t.preT[tq] * sumS + t.cntT[tq] * t.preS[sq];
  count = t.cntT[tq] * t.cntS[sq];
}

// One block per (group of query blocks, head); one warp per query block (= one CSR row and
// one row of the byte mask).  Lanes cover 32 consecutive key blocks per step: coalesced mask
// bytes, ballot-compacted ascending column ids.
__global__ void __launch_bounds__(256)
mask_build_kernel(const HeadParamsArray hp, const HeadBases hb, const Geom g, int n_heads_here, int rows_per_block,
                  uint8_t* __restrict__ block_mask, int* __restrict__ row_ptr, int* __restrict__ col_idx,
                  int total_nnz) {
  extern __shared__ __align__(16) uint8_t smem_tab[];
  const int h = blockIdx.y;
  const Tables t = carve_tables(smem_tab, g);
  build_tables(t, hp.p[h], g);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const int q0 = blockIdx.x * rows_per_block;
  const int q1 = min(g.NB, q0 + rows_per_block);
  const long long nb2 = (long long)g.NB * g.NB;
  for (int qb = q0 + warp; qb < q1; qb += nwarps) {
    const int tq = qb / g.Sp, sq = qb % g.Sp;
    int offset, count;
    row_extent(t, g, tq, sq, offset, count);
    int pos = hb.base[h] + offset;
    if (row_ptr && lane == 0) row_ptr[(long long)h * g.NB + qb] = pos;
    uint8_t* mrow = block_mask ? block_mask + (long long)h * nb2 + (long long)qb * g.NB : nullptr;
    if (mrow == nullptr && col_idx == nullptr) continue;
    const uint8_t* aT = t.attT + (g.Tp - 1 - tq);
    const uint8_t* aS = t.attS + (g.Sp - 1 - sq);
    int tk = lane / g.Sp, sk = lane % g.Sp;       // coordinates of key block `lane`
    const int dt = 32 / g.Sp, ds = 32 % g.Sp;     // advance of 32 key blocks
    for (int base = 0; base < g.NB; base += 32) {
      const int kb = base + lane;
      const bool att = kb < g.NB && aT[tk] && aS[sk];
      if (mrow && kb < g.NB) mrow[kb] = att ? 1 : 0;
      if (col_idx) {
        const unsigned m = __ballot_sync(0xffffffffu, att);
        if (att) col_idx[pos + __popc(m & ((1u << lane) - 1u))] = kb;
        pos += __popc(m);
      }
      tk += dt;
      sk += ds;
      if (sk >= g.Sp) { sk -= g.Sp; ++tk; }
    }
  }
  if (row_ptr && blockIdx.x == 0 && h == n_heads_here - 1 && threadIdx.x == 0)
    row_ptr[(long long)n_heads_here * g.NB] = total_nnz;
}

cudaError_t launch_mask_build(const HeadParamsArray& hp, const int* head_bases, const Geom& g, int n_heads_here,
                              uint8_t* block_mask, int* row_ptr, int* col_idx, int total_nnz_through_chunk,
                              int n_sms, cudaStream_t stream, int* launches) {
  HeadBases hb;
  for (int h = 0; h < kMaxHeads; ++h) hb.base[h] = h < n_heads_here ? head_bases[h] : 0;
  const size_t smem = tables_bytes(g);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(mask_build_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  // enough blocks per head to fill every SM's thread slots (8 blocks of 256 threads each),
  // at least 8 rows (one per warp) per block
  int blocks_per_head = (8 * n_sms + n_heads_here - 1) / n_heads_here;
  if (blocks_per_head < 1) blocks_per_head = 1;
  int rows_per_block = (g.NB + blocks_per_head - 1) / blocks_per_head;
  if (rows_per_block < 8) rows_per_block = 8;
  blocks_per_head = (g.NB + rows_per_block - 1) / rows_per_block;
  dim3 grid(blocks_per_head, n_heads_here);
  mask_build_kernel<<<grid, 256, smem, stream>>>(hp, hb, g, n_heads_here, rows_per_block, block_mask, row_ptr, col_idx,
                                                 total_nnz_through_chunk);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace psa
