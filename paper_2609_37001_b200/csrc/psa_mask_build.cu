// psa_mask_build: block mask and GetKVBlocks index lists from the stripe parameters
// (Algorithm 1 evaluated on block coordinates; Algorithm 2, producer side).
// Integer work only.  Two kernels: one for block grids of at most 64 temporal x 32 spatial
// coordinates (mask_build_small_kernel, further down: one thread block per head and temporal
// query coordinate), and the general one described here.
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

// Fast path for block grids with at most 64 temporal and 32 spatial block coordinates (all the
// paper's shapes): no block-wide table building.  The host evaluates the two axis conditions of
// Algorithm 1 once per head for every coordinate difference and hands the kernel two bit sets
// per head (127 and 63 bits; bit d + n - 1 of an axis' set = "difference d attends"), so the key
// coordinates a query coordinate x attends are one shift away: (set >> (n - 1 - x)) & ((1 << n) - 1).
//
// One thread block per (head, temporal query coordinate tq): its S' rows are consecutive, so
// their mask bytes are one contiguous region and their column lists one contiguous range.
//   * Warp 0 derives the row counts (popcounts), their prefix sums (one warp scan), the block's
//     first list offset, "the r-th attended temporal coordinate" of tq, and writes the S' row
//     offsets.
//   * Meanwhile all threads write the mask region 32 bytes at a time: a thread assembles 32
//     consecutive mask bits (the row of the Kronecker product is the spatial bit pattern repeated
//     under the temporal bits), spreads them to bytes with four multiplies per 16 and stores two
//     16-byte words.
//   * After one barrier the rows of the block are taken by sub-groups of 8, 16 or 32 lanes: entry e
//     of a row's list is (the (e / cS)-th attended temporal coordinate, the (e % cS)-th attended
//     spatial one); the division is a multiply and a shift (e < 2048, cS <= 32).
struct HeadSets {
  unsigned long long setT[kMaxHeads], setT_hi[kMaxHeads], setS[kMaxHeads];   // temporal set: 127 bits
  int base[kMaxHeads];  // number of attended block pairs of all earlier heads
};

// Constants of the closed-form 32-bit mask window (see the kernel).  groups = temporal groups a
// window can touch; mul / keep spread `groups` consecutive temporal bits to a spacing of S' bits
// (bit i lands on i * S'; all partial products fall on distinct bits while groups <= S' - 1).
struct WindowConsts {
  unsigned long long mul, keep;
  int groups, enabled;
};

// n / d for n < 2^16, d <= 2^11 with m = ceil(2^40 / d): exact (n * (m * d - 2^40) < 2^40)
__device__ __forceinline__ int div_magic(int n, unsigned long long m) { return (int)(((unsigned long long)(unsigned)n * m) >> 40); }

// (Six resident blocks per SM -- 40 registers -- let the 840 blocks of the Wan 14B shape start in one wave.)
__global__ void __launch_bounds__(256, 6)
mask_build_small_kernel(const HeadSets hs, const Geom g, int n_heads_here, unsigned long long magic_nb,
                        unsigned long long magic_sp, const WindowConsts wc, uint8_t* __restrict__ block_mask, int* __restrict__ row_ptr,
                        int* __restrict__ col_idx, int total_nnz) {
  const int h = blockIdx.y, tq = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const int Tp = g.Tp, Sp = g.Sp, NB = g.NB;
  __shared__ int s_preS[32], s_cS[32], s_tsel[64], s_hdr[2];
  __shared__ int s_strip[8 * 4 * 32];      // per warp and sub-group: the r-th attended spatial coordinate of its row
  __shared__ unsigned s_inv[33];           // ceil(2^20 / c): e / c = (e * inv) >> 20 for e < 2048, c <= 32
  const unsigned long long setT = hs.setT[h], setT_hi = hs.setT_hi[h], setS = hs.setS[h];
  const unsigned long long maskT = Tp == 64 ? ~0ull : ((1ull << Tp) - 1ull);
  const unsigned maskS = Sp == 32 ? 0xffffffffu : ((1u << Sp) - 1u);
  // temporal key coordinates attended by query coordinate x (up to 64 of them: a 64-bit mask)
  auto rowT = [&](int x) -> unsigned long long {
    const int sh = Tp - 1 - x;   // 0 .. 63
    const unsigned long long lo = setT >> sh, hi = sh ? (setT_hi << (64 - sh)) : 0ull;
    return (lo | hi) & maskT;
  };
  auto rowS = [&](int x) -> unsigned { return (unsigned)(setS >> (Sp - 1 - x)) & maskS; };
  const unsigned long long mT = rowT(tq);
  const unsigned lane_lt = (1u << lane) - 1u;

  if (threadIdx.x >= 64 && threadIdx.x <= 96) {
    const unsigned c = threadIdx.x - 64;
    s_inv[c] = c ? ((1u << 20) + c - 1u) / c : 0u;
  }
  if (warp == 0) {
    // lane x holds the counts of coordinates x (and x + 32 on the temporal axis) and the exclusive
    // prefixes of the counts before them
    const int cntT0 = lane < Tp ? __popcll(rowT(lane)) : 0, cntT1 = lane + 32 < Tp ? __popcll(rowT(lane + 32)) : 0;
    const int cntS = lane < Sp ? __popc(rowS(lane)) : 0;
    int incT0 = cntT0, incT1 = cntT1, incS = cntS;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int a = __shfl_up_sync(0xffffffffu, incT0, off), c = __shfl_up_sync(0xffffffffu, incT1, off);
      const int b = __shfl_up_sync(0xffffffffu, incS, off);
      if (lane >= off) { incT0 += a; incT1 += c; incS += b; }
    }
    const int sumT0 = __shfl_sync(0xffffffffu, incT0, 31);
    const int preT0 = incT0 - cntT0, preT1 = sumT0 + incT1 - cntT1, preS = incS - cntS;
    const int sumS = __shfl_sync(0xffffffffu, incS, 31);
    const int cT = __popcll(mT);
    const int pT = __shfl_sync(0xffffffffu, tq < 32 ? preT0 : preT1, tq & 31);
    const int pos0 = hs.base[h] + pT * sumS;
    s_preS[lane] = preS;
    s_cS[lane] = cntS;
    if ((mT >> lane) & 1ull) s_tsel[__popcll(mT & (unsigned long long)lane_lt)] = lane;
    if ((mT >> (lane + 32)) & 1ull) s_tsel[__popcll(mT & ((1ull << (lane + 32)) - 1ull))] = lane + 32;
    if (lane == 0) { s_hdr[0] = cT; s_hdr[1] = pos0; }
    if (row_ptr) {
      if (lane < Sp) row_ptr[(long long)h * NB + tq * Sp + lane] = pos0 + cT * preS;
      if (tq == 0 && h == n_heads_here - 1 && lane == 0) row_ptr[(long long)n_heads_here * NB] = total_nnz;
    }
  }

  if (block_mask) {
    // The block writes the 32-byte aligned chunks that START inside its rows' region; its last chunk
    // runs on into the next region (next tq, or the next head), whose own first chunk starts at the
    // next aligned address.  Only the very first bytes of the whole mask (when its base is not
    // aligned) and a clipped chunk at its very end are written bytewise.
    const int len = Sp * NB;                                 // bytes of this block's rows
    uint8_t* p0 = block_mask + ((long long)h * NB + (long long)tq * Sp) * NB;
    const int lead = (int)((32u - (unsigned)(reinterpret_cast<uintptr_t>(p0) & 31u)) & 31u);   // first aligned offset
    // up to `limit` mask bytes from region offset r on (bit i of the result = byte r + i); *got = bytes that exist
    auto gen = [&](int r, int limit, int* got) -> unsigned {
      int hh = h, tq_ = tq;
      int sq = div_magic(r, magic_nb), kb = r - sq * NB;
      int tk = div_magic(kb, magic_sp), sk = kb - tk * Sp;
      unsigned long long sT = setT, sT_hi = setT_hi, sS = setS, mT_ = mT;
      unsigned mS = (unsigned)(sS >> (Sp - 1 - sq)) & maskS;
      unsigned bits = 0u;
      int n = 0;
      while (n < limit && hh < n_heads_here) {
        const unsigned grp = ((mT_ >> tk) & 1ull) ? (mS >> sk) : 0u;   // Sp - sk key blocks of temporal group tk
        int take = Sp - sk;
        if (take > limit - n) take = limit - n;
        bits |= (take >= 32 ? grp : (grp & ((1u << take) - 1u))) << n;
        n += take;
        sk += take;
        if (sk == Sp) {
          sk = 0;
          if (++tk == Tp) {
            tk = 0;
            if (++sq == Sp) {   // rare: the chunk runs on into the next region
              sq = 0;
              if (++tq_ == Tp) {
                tq_ = 0;
                if (++hh < n_heads_here) { sT = hs.setT[hh]; sT_hi = hs.setT_hi[hh]; sS = hs.setS[hh]; }
              }
              const int sh = Tp - 1 - tq_;
              mT_ = ((sT >> sh) | (sh ? (sT_hi << (64 - sh)) : 0ull)) & maskT;
            }
            mS = (unsigned)(sS >> (Sp - 1 - sq)) & maskS;
          }
        }
      }
      *got = n;
      return bits;
    };
    const int nchunks = len > lead ? (len - lead + 31) >> 5 : 0;
    // Closed form of a window that stays inside the block's rows: the temporal bits tk, tk + 1, ...
    // are spread to a spacing of S' bits by one multiplication, widened to runs of S' ones
    // ((x << S') - x), and combined with the spatial pattern repeated with period S'; the window
    // starts sk bits in.  A window that leaves the block's rows takes the general loop above.
    auto periodic = [&](unsigned m) -> unsigned long long {
      unsigned long long r = m;
      for (int wd = Sp; wd < 64; wd <<= 1) r |= r << wd;
      return r;
    };
    auto runs = [&](int tk) -> unsigned long long {
      const unsigned long long tw = (mT >> tk) & ((1ull << wc.groups) - 1ull);
      const unsigned long long spread = (tw * wc.mul) & wc.keep;
      return (spread << Sp) - spread;
    };
    const unsigned long long runs0 = runs(0);
    for (int c = threadIdx.x; c < nchunks; c += blockDim.x) {
      const int r = lead + 32 * c;
      int n = 32;
      unsigned bits;
      const int sq = div_magic(r, magic_nb), kb = r - sq * NB;
      if (wc.enabled && (kb + 32 <= NB || sq + 1 < Sp)) {
        const int tk = div_magic(kb, magic_sp), sk = kb - tk * Sp;
        bits = (unsigned)((runs(tk) & periodic(rowS(sq))) >> sk);
        if (kb + 32 > NB) bits |= (unsigned)(runs0 & periodic(rowS(sq + 1))) << (NB - kb);   // on into the next row
      } else {
        bits = gen(r, 32, &n);
      }
      if (n == 32) {
        uint32_t w[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) w[k] = (((bits >> (4 * k)) & 15u) * 0x00204081u) & 0x01010101u;
        uint4* dst = reinterpret_cast<uint4*>(p0 + r);
        dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
        dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
      } else {
        for (int i = 0; i < n; ++i) p0[r + i] = (uint8_t)((bits >> i) & 1u);   // the end of the whole mask
      }
    }
    if (h == 0 && tq == 0 && lead > 0 && threadIdx.x == blockDim.x - 1) {   // unaligned start of the whole mask
      int n;
      const unsigned bits = gen(0, lead, &n);
      for (int i = 0; i < n; ++i) p0[i] = (uint8_t)((bits >> i) & 1u);
    }
  }
  __syncthreads();

  if (col_idx) {
    // Sub-groups of 8, 16 or 32 lanes take one row each, so that the S' rows of the block are
    // all in flight at once (S' <= 8, 16, 32 with eight warps).
    const int cT = s_hdr[0], pos0 = s_hdr[1];
    const int lg = Sp > 16 ? 2 : (Sp > 8 ? 1 : 0);          // log2 of the sub-groups per warp
    const int W = 32 >> lg, grp = lane >> (5 - lg), sl = lane & (W - 1);
    int* strip = s_strip + ((warp << 2) + grp) * 32;         // the r-th attended spatial coordinate of the row
    for (int sq0 = warp << lg; sq0 < Sp && cT > 0; sq0 += nwarps << lg) {
      const int sq = sq0 + grp;
      const bool act = sq < Sp;
      const int cS = act ? s_cS[sq] : 0;
      const int pos = pos0 + cT * (act ? s_preS[sq] : 0);
      const unsigned mS = act ? rowS(sq) : 0u;
      for (int b = sl; b < 32; b += W)
        if ((mS >> b) & 1u) strip[__popc(mS & ((1u << b) - 1u))] = b;
      __syncwarp();
      const int count = cT * cS;
      const unsigned inv = s_inv[cS];
      for (int e = sl; e < count; e += W) {
        const int it = (int)(((unsigned)e * inv) >> 20), is = e - it * cS;
        col_idx[pos + e] = s_tsel[it] * Sp + strip[is];
      }
      __syncwarp();
    }
  }
}

cudaError_t launch_mask_build(const HeadParamsArray& hp, const int* head_bases, const Geom& g, int n_heads_here,
                              uint8_t* block_mask, int* row_ptr, int* col_idx, int total_nnz_through_chunk,
                              int n_sms, cudaStream_t stream, int* launches) {
  HeadBases hb;
  for (int h = 0; h < kMaxHeads; ++h) hb.base[h] = h < n_heads_here ? head_bases[h] : 0;
  if (g.Tp <= 64 && g.Sp <= 32) {
    HeadSets hs;
    for (int h = 0; h < kMaxHeads; ++h) {
      unsigned long long st = 0, st_hi = 0, ss = 0;
      if (h < n_heads_here) {
        const psa_head_params& p = hp.p[h];
        for (int i = 0; i < 2 * g.Tp - 1; ++i)
          if (axis_attends(i - (g.Tp - 1), p.Tw, p.To, p.Ts)) (i < 64 ? st : st_hi) |= 1ull << (i & 63);
        for (int i = 0; i < 2 * g.Sp - 1; ++i)
          if (axis_attends(i - (g.Sp - 1), p.Sw, p.So, p.Ss)) ss |= 1ull << i;
      }
      hs.setT[h] = st;
      hs.setT_hi[h] = st_hi;
      hs.setS[h] = ss;
      hs.base[h] = h < n_heads_here ? head_bases[h] : 0;
    }
    const unsigned long long two40 = 1ull << 40;
    const unsigned long long magic_nb = (two40 + (unsigned long long)g.NB - 1ull) / (unsigned long long)g.NB;
    const unsigned long long magic_sp = (two40 + (unsigned long long)g.Sp - 1ull) / (unsigned long long)g.Sp;
    // the closed-form window needs its partial products on distinct bits and at most one row end per window
    WindowConsts wc;
    wc.groups = (g.Sp - 1 + 31) / g.Sp + 1;
    wc.enabled = (wc.groups <= g.Sp - 1 && g.NB >= 32) ? 1 : 0;
    wc.mul = 0;
    wc.keep = 0;
    if (wc.enabled)
      for (int i = 0; i < wc.groups; ++i) {
        wc.mul |= 1ull << (i * (g.Sp - 1));
        if (i * g.Sp < 64) wc.keep |= 1ull << (i * g.Sp);
      }
    dim3 grid(g.Tp, n_heads_here);   // one block per (head, temporal query coordinate)
    mask_build_small_kernel<<<grid, 256, 0, stream>>>(
        hs, g, n_heads_here, magic_nb, magic_sp, wc, block_mask, row_ptr, col_idx, total_nnz_through_chunk);
    ++*launches;
    return cudaGetLastError();
  }
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
