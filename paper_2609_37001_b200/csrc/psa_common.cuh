// Shared host/device definitions of the PSA library (not part of the public ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "psa.h"

namespace psa {

constexpr int kHeadDim = 128;     // head dimension the attention kernel is built for
constexpr int kSlabTokens = 128;  // tokens per compute slab (one MMA tile of rows / keys)
constexpr int kMaxHeads = 128;    // heads per launch (parameters travel by value)
constexpr int kMaxTp = 256;       // limits of the in-kernel key-block bitmasks
constexpr int kMaxSp = 2048;

// Problem geometry handed to every kernel by value.
struct Geom {
  int T, H, W;             // real token grid
  int bt, bh, bw;          // mask block (PSABlock) extents in tokens
  int Tp, Hp, Wp, Sp, NB;  // block grid after 3D-padding; Sp = Hp*Wp, NB = Tp*Sp
  int ct, ch, cw;          // 128-token slab = one TMA box (ct*ch*cw == 128)
  int n_sub;               // slabs per mask block (1..3)
  int sub_axis;            // axis along which the slabs of a block stack: 0 = t, 1 = h, 2 = w
  int c_last;              // extent of a block's LAST slab along sub_axis (<= the full slab's)
  int n_last;              // tokens of that last slab: 128, 112, 96 or 64
  int n_heads;
  int items_per_block;     // work items per query block = ceil(n_sub / 2)
  float scale_log2;        // softmax scale times log2(e)
  long long L;             // T*H*W
  // joint video + text sequences: n_text text tokens follow the L video tokens of every head
  int n_text;              // 0: video only
  int n_ts;                // text slabs of 128 tokens = ceil(n_text / 128)
  int n_titems;            // work items of the text queries per head = ceil(n_ts / 2)
  int items_per_head;      // NB * items_per_block + n_titems
  long long Lt;            // L + n_text: tokens per head, row length of lse
};

struct HeadParamsArray {
  psa_head_params p[kMaxHeads];
};

// One unit of work of the attention kernel: up to two query slabs of one query block.
// x = head, y = query block id, z = number of attended key blocks,
// w = first slab index | (number of slabs << 16) | (split-KV mode << 24) | (text-query item << 25)
typedef int4 WorkItem;

// Layout of the per-device workspace (all int32 words).
constexpr int kWsStatus = 0;     // first device-side error (0 = none)
constexpr int kWsDetail = 1;     // diagnostic of that error
constexpr int kWsCounter = 2;    // dynamic scheduler ticket
constexpr int kWsHeaderWords = 16;

// One axis condition of the stripe mask (Algorithm 1): delta is key minus query
// coordinate in blocks; stride 0 encodes an infinite stride.
__host__ __device__ __forceinline__ bool axis_attends(int delta, int width, int offset, int stride) {
  int x = delta - offset;
  x = x < 0 ? -x : x;
  if (stride != 0) x = x % stride;
  return x <= width - 1;
}

}  // namespace psa
