// Host side of the PSA library: argument validation, geometry, per-device workspace,
// TMA descriptors and the extern "C" entry points declared in psa.h.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

#include "psa_common.cuh"

namespace psa {
cudaError_t launch_mask_build(const HeadParamsArray& hp, const int* head_bases, const Geom& g, int n_heads_here,
                              uint8_t* block_mask, int* row_ptr, int* col_idx, int total_nnz_through_chunk,
                              int n_sms, cudaStream_t stream, int* launches);
cudaError_t launch_plan(const HeadParamsArray& hp, const Geom& g, int head0, int n_heads_here, bool clear_status,
                        int* ws_header, psa_head_params* hp_dev, WorkItem* items, cudaStream_t stream);
struct TensorMaps {
  CUtensorMap q[3], k[3], v[3], o[3];  // [0]: full 128-token slab box, [1]: a block's last slab, [2]: text slab
};
cudaError_t launch_attn(const TensorMaps& tm, const Geom& g, const WorkItem* items, const psa_head_params* hp_dev,
                        int* ws_header, float* lse, int n_items, int n_sms, bool shared_qkv, cudaStream_t stream);
size_t search_partial_bytes(int n_cand);
cudaError_t launch_search_losses(const void* outs, const void* ref, long long elems_per_cand, int n_cand, double* partial,
                                 float* losses, cudaStream_t stream, int* launches);
cudaError_t launch_wait_probe(int* ws_header, unsigned long long limit_ns, cudaStream_t stream);
}  // namespace psa

namespace {

using namespace psa;

std::atomic<long long> g_launches{0};
std::mutex g_mu;

constexpr int kMaxDevices = 64;
struct Workspace {
  void* base = nullptr;
  size_t bytes = 0;
  int n_sms = 0;
  int cc_major = 0;
};
Workspace g_ws[kMaxDevices];

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
cudaEvent_t g_ev_start = nullptr, g_ev_stop = nullptr;

int load_driver_entry() {
  if (g_encode) return PSA_OK;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || fn == nullptr) {
    return PSA_ERR_CUDA;
  }
  g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  return PSA_OK;
}

bool valid_params(const psa_head_params& p) {
  const int lim = 1 << 30;
  return p.Tw >= 1 && p.Sw >= 1 && p.Ts >= 0 && p.Ss >= 0 && p.To > -lim && p.To < lim && p.So > -lim && p.So < lim;
}

// Chunks of a host-tensor call: 20 from a measured sweep at the 75,600-token, 40-head shape
// (4: 54.3 ms, 8: 50.3, 10: 48.9, 20: 47.6, 40: 49.7); PSA_HOST_CHUNKS overrides it for measurements.
int host_chunks() {
  static int v = 0;
  if (v == 0) {
    const char* e = std::getenv("PSA_HOST_CHUNKS");
    const int n = e ? std::atoi(e) : 0;
    v = n >= 1 ? n : 20;
  }
  return v;
}

// Geometry of the block grid; `for_attn` additionally derives the 128-token slab.
int make_geom(const psa_problem* prob, int T, int H, int W, bool for_attn, Geom* g) {
  if (!prob || T < 1 || H < 1 || W < 1 || prob->n_heads < 1) return PSA_ERR_INVALID_ARG;
  const psa_tile t = prob->tile;
  if (t.bt < 1 || t.bh < 1 || t.bw < 1) return PSA_ERR_INVALID_ARG;
  const long long L = (long long)T * H * W;
  if (L >= (1ll << 31)) return PSA_ERR_INVALID_ARG;
  std::memset(g, 0, sizeof(*g));
  g->T = T; g->H = H; g->W = W;
  g->bt = t.bt; g->bh = t.bh; g->bw = t.bw;
  g->Tp = (T + t.bt - 1) / t.bt;
  g->Hp = (H + t.bh - 1) / t.bh;
  g->Wp = (W + t.bw - 1) / t.bw;
  g->Sp = g->Hp * g->Wp;
  const long long nb = (long long)g->Tp * g->Sp;
  if (nb > (1 << 20)) return PSA_ERR_UNSUPPORTED;
  g->NB = (int)nb;
  g->n_heads = prob->n_heads;
  g->L = L;
  g->ct = t.bt; g->ch = t.bh; g->cw = t.bw;
  g->n_sub = 1;
  g->sub_axis = 0;
  g->items_per_block = 1;
  if (for_attn) {
    g->c_last = 1;
    g->n_last = kSlabTokens;
    if (prob->head_dim != kHeadDim) return PSA_ERR_UNSUPPORTED;
    if (!(prob->scale > 0.f) || !std::isfinite(prob->scale)) return PSA_ERR_INVALID_ARG;
    // Split the block into slabs along its outermost axis of extent > 1: full slabs of 128
    // tokens, and a last slab that may be shorter (112, 96 or 64 tokens) so that blocks such
    // as 1x15x16 tile a 45-row grid without padding.
    const long long tokens = (long long)t.bt * t.bh * t.bw;
    if (tokens < 128 || tokens > 384) return PSA_ERR_UNSUPPORTED;
    int axis, extent;
    long long other;
    if (t.bt > 1 || (t.bh == 1 && t.bw == 1)) { axis = 0; extent = t.bt; other = (long long)t.bh * t.bw; }
    else if (t.bh > 1) { axis = 1; extent = t.bh; other = (long long)t.bt * t.bw; }
    else { axis = 2; extent = t.bw; other = (long long)t.bt * t.bh; }
    if (other > kSlabTokens || (kSlabTokens % other) != 0) return PSA_ERR_UNSUPPORTED;
    const int c0 = (int)(kSlabTokens / other);
    const int n_sub = (extent + c0 - 1) / c0;
    const int c_last = extent - (n_sub - 1) * c0;
    const int n_last = (int)(c_last * other);
    if (n_sub > 3 || !(n_last == 128 || n_last == 112 || n_last == 96 || n_last == 64)) return PSA_ERR_UNSUPPORTED;
    if (axis == 0) g->ct = c0; else if (axis == 1) g->ch = c0; else g->cw = c0;
    g->sub_axis = axis;
    g->c_last = c_last;
    g->n_last = n_last;
    if (g->ct > 128 || g->ch > 128 || g->cw > 128) return PSA_ERR_UNSUPPORTED;
    if (g->Tp > kMaxTp || g->Sp > kMaxSp) return PSA_ERR_UNSUPPORTED;
    g->n_sub = n_sub;
    g->items_per_block = (n_sub + 1) / 2;
    g->scale_log2 = prob->scale * 1.4426950408889634f;
  }
  g->items_per_head = g->NB * g->items_per_block;
  g->Lt = L;
  return PSA_OK;
}

// Adds n_text text tokens per head to an attention geometry.
int set_text(Geom* g, long long n_text) {
  if (n_text < 0 || g->L + n_text >= (1ll << 31)) return PSA_ERR_INVALID_ARG;
  g->n_text = (int)n_text;
  g->n_ts = (int)((n_text + kSlabTokens - 1) / kSlabTokens);
  if (g->n_ts > 0xffff) return PSA_ERR_UNSUPPORTED;
  g->n_titems = (g->n_ts + 1) / 2;
  g->items_per_head = g->NB * g->items_per_block + g->n_titems;
  g->Lt = g->L + n_text;
  return PSA_OK;
}

// Attended block pairs of one head: product of the two axis pair counts.
long long head_nnz(const psa_head_params& p, const Geom& g) {
  long long ct = 0, cs = 0;
  for (int d = -(g.Tp - 1); d <= g.Tp - 1; ++d)
    if (axis_attends(d, p.Tw, p.To, p.Ts)) ct += g.Tp - (d < 0 ? -d : d);
  for (int d = -(g.Sp - 1); d <= g.Sp - 1; ++d)
    if (axis_attends(d, p.Sw, p.So, p.Ss)) cs += g.Sp - (d < 0 ? -d : d);
  return ct * cs;
}

int device_info(int* dev, Workspace** ws) {
  if (cudaGetDevice(dev) != cudaSuccess) return PSA_ERR_CUDA;
  if (*dev < 0 || *dev >= kMaxDevices) return PSA_ERR_UNSUPPORTED;
  Workspace& w = g_ws[*dev];
  if (w.n_sms == 0) {
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, *dev) != cudaSuccess) return PSA_ERR_CUDA;
    w.n_sms = prop.multiProcessorCount;
    w.cc_major = prop.major;
  }
  *ws = &w;
  return PSA_OK;
}

int ensure_workspace(Workspace* w, size_t bytes) {
  if (w->bytes >= bytes) return PSA_OK;
  if (w->base) {
    if (cudaDeviceSynchronize() != cudaSuccess) return PSA_ERR_CUDA;
    cudaFree(w->base);
    w->base = nullptr;
    w->bytes = 0;
  }
  const size_t want = bytes + bytes / 4 + 4096;
  if (cudaMalloc(&w->base, want) != cudaSuccess) return PSA_ERR_CUDA;
  if (cudaMemset(w->base, 0, want) != cudaSuccess) return PSA_ERR_CUDA;
  w->bytes = want;
  return PSA_OK;
}

// `last`: box of a block's last (possibly shorter) slab instead of the full 128-token slab.
int encode_map(CUtensorMap* tm, const void* base, const Geom& g, long long stride_head, long long stride_token,
               int n_heads_here, bool last) {
  const cuuint64_t dims[5] = {(cuuint64_t)kHeadDim, (cuuint64_t)g.W, (cuuint64_t)g.H, (cuuint64_t)g.T,
                              (cuuint64_t)n_heads_here};
  const cuuint64_t st = (cuuint64_t)stride_token * 2;
  const cuuint64_t strides[4] = {st, st * g.W, st * g.W * g.H,
                                 n_heads_here > 1 ? (cuuint64_t)stride_head * 2 : st * g.W * g.H * g.T};
  cuuint32_t box[5] = {64, (cuuint32_t)g.cw, (cuuint32_t)g.ch, (cuuint32_t)g.ct, 1};
  if (last) box[3 - g.sub_axis] = (cuuint32_t)g.c_last;
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  const CUresult r = g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box,
                              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? PSA_OK : PSA_ERR_INVALID_ARG;
}

// Map of the text tokens of every head: a [heads][n_text][128] view starting L tokens into each head,
// box = 128 tokens x 64 columns (same shared-memory image as a full video slab).
int encode_text_map(CUtensorMap* tm, const void* base, const Geom& g, long long stride_head, long long stride_token,
                    int n_heads_here) {
  const cuuint64_t st = (cuuint64_t)stride_token * 2;
  const cuuint64_t dims[5] = {(cuuint64_t)kHeadDim, (cuuint64_t)g.n_text, 1, 1, (cuuint64_t)n_heads_here};
  const cuuint64_t strides[4] = {st, st * g.n_text, st * g.n_text,
                                 n_heads_here > 1 ? (cuuint64_t)stride_head * 2 : st * g.n_text};
  const cuuint32_t box[5] = {64, (cuuint32_t)kSlabTokens, 1, 1, 1};
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  const void* text0 = static_cast<const uint16_t*>(base) + g.L * stride_token;
  const CUresult r = g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(text0), dims, strides, box,
                              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? PSA_OK : PSA_ERR_INVALID_ARG;
}

// Strides (in elements) of the inputs and of the output of one attention launch.
struct Layout {
  long long in_head, in_token;    // q, k, v
  long long out_head, out_token;  // out
  bool shared_qkv;                // every head reads head 0 of q, k, v
};

// The four tensors, each with the full-slab box ([0]) and the last-slab box ([1]).
int encode_maps(TensorMaps* tm, const void* q, const void* k, const void* v, void* out, const Geom& g,
                const Layout& lay, int n_heads_here) {
  int rc;
  const int n_in = lay.shared_qkv ? 1 : n_heads_here;
  for (int last = 0; last < 2; ++last) {
    if ((rc = encode_map(&tm->q[last], q, g, lay.in_head, lay.in_token, n_in, last != 0)) != PSA_OK) return rc;
    if ((rc = encode_map(&tm->k[last], k, g, lay.in_head, lay.in_token, n_in, last != 0)) != PSA_OK) return rc;
    if ((rc = encode_map(&tm->v[last], v, g, lay.in_head, lay.in_token, n_in, last != 0)) != PSA_OK) return rc;
    if ((rc = encode_map(&tm->o[last], out, g, lay.out_head, lay.out_token, n_heads_here, last != 0)) != PSA_OK) return rc;
  }
  if (g.n_text > 0) {
    if ((rc = encode_text_map(&tm->q[2], q, g, lay.in_head, lay.in_token, n_in)) != PSA_OK) return rc;
    if ((rc = encode_text_map(&tm->k[2], k, g, lay.in_head, lay.in_token, n_in)) != PSA_OK) return rc;
    if ((rc = encode_text_map(&tm->v[2], v, g, lay.in_head, lay.in_token, n_in)) != PSA_OK) return rc;
    if ((rc = encode_text_map(&tm->o[2], out, g, lay.out_head, lay.out_token, n_heads_here)) != PSA_OK) return rc;
  } else {  // never used; keep the descriptors valid
    tm->q[2] = tm->q[0]; tm->k[2] = tm->k[0]; tm->v[2] = tm->v[0]; tm->o[2] = tm->o[0];
  }
  return PSA_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---- helper streams of psa_attn_fwd_host (one set per device, created on first use) ----------
constexpr int kHostChunks = 64;   // upper bound on the chunks of one host-tensor call
struct HostPipe {
  bool ready = false;
  cudaStream_t h2d = nullptr, d2h = nullptr;
  cudaEvent_t ev_start = nullptr, ev_end = nullptr, ev_in[kHostChunks] = {}, ev_done[kHostChunks] = {};
};
HostPipe g_pipe[kMaxDevices];

HostPipe* host_pipe(int dev) {   // caller holds g_mu; returns nullptr if the streams cannot be created
  HostPipe& p = g_pipe[dev];
  if (p.ready) return &p;
  if (cudaStreamCreateWithFlags(&p.h2d, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
  if (cudaStreamCreateWithFlags(&p.d2h, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
  if (cudaEventCreateWithFlags(&p.ev_start, cudaEventDisableTiming) != cudaSuccess) return nullptr;
  if (cudaEventCreateWithFlags(&p.ev_end, cudaEventDisableTiming) != cudaSuccess) return nullptr;
  for (int i = 0; i < kHostChunks; ++i) {
    if (cudaEventCreateWithFlags(&p.ev_in[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&p.ev_done[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
  }
  p.ready = true;
  return &p;
}

// ---- scratch of psa_attn_fwd_noalloc ------------------------------------------------------
// Layout: 16 int32 header words (status, detail, scheduler ticket), kMaxHeads head parameter
// records, then up to kNoAllocMaxItems work items.  It lives in every GPU that loads the
// library, from load to exit.
constexpr int kNoAllocMaxItems = 16384;
constexpr size_t kNoAllocParamsOff = sizeof(int) * kWsHeaderWords;
constexpr size_t kNoAllocItemsOff = (kNoAllocParamsOff + sizeof(psa_head_params) * kMaxHeads + 255) & ~size_t(255);
constexpr size_t kNoAllocBytes = kNoAllocItemsOff + sizeof(WorkItem) * (size_t)kNoAllocMaxItems;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

// Device address of the array, looked up once per device with that device current.  In host
// code the array's name is only a handle for the runtime, never an address a kernel may use.
void* g_noalloc_ptr[kMaxDevices] = {};

int noalloc_scratch(int dev, void** ptr) {
  if (!g_noalloc_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) return PSA_ERR_CUDA;
    g_noalloc_ptr[dev] = p;
  }
  *ptr = g_noalloc_ptr[dev];
  return PSA_OK;
}

}  // namespace

extern "C" {

const char* psa_status_string(int status) {
  switch (status) {
    case PSA_OK: return "ok";
    case PSA_ERR_INVALID_ARG: return "invalid argument";
    case PSA_ERR_UNSUPPORTED: return "unsupported configuration";
    case PSA_ERR_CAPACITY: return "capacity exceeded (col_idx too small, or problem beyond the fixed scratch)";
    case PSA_ERR_CUDA: return "CUDA call failed";
    case PSA_ERR_TIMEOUT: return "device-side wait timed out";
    case PSA_ERR_INTERNAL: return "kernel-side consistency check failed (checked build)";
    default: return "unknown status";
  }
}

int64_t psa_launch_count(void) { return g_launches.load(); }

int psa_profile_events(void* start_event, void* stop_event) {
  std::lock_guard<std::mutex> lock(g_mu);
  if ((start_event == nullptr) != (stop_event == nullptr)) return PSA_ERR_INVALID_ARG;
  g_ev_start = static_cast<cudaEvent_t>(start_event);
  g_ev_stop = static_cast<cudaEvent_t>(stop_event);
  return PSA_OK;
}

int psa_mask_sizes(const psa_head_params* params, const psa_problem* prob, int T, int H, int W, int64_t* nb,
                   int64_t* nnz) {
  Geom g;
  const int rc = make_geom(prob, T, H, W, false, &g);
  if (rc != PSA_OK) return rc;
  if (nb) *nb = g.NB;
  if (nnz) {
    if (!params) return PSA_ERR_INVALID_ARG;
    long long tot = 0;
    for (int h = 0; h < prob->n_heads; ++h) {
      if (!valid_params(params[h])) return PSA_ERR_INVALID_ARG;
      tot += head_nnz(params[h], g);
    }
    *nnz = tot;
  }
  return PSA_OK;
}

int psa_mask_build(const psa_head_params* params, const psa_problem* prob, int T, int H, int W, uint8_t* block_mask,
                   int32_t* row_ptr, int32_t* col_idx, int64_t col_capacity, void* stream) {
  Geom g;
  int rc = make_geom(prob, T, H, W, false, &g);
  if (rc != PSA_OK) return rc;
  if (!params) return PSA_ERR_INVALID_ARG;
  if (col_idx && !row_ptr) return PSA_ERR_INVALID_ARG;
  if (block_mask && !aligned16(block_mask)) return PSA_ERR_INVALID_ARG;
  if ((row_ptr && (reinterpret_cast<uintptr_t>(row_ptr) & 3u)) || (col_idx && (reinterpret_cast<uintptr_t>(col_idx) & 3u)))
    return PSA_ERR_INVALID_ARG;
  // exclusive prefix of the per-head pair counts (host arithmetic, a few thousand operations)
  std::vector<long long> base(prob->n_heads + 1, 0);
  for (int h = 0; h < prob->n_heads; ++h) {
    if (!valid_params(params[h])) return PSA_ERR_INVALID_ARG;
    base[h + 1] = base[h] + head_nnz(params[h], g);
  }
  const long long nnz = base[prob->n_heads];
  if (nnz >= (1ll << 31) || (long long)prob->n_heads * g.NB >= (1ll << 31) - 1) return PSA_ERR_UNSUPPORTED;
  if (col_idx && col_capacity < nnz) return PSA_ERR_CAPACITY;
  int dev;
  Workspace* ws;
  std::lock_guard<std::mutex> lock(g_mu);
  rc = device_info(&dev, &ws);
  if (rc != PSA_OK) return rc;
  for (int head0 = 0; head0 < prob->n_heads; head0 += kMaxHeads) {
    const int n_here = prob->n_heads - head0 < kMaxHeads ? prob->n_heads - head0 : kMaxHeads;
    HeadParamsArray hp;
    int bases[kMaxHeads];
    for (int h = 0; h < n_here; ++h) {
      hp.p[h] = params[head0 + h];
      bases[h] = (int)base[head0 + h];
    }
    int launches = 0;
    const cudaError_t e = launch_mask_build(hp, bases, g, n_here, block_mask ? block_mask + (long long)head0 * g.NB * g.NB : nullptr,
                                            row_ptr ? row_ptr + (long long)head0 * g.NB : nullptr, col_idx,
                                            (int)base[head0 + n_here], ws->n_sms, static_cast<cudaStream_t>(stream), &launches);
    g_launches += launches;
    if (e != cudaSuccess) return PSA_ERR_CUDA;
  }
  return PSA_OK;
}

// Planning + attention launches for n_heads heads (in launches of at most kMaxHeads) on the cached
// per-device workspace.  Arguments are already validated; g_mu is held by the caller.
// clear_status: this is the first launch sequence of an API call (later ones keep the status word).
static int run_attn(const void* q, const void* k, const void* v, void* out, float* lse, const psa_head_params* head_params,
                    int n_heads, const Geom& g, const Layout& lay, cudaStream_t st, bool clear_status = true) {
  int dev;
  Workspace* ws;
  int rc = device_info(&dev, &ws);
  if (rc != PSA_OK) return rc;
  if (ws->cc_major != 10) return PSA_ERR_UNSUPPORTED;
  rc = load_driver_entry();
  if (rc != PSA_OK) return rc;
  const int chunk = n_heads < kMaxHeads ? n_heads : kMaxHeads;
  const size_t items_bytes = sizeof(WorkItem) * (size_t)chunk * g.items_per_head;
  const size_t hp_off = sizeof(int) * kWsHeaderWords;
  const size_t items_off = (hp_off + sizeof(psa_head_params) * kMaxHeads + 255) & ~size_t(255);
  rc = ensure_workspace(ws, items_off + items_bytes);
  if (rc != PSA_OK) return rc;
  int* ws_header = static_cast<int*>(ws->base);
  psa_head_params* hp_dev = reinterpret_cast<psa_head_params*>(static_cast<char*>(ws->base) + hp_off);
  WorkItem* items = reinterpret_cast<WorkItem*>(static_cast<char*>(ws->base) + items_off);
  for (int head0 = 0; head0 < n_heads; head0 += kMaxHeads) {
    const int n_here = n_heads - head0 < kMaxHeads ? n_heads - head0 : kMaxHeads;
    HeadParamsArray hp;
    std::memset(&hp, 0, sizeof(hp));
    for (int h = 0; h < n_here; ++h) hp.p[h] = head_params[head0 + h];
    const long long in_off = lay.shared_qkv ? 0 : (long long)head0 * lay.in_head;
    const long long out_off = (long long)head0 * lay.out_head;
    TensorMaps tm;
    if ((rc = encode_maps(&tm, static_cast<const uint16_t*>(q) + in_off, static_cast<const uint16_t*>(k) + in_off,
                          static_cast<const uint16_t*>(v) + in_off, static_cast<uint16_t*>(out) + out_off, g, lay, n_here)) != PSA_OK)
      return rc;
    Geom gh = g;
    gh.n_heads = n_here;
    if (launch_plan(hp, gh, 0, n_here, clear_status && head0 == 0, ws_header, hp_dev, items, st) != cudaSuccess)
      return PSA_ERR_CUDA;
    ++g_launches;
    const int n_items = n_here * g.items_per_head;
    if (g_ev_start && g_ev_stop) cudaEventRecord(g_ev_start, st);
    if (launch_attn(tm, gh, items, hp_dev, ws_header, lse + (long long)head0 * g.Lt, n_items, ws->n_sms, lay.shared_qkv, st) !=
        cudaSuccess)
      return PSA_ERR_CUDA;
    if (g_ev_start && g_ev_stop) cudaEventRecord(g_ev_stop, st);
    ++g_launches;
  }
  return PSA_OK;
}

// psa_attn_fwd with the choice of keeping the status word (chunks of one host-tensor call).
static int attn_fwd_checked(const void* q, const void* k, const void* v, void* out, float* lse,
                            const psa_head_params* head_params, const psa_problem* prob, int T, int H, int W, void* stream,
                            bool clear_status) {
  Geom g;
  int rc = make_geom(prob, T, H, W, true, &g);
  if (rc != PSA_OK) return rc;
  if (!q || !k || !v || !out || !lse || !head_params) return PSA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || (reinterpret_cast<uintptr_t>(lse) & 3u))
    return PSA_ERR_INVALID_ARG;
  if (out == q || out == k || out == v) return PSA_ERR_INVALID_ARG;
  if (prob->stride_token < kHeadDim || (prob->stride_token % 8) != 0) return PSA_ERR_INVALID_ARG;
  if (prob->n_heads > 1 && (prob->stride_head < kHeadDim || (prob->stride_head % 8) != 0)) return PSA_ERR_INVALID_ARG;
  for (int h = 0; h < prob->n_heads; ++h)
    if (!valid_params(head_params[h])) return PSA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_mu);
  const Layout lay = {prob->stride_head, prob->stride_token, prob->stride_head, prob->stride_token, false};
  return run_attn(q, k, v, out, lse, head_params, prob->n_heads, g, lay, static_cast<cudaStream_t>(stream), clear_status);
}

int psa_attn_fwd(const void* q, const void* k, const void* v, void* out, float* lse, const psa_head_params* head_params,
                 const psa_problem* prob, int T, int H, int W, void* stream) {
  return attn_fwd_checked(q, k, v, out, lse, head_params, prob, T, H, W, stream, true);
}

int psa_search_select_at_sparsity(const float* losses, const float* sparsity, int n, float target) {
  if (!losses || !sparsity || n < 1) return PSA_ERR_INVALID_ARG;
  int best = -1;
  for (int i = 0; i < n; ++i)
    if (sparsity[i] >= target && (best < 0 || losses[i] < losses[best])) best = i;
  return best < 0 ? PSA_ERR_CAPACITY : best;
}

int psa_attn_fwd_batched(const void* q, const void* k, const void* v, void* out, float* lse,
                         const psa_head_params* head_params, const psa_problem* prob, int n_batch, int64_t stride_batch,
                         int T, int H, int W, void* stream) {
  Geom g;
  int rc = make_geom(prob, T, H, W, true, &g);
  if (rc != PSA_OK) return rc;
  if (!q || !k || !v || !out || !lse || !head_params || n_batch < 1) return PSA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || (reinterpret_cast<uintptr_t>(lse) & 3u))
    return PSA_ERR_INVALID_ARG;
  if (out == q || out == k || out == v) return PSA_ERR_INVALID_ARG;
  if (prob->stride_token < kHeadDim || (prob->stride_token % 8) != 0) return PSA_ERR_INVALID_ARG;
  if (prob->n_heads > 1 && (prob->stride_head < kHeadDim || (prob->stride_head % 8) != 0)) return PSA_ERR_INVALID_ARG;
  if (n_batch > 1 && (stride_batch < kHeadDim || (stride_batch % 8) != 0)) return PSA_ERR_INVALID_ARG;
  for (int h = 0; h < prob->n_heads; ++h)
    if (!valid_params(head_params[h])) return PSA_ERR_INVALID_ARG;
  const int nh = prob->n_heads;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  std::lock_guard<std::mutex> lock(g_mu);
  const bool fold = n_batch == 1 || (nh == 1 ? true : stride_batch == (int64_t)nh * prob->stride_head);
  if (fold) {
    // samples are evenly spaced heads: one launch sequence over n_batch * n_heads heads
    if ((long long)n_batch * nh >= (1ll << 24)) return PSA_ERR_UNSUPPORTED;
    std::vector<psa_head_params> params((size_t)n_batch * nh);
    for (int b = 0; b < n_batch; ++b)
      for (int h = 0; h < nh; ++h) params[(size_t)b * nh + h] = head_params[h];
    const long long hs = nh == 1 ? (n_batch > 1 ? stride_batch : prob->stride_head) : prob->stride_head;
    const Layout lay = {hs, prob->stride_token, hs, prob->stride_token, false};
    return run_attn(q, k, v, out, lse, params.data(), n_batch * nh, g, lay, st);
  }
  const Layout lay = {prob->stride_head, prob->stride_token, prob->stride_head, prob->stride_token, false};
  for (int b = 0; b < n_batch; ++b) {
    const long long off = (long long)b * stride_batch;
    rc = run_attn(static_cast<const uint16_t*>(q) + off, static_cast<const uint16_t*>(k) + off,
                  static_cast<const uint16_t*>(v) + off, static_cast<uint16_t*>(out) + off,
                  lse + (long long)b * nh * g.L, head_params, nh, g, lay, st, b == 0);
    if (rc != PSA_OK) return rc;
  }
  return PSA_OK;
}

int psa_attn_fwd_joint(const void* q, const void* k, const void* v, void* out, float* lse,
                       const psa_head_params* head_params, const psa_problem* prob, int64_t n_text, int T, int H, int W,
                       void* stream) {
  Geom g;
  int rc = make_geom(prob, T, H, W, true, &g);
  if (rc != PSA_OK) return rc;
  if ((rc = set_text(&g, n_text)) != PSA_OK) return rc;
  if (!q || !k || !v || !out || !lse || !head_params) return PSA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || (reinterpret_cast<uintptr_t>(lse) & 3u))
    return PSA_ERR_INVALID_ARG;
  if (out == q || out == k || out == v) return PSA_ERR_INVALID_ARG;
  if (prob->stride_token < kHeadDim || (prob->stride_token % 8) != 0) return PSA_ERR_INVALID_ARG;
  if (prob->n_heads > 1 && (prob->stride_head < kHeadDim || (prob->stride_head % 8) != 0)) return PSA_ERR_INVALID_ARG;
  for (int h = 0; h < prob->n_heads; ++h)
    if (!valid_params(head_params[h])) return PSA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_mu);
  const Layout lay = {prob->stride_head, prob->stride_token, prob->stride_head, prob->stride_token, false};
  return run_attn(q, k, v, out, lse, head_params, prob->n_heads, g, lay, static_cast<cudaStream_t>(stream));
}

// ---- PSA-Search for one head (Algorithm 3) ------------------------------------------------------
// scratch layout: outputs of the n_cand candidates and of full attention ((n_cand + 1) x L x 128 bf16),
// their lse ((n_cand + 1) x L fp32), the partial sums of the loss reduction.
static size_t search_out_bytes(int n_cand, long long L) { return ((size_t)(n_cand + 1) * L * kHeadDim * 2 + 255) & ~size_t(255); }
static size_t search_lse_bytes(int n_cand, long long L) { return ((size_t)(n_cand + 1) * L * 4 + 255) & ~size_t(255); }

int64_t psa_search_scratch_bytes(int n_cand, int T, int H, int W) {
  if (n_cand < 1 || T < 1 || H < 1 || W < 1) return PSA_ERR_INVALID_ARG;
  const long long L = (long long)T * H * W;
  return (int64_t)(search_out_bytes(n_cand, L) + search_lse_bytes(n_cand, L) + search_partial_bytes(n_cand));
}

int psa_search_losses(const void* q, const void* k, const void* v, const psa_head_params* candidates, int n_cand,
                      const psa_problem* prob, int T, int H, int W, void* scratch, float* losses, void* stream) {
  Geom g;
  int rc = make_geom(prob, T, H, W, true, &g);
  if (rc != PSA_OK) return rc;
  if (!q || !k || !v || !candidates || !scratch || !losses || n_cand < 1) return PSA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || (reinterpret_cast<uintptr_t>(scratch) & 255u) ||
      (reinterpret_cast<uintptr_t>(losses) & 3u))
    return PSA_ERR_INVALID_ARG;
  if (prob->stride_token < kHeadDim || (prob->stride_token % 8) != 0) return PSA_ERR_INVALID_ARG;
  // candidate masks, then one all-covering mask: full attention with the same kernel
  std::vector<psa_head_params> params(candidates, candidates + n_cand);
  for (int c = 0; c < n_cand; ++c)
    if (!valid_params(params[c])) return PSA_ERR_INVALID_ARG;
  const psa_head_params full = {g.Tp, 0, 0, g.Sp, 0, 0};
  params.push_back(full);
  char* base = static_cast<char*>(scratch);
  uint16_t* outs = reinterpret_cast<uint16_t*>(base);
  float* lse = reinterpret_cast<float*>(base + search_out_bytes(n_cand, g.L));
  double* partial = reinterpret_cast<double*>(base + search_out_bytes(n_cand, g.L) + search_lse_bytes(n_cand, g.L));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  std::lock_guard<std::mutex> lock(g_mu);
  const Layout lay = {0, prob->stride_token, g.L * kHeadDim, kHeadDim, true};
  rc = run_attn(q, k, v, outs, lse, params.data(), n_cand + 1, g, lay, st);
  if (rc != PSA_OK) return rc;
  int launches = 0;
  const cudaError_t e = launch_search_losses(outs, outs + (long long)n_cand * g.L * kHeadDim, g.L * kHeadDim, n_cand, partial,
                                             losses, st, &launches);
  g_launches += launches;
  return e == cudaSuccess ? PSA_OK : PSA_ERR_CUDA;
}

int psa_search_select(const float* losses, const float* sparsity, int n, float alpha) {
  if (!losses || !sparsity || n < 1) return PSA_ERR_INVALID_ARG;
  // Algorithm 3 walks the candidates in order of (loss, index), starts at the first and moves to
  // any strictly sparser one whose loss is within alpha.  Its result, stated directly: if no loss
  // is within alpha, the candidate of minimal (loss, index); otherwise the sparsest candidate
  // among those within alpha, ties by minimal (loss, index).
  int lowest = -1, best = -1;
  for (int i = 0; i < n; ++i) {
    if (!std::isfinite(losses[i]) || std::isnan(sparsity[i])) return PSA_ERR_INVALID_ARG;
    if (lowest < 0 || losses[i] < losses[lowest]) lowest = i;
    if (losses[i] <= alpha &&
        (best < 0 || sparsity[i] > sparsity[best] || (sparsity[i] == sparsity[best] && losses[i] < losses[best])))
      best = i;
  }
  return best >= 0 ? best : lowest;
}

int psa_attn_fwd_noalloc(const void* q, const void* k, const void* v, void* out, float* lse,
                         const psa_head_params* head_params, const psa_problem* prob, int T, int H, int W, void* stream,
                         int32_t* status_detail) {
  Geom g;
  int rc = make_geom(prob, T, H, W, true, &g);
  if (rc != PSA_OK) return rc;
  if (!q || !k || !v || !out || !lse || !head_params) return PSA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || (reinterpret_cast<uintptr_t>(lse) & 3u))
    return PSA_ERR_INVALID_ARG;
  if (out == q || out == k || out == v) return PSA_ERR_INVALID_ARG;
  if (prob->stride_token < kHeadDim || (prob->stride_token % 8) != 0) return PSA_ERR_INVALID_ARG;
  if (prob->n_heads > 1 && (prob->stride_head < kHeadDim || (prob->stride_head % 8) != 0)) return PSA_ERR_INVALID_ARG;
  for (int h = 0; h < prob->n_heads; ++h)
    if (!valid_params(head_params[h])) return PSA_ERR_INVALID_ARG;
  // the fixed scratch bounds the problem: one launch worth of heads and kNoAllocMaxItems items
  const long long n_items_ll = (long long)prob->n_heads * g.items_per_head;
  if (prob->n_heads > kMaxHeads || n_items_ll > kNoAllocMaxItems) return PSA_ERR_CAPACITY;

  std::lock_guard<std::mutex> lock(g_mu);
  int dev;
  Workspace* ws;
  rc = device_info(&dev, &ws);
  if (rc != PSA_OK) return rc;
  if (ws->cc_major != 10) return PSA_ERR_UNSUPPORTED;
  rc = load_driver_entry();
  if (rc != PSA_OK) return rc;
  void* base = nullptr;
  rc = noalloc_scratch(dev, &base);
  if (rc != PSA_OK) return rc;
  int* header = static_cast<int*>(base);
  psa_head_params* hp_dev = reinterpret_cast<psa_head_params*>(static_cast<char*>(base) + kNoAllocParamsOff);
  WorkItem* items = reinterpret_cast<WorkItem*>(static_cast<char*>(base) + kNoAllocItemsOff);
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  HeadParamsArray hp;
  std::memset(&hp, 0, sizeof(hp));
  for (int h = 0; h < prob->n_heads; ++h) hp.p[h] = head_params[h];
  TensorMaps tm;
  const Layout lay = {prob->stride_head, prob->stride_token, prob->stride_head, prob->stride_token, false};
  if ((rc = encode_maps(&tm, q, k, v, out, g, lay, prob->n_heads)) != PSA_OK) return rc;
  // The planning kernel clears the header words (status, ticket) and rewrites the parameter
  // records and every work item of this call, so nothing of the previous call is read.
  if (launch_plan(hp, g, 0, prob->n_heads, true, header, hp_dev, items, st) != cudaSuccess) return PSA_ERR_CUDA;
  ++g_launches;
  if (launch_attn(tm, g, items, hp_dev, header, lse, (int)n_items_ll, ws->n_sms, false, st) != cudaSuccess)
    return PSA_ERR_CUDA;
  ++g_launches;
  if (status_detail) {
    if (cudaStreamSynchronize(st) != cudaSuccess) return PSA_ERR_CUDA;
    int hdr[2] = {0, 0};
    if (cudaMemcpy(hdr, header, sizeof(hdr), cudaMemcpyDeviceToHost) != cudaSuccess) return PSA_ERR_CUDA;
    *status_detail = hdr[1];
    return hdr[0];
  }
  return PSA_OK;
}

int psa_attn_fwd_host(const void* q, const void* k, const void* v, void* out, float* lse, void* d_q, void* d_k, void* d_v,
                      void* d_out, float* d_lse, const psa_head_params* head_params, const psa_problem* prob, int T, int H,
                      int W, void* stream) {
  if (!prob || !q || !k || !v || !out || !lse || !d_q || !d_k || !d_v || !d_out || !d_lse || !head_params)
    return PSA_ERR_INVALID_ARG;
  if (T < 1 || H < 1 || W < 1 || prob->n_heads < 1) return PSA_ERR_INVALID_ARG;
  const long long L = (long long)T * H * W;
  const size_t head_span = (size_t)(L - 1) * prob->stride_token + prob->head_dim;  // elements one head touches
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  // Heads are independent problems: when they are the outermost dimension of the layout the
  // call is pipelined over chunks of heads -- chunk c+1 is copied in and chunk c-1 copied out
  // while chunk c computes (two helper streams per device, created on first use).
  const bool head_major = prob->n_heads == 1 || (size_t)prob->stride_head >= head_span;
  int dev = 0;
  HostPipe* pipe = nullptr;
  if (head_major && prob->n_heads >= 2 && cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < kMaxDevices) {
    std::lock_guard<std::mutex> lock(g_mu);
    pipe = host_pipe(dev);
  }
  if (!pipe) {
    const size_t bytes = ((size_t)(prob->n_heads - 1) * prob->stride_head + head_span) * 2;
    if (cudaMemcpyAsync(d_q, q, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return PSA_ERR_CUDA;
    if (cudaMemcpyAsync(d_k, k, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return PSA_ERR_CUDA;
    if (cudaMemcpyAsync(d_v, v, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return PSA_ERR_CUDA;
    const int rc = psa_attn_fwd(d_q, d_k, d_v, d_out, d_lse, head_params, prob, T, H, W, stream);
    if (rc != PSA_OK) return rc;
    if (cudaMemcpyAsync(out, d_out, bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return PSA_ERR_CUDA;
    if (cudaMemcpyAsync(lse, d_lse, sizeof(float) * (size_t)prob->n_heads * L, cudaMemcpyDeviceToHost, st) != cudaSuccess)
      return PSA_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return PSA_ERR_CUDA;
    return PSA_OK;
  }

  // Chunk size: the call is bound by the host-to-device copies, so what is exposed is the first
  // chunk's copy-in and the last chunk's compute and copy-out -- both shrink with the chunk.
  int want = host_chunks();
  if (want > kHostChunks - 8) want = kHostChunks - 8;   // single-head edge chunks and broken runs add a few
  const int n_chunks = prob->n_heads < want ? prob->n_heads : want;
  const int per = (prob->n_heads + n_chunks - 1) / n_chunks;
  // everything enqueued on `stream` before this call precedes the first copy
  if (cudaEventRecord(pipe->ev_start, st) != cudaSuccess) return PSA_ERR_CUDA;
  if (cudaStreamWaitEvent(pipe->h2d, pipe->ev_start, 0) != cudaSuccess) return PSA_ERR_CUDA;
  if (cudaStreamWaitEvent(pipe->d2h, pipe->ev_start, 0) != cudaSuccess) return PSA_ERR_CUDA;
  // The first and the last chunks are the exposed ones, so the call starts and ends with
  // single-head chunks (two at each end, when the regular chunk is larger than that), and the two
  // heads with the fewest attended block pairs (the shortest kernels) are kept for the end: what
  // remains after the last byte has arrived is the lightest head's kernel and its copy-out.
  const int n_edge = (per >= 2 && prob->n_heads >= 4 * per) ? 2 : 0;
  struct Chunk { int h0, nh; };
  Chunk chunks[kHostChunks];
  int n_list = 0;
  int last1 = -1, last2 = -1;   // lightest and second-lightest head
  if (n_edge) {
    Geom g;
    const int rcg = make_geom(prob, T, H, W, true, &g);
    if (rcg != PSA_OK) return rcg;
    long long w1 = 0, w2 = 0;
    for (int h = 0; h < prob->n_heads; ++h) {
      if (!valid_params(head_params[h])) return PSA_ERR_INVALID_ARG;
      const long long w = head_nnz(head_params[h], g);
      if (last1 < 0 || w < w1) { last2 = last1; w2 = w1; last1 = h; w1 = w; }
      else if (last2 < 0 || w < w2) { last2 = h; w2 = w; }
    }
  }
  {
    int singles = n_edge;   // single-head chunks still to open the call with
    int h = 0;
    while (h < prob->n_heads) {
      if (h == last1 || h == last2) { ++h; continue; }
      int nh = 1;
      if (singles > 0) --singles;
      else
        while (nh < per && h + nh < prob->n_heads && h + nh != last1 && h + nh != last2) ++nh;
      if (n_list >= kHostChunks - 2) return PSA_ERR_UNSUPPORTED;
      chunks[n_list++] = Chunk{h, nh};
      h += nh;
    }
    if (last2 >= 0) chunks[n_list++] = Chunk{last2, 1};
    if (last1 >= 0) chunks[n_list++] = Chunk{last1, 1};
  }
  for (int c = 0; c < n_list; ++c) {
    const int h0 = chunks[c].h0, nh = chunks[c].nh;
    const size_t off = (size_t)h0 * prob->stride_head;                       // elements
    const size_t bytes = ((size_t)(nh - 1) * prob->stride_head + head_span) * 2;
    const uint16_t *hq = static_cast<const uint16_t*>(q) + off, *hk = static_cast<const uint16_t*>(k) + off,
                   *hv = static_cast<const uint16_t*>(v) + off;
    uint16_t *dq = static_cast<uint16_t*>(d_q) + off, *dk = static_cast<uint16_t*>(d_k) + off,
             *dv = static_cast<uint16_t*>(d_v) + off, *dout = static_cast<uint16_t*>(d_out) + off;
    if (cudaMemcpyAsync(dq, hq, bytes, cudaMemcpyHostToDevice, pipe->h2d) != cudaSuccess) return PSA_ERR_CUDA;
    if (cudaMemcpyAsync(dk, hk, bytes, cudaMemcpyHostToDevice, pipe->h2d) != cudaSuccess) return PSA_ERR_CUDA;
    if (cudaMemcpyAsync(dv, hv, bytes, cudaMemcpyHostToDevice, pipe->h2d) != cudaSuccess) return PSA_ERR_CUDA;
    if (cudaEventRecord(pipe->ev_in[c], pipe->h2d) != cudaSuccess) return PSA_ERR_CUDA;
    if (cudaStreamWaitEvent(st, pipe->ev_in[c], 0) != cudaSuccess) return PSA_ERR_CUDA;
    psa_problem sub = *prob;
    sub.n_heads = nh;
    const int rc = attn_fwd_checked(dq, dk, dv, dout, d_lse + (size_t)h0 * L, head_params + h0, &sub, T, H, W, stream, c == 0);
    if (rc != PSA_OK) return rc;
    if (cudaEventRecord(pipe->ev_done[c], st) != cudaSuccess) return PSA_ERR_CUDA;
    if (cudaStreamWaitEvent(pipe->d2h, pipe->ev_done[c], 0) != cudaSuccess) return PSA_ERR_CUDA;
    if (cudaMemcpyAsync(static_cast<uint16_t*>(out) + off, dout, bytes, cudaMemcpyDeviceToHost, pipe->d2h) != cudaSuccess)
      return PSA_ERR_CUDA;
    if (cudaMemcpyAsync(lse + (size_t)h0 * L, d_lse + (size_t)h0 * L, sizeof(float) * (size_t)nh * L, cudaMemcpyDeviceToHost,
                        pipe->d2h) != cudaSuccess)
      return PSA_ERR_CUDA;
  }
  if (cudaEventRecord(pipe->ev_end, pipe->d2h) != cudaSuccess) return PSA_ERR_CUDA;
  if (cudaStreamWaitEvent(st, pipe->ev_end, 0) != cudaSuccess) return PSA_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return PSA_ERR_CUDA;
  return PSA_OK;
}

int psa_selftest_wait_timeout(int limit_ms, void* stream) {
  if (limit_ms < 1 || limit_ms > 1000) return PSA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_mu);
  int dev;
  Workspace* ws;
  int rc = device_info(&dev, &ws);
  if (rc != PSA_OK) return rc;
  rc = ensure_workspace(ws, 4096);
  if (rc != PSA_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(ws->base, 0, sizeof(int) * kWsHeaderWords, st) != cudaSuccess) return PSA_ERR_CUDA;
  if (launch_wait_probe(static_cast<int*>(ws->base), 1000000ull * (unsigned long long)limit_ms, st) != cudaSuccess)
    return PSA_ERR_CUDA;
  ++g_launches;
  return PSA_OK;
}

int psa_last_device_status(int32_t* detail) {
  std::lock_guard<std::mutex> lock(g_mu);
  int dev;
  Workspace* ws;
  int rc = device_info(&dev, &ws);
  if (rc != PSA_OK) return rc;
  if (cudaDeviceSynchronize() != cudaSuccess) return PSA_ERR_CUDA;
  if (detail) *detail = 0;
  if (!ws->base) return PSA_OK;
  int hdr[2] = {0, 0};
  if (cudaMemcpy(hdr, ws->base, sizeof(hdr), cudaMemcpyDeviceToHost) != cudaSuccess) return PSA_ERR_CUDA;
  if (detail) *detail = hdr[1];
  return hdr[0];
}

int psa_shutdown(void) {
  std::lock_guard<std::mutex> lock(g_mu);
  int cur = 0;
  if (cudaGetDevice(&cur) != cudaSuccess) return PSA_OK;  // no usable device: nothing was allocated
  for (int d = 0; d < kMaxDevices; ++d) {
    if (g_ws[d].base) {
      cudaSetDevice(d);
      cudaDeviceSynchronize();
      cudaFree(g_ws[d].base);
      g_ws[d].base = nullptr;
      g_ws[d].bytes = 0;
    }
  }
  cudaSetDevice(cur);
  return PSA_OK;
}

}  // extern "C"
