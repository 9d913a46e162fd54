/*
 * psa.h -- C ABI of the B200 (sm_100a) parameterized-stripe-attention library.
 *
 * The library computes the forward pass of block-sparse video attention whose
 * per-head mask is generated from six integers M(T_w, T_o, T_s, S_w, S_o, S_s)
 * (Section 3.2, "Unified Representation", and Algorithm 1), applied at PSABlock
 * granularity (Section 3.2, "Hardware-Aware Design") on the 3D-padded block grid
 * (Section 3.2, "3D-Padding"), followed by flash-style attention over the
 * surviving blocks (Appendix B, Algorithm 2).
 *
 * Conventions shared by every call
 *   - Tokens are in frame-major, row-major order i = t*H*W + h*W + w (Appendix D,
 *     Proposition 1).  L = T*H*W.
 *   - A mask block (the paper's PSABlock) is a brick of tile.bt x tile.bh x tile.bw
 *     tokens.  Block grid T' = ceil(T/bt), H' = ceil(H/bh), W' = ceil(W/bw),
 *     S' = H'*W', NB = T'*S'.  Block id = t'*S' + h'*W' + w'.
 *   - The six parameters are in block units.  Query block (t'_q, s'_q) attends key
 *     block (t'_k, s'_k) iff  (|t'_k - t'_q - T_o| mod T_s) <= T_w - 1  and
 *     (|s'_k - s'_q - S_o| mod S_s) <= S_w - 1  (Algorithm 1).  A stride of 0 encodes
 *     an infinite stride: no modulo, one diagonal band (Appendix C.2).
 *   - "host" / "device" on a pointer says where the memory must live.  The library
 *     never takes ownership of caller memory.  Device work is enqueued on `stream`
 *     (a cudaStream_t passed as void*; NULL = the default stream) and the calls
 *     return without synchronising unless stated.
 *   - Return value: PSA_OK (0) or a negative psa_status.  Nothing is thrown, printed
 *     or aborted.
 *   - The library keeps one lazily created device workspace per device (work order,
 *     status word); calls that overlap on the GPU from different streams race on it.
 *     psa_shutdown() frees it.  Once a call has sized that workspace, psa_mask_build and
 *     psa_attn_fwd of the same or a smaller problem allocate nothing and synchronise nothing:
 *     they can be captured in a CUDA graph and replayed (all arguments are captured by value;
 *     the buffers' contents may change between replays).
 */
#ifndef PSA_H_
#define PSA_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  PSA_OK = 0,
  PSA_ERR_INVALID_ARG = -1, /* null/misaligned pointer, non-positive extent, bad parameter   */
  PSA_ERR_UNSUPPORTED = -2, /* head_dim != 128, unsupported tile shape, not sm_100             */
  PSA_ERR_CAPACITY = -3,    /* col_capacity < nnz                                             */
  PSA_ERR_CUDA = -4,        /* a CUDA runtime/driver call failed                              */
  PSA_ERR_TIMEOUT = -5,     /* a bounded device-side wait expired (see psa_last_device_status) */
  PSA_ERR_INTERNAL = -6     /* checked build only: a kernel-side index / coordinate check failed    */
} psa_status;

/* Six stripe parameters of one head, in block units (Section 3.2).  Ts == 0 / Ss == 0
 * mean an infinite stride.  Valid: Tw, Sw >= 1; Ts, Ss >= 0; |To|, |So| < 2^30. */
typedef struct { int32_t Tw, To, Ts, Sw, So, Ss; } psa_head_params;

/* Mask block (PSABlock) extents in tokens.  psa_attn_fwd splits a block into compute slabs
 * along its outermost axis of extent > 1: slabs of exactly 128 tokens plus a last slab of
 * 128, 112, 96 or 64 tokens, at most three slabs (128 <= bt*bh*bw <= 384).  Examples:
 * 1x16x16 = 128+128, 3x8x16 = 3 x 128, 1x15x16 = 128+112 (tiles a 45-row grid without
 * padding).  Other shapes return PSA_ERR_UNSUPPORTED. */
typedef struct { int32_t bt, bh, bw; } psa_tile;

typedef struct {
  int32_t  n_heads;      /* >= 1                                                          */
  int32_t  head_dim;     /* must be 128 for psa_attn_fwd                                   */
  psa_tile tile;
  float    scale;        /* softmax scale applied to q.k (the configs use 1/sqrt(128))     */
  int64_t  stride_head;  /* elements between heads, shared by q, k, v, out                 */
  int64_t  stride_token; /* elements between tokens (>= head_dim, multiple of 8)           */
} psa_problem;

/* Sizes of psa_mask_build's outputs.  *nb = NB; *nnz = number of attended block pairs
 * summed over heads (exact; params is host memory, n_heads entries).  Pure host code. */
int psa_mask_sizes(const psa_head_params* params, const psa_problem* prob,
                   int T, int H, int W, int64_t* nb, int64_t* nnz);

/* GetKVBlocks for every (head, query block) (Algorithm 2, producer; Algorithm 1):
 *   block_mask  device uint8 [n_heads][NB][NB], 1 = attended (row = query block)
 *   row_ptr     device int32 [n_heads*NB + 1], exclusive prefix sum of row counts in
 *               (head, query block) order
 *   col_idx     device int32 [col_capacity], ascending key-block ids of each row
 * params: host, n_heads entries.  If col_capacity < nnz nothing is launched and
 * PSA_ERR_CAPACITY is returned (use psa_mask_sizes).  Any of the three outputs may be
 * NULL to skip it (col_idx needs row_ptr).  Integer work only; results are exact. */
int psa_mask_build(const psa_head_params* params, const psa_problem* prob,
                   int T, int H, int W, uint8_t* block_mask, int32_t* row_ptr,
                   int32_t* col_idx, int64_t col_capacity, void* stream);

/* Forward pass (Algorithm 2 with the mask of Algorithm 1 decided in-kernel):
 *   q, k, v   device bf16, element (head, token, c) at head*stride_head + token*stride_token + c
 *   out       device bf16, same strides; must not alias the inputs
 *   lse       device fp32 [n_heads][L], natural log of the sum of exp(scale * q.k) over
 *             attended real keys
 *   head_params host, n_heads entries
 * Rows whose query block attends no key block get out = 0 and lse = -inf.  Padded
 * positions (Section 3.2, "3D-Padding") are never read from or written to memory.
 * Pointers must be 16-byte aligned.  bf16 inputs, fp32 accumulation.
 * Precondition: the attention kernel takes every SM whole (one CTA with 226 KB of shared memory
 * and all 512 tensor-memory columns) and its tensor-memory allocation blocks until the columns are
 * free, so no other kernel that allocates tensor memory may run on the device at the same time
 * (other processes, or other streams of this process).  Every later wait inside the kernel has
 * a time limit and is reported through psa_last_device_status(). */
int psa_attn_fwd(const void* q, const void* k, const void* v, void* out, float* lse,
                 const psa_head_params* head_params, const psa_problem* prob,
                 int T, int H, int W, void* stream);

/* psa_attn_fwd for callers that must not allocate device memory (the paper has no
 * counterpart; this is a property of the library, not of the method).
 *
 * Some callers cannot tolerate a cudaMalloc inside a library call: a serving loop whose
 * device memory is entirely owned by a framework's pool, a plugin hook whose contract forbids
 * allocation, or latency-critical code for which the device-wide synchronisation that
 * cudaMalloc/cudaFree imply is unacceptable.  psa_attn_fwd grows a cached workspace with
 * cudaMalloc when a larger problem arrives; this variant never does.  Its scratch (status
 * word, scheduler ticket, per-head parameters, work order) is a fixed array of about 260 KB
 * that is part of the library image: every GPU that loads the library holds it until exit.
 *
 * Same arguments, layouts and results as psa_attn_fwd, plus:
 *   status_detail  host, optional.  NULL: the call only enqueues work on `stream`.  Non-NULL:
 *                  the call synchronises `stream`, stores the kernel's diagnostic word there
 *                  and returns PSA_ERR_TIMEOUT if a bounded device-side wait expired.
 * Limits: n_heads <= 128 and n_heads * NB * ceil(slabs_per_block / 2) <= 16384 work items
 * (Wan 2.1 14B at 1x16x16: 12,600); larger problems return PSA_ERR_CAPACITY and launch nothing.
 * The first call on a device looks up the array's device address (with that device current);
 * make that first call before any stream capture begins.  Every call on a device shares the
 * array: the planning kernel clears the words that must start at zero and rewrites the rest,
 * so back-to-back calls on one stream are fine, but calls that overlap on the GPU (different
 * streams) race on it.  The status word of this variant is not visible to
 * psa_last_device_status(), and the event pair registered with psa_profile_events() is not
 * recorded by it.  No cudaMalloc, cudaFree or other allocating call is made. */
int psa_attn_fwd_noalloc(const void* q, const void* k, const void* v, void* out, float* lse,
                         const psa_head_params* head_params, const psa_problem* prob,
                         int T, int H, int W, void* stream, int32_t* status_detail);

/* The same call for HOST tensors: copies q, k, v (host; pinned memory is needed for the
 * copies to overlap) into the caller's device staging buffers d_q, d_k, d_v, runs
 * psa_attn_fwd into d_out / d_lse and copies the results to out / lse (host), ordered
 * after the work already on `stream`, then synchronises `stream`.  When heads are the
 * outermost dimension of the layout the call is pipelined over chunks of heads (20 by default,
 * from a measured sweep; the environment variable PSA_HOST_CHUNKS overrides it) on two internal
 * helper streams: the next chunk is copied in and the previous one copied out while a chunk
 * computes.  Chunks are contiguous head ranges but need not run in head order: the call opens
 * with single heads and keeps the two heads with the fewest attended block pairs for the end.
 * Each staging buffer must hold the full strided extent of its tensor:
 * (n_heads-1)*stride_head + (L-1)*stride_token + head_dim elements. */
int psa_attn_fwd_host(const void* q, const void* k, const void* v, void* out, float* lse,
                      void* d_q, void* d_k, void* d_v, void* d_out, float* d_lse,
                      const psa_head_params* head_params, const psa_problem* prob,
                      int T, int H, int W, void* stream);

/* Batched call (what one DiT attention layer issues: batch > 1, or the conditional / unconditional
 * pair of classifier-free guidance).  The paper assigns masks per head, not per sample, so all
 * n_batch samples use the same head_params.  Element (b, head, token, c) of q, k, v, out sits at
 * b*stride_batch + head*stride_head + token*stride_token + c; lse is [n_batch][n_heads][L].
 * When the batches are evenly spaced heads (stride_batch == n_heads*stride_head) all samples run in
 * one launch sequence, otherwise sample by sample.  Everything else as psa_attn_fwd. */
int psa_attn_fwd_batched(const void* q, const void* k, const void* v, void* out, float* lse,
                         const psa_head_params* head_params, const psa_problem* prob, int n_batch,
                         int64_t stride_batch, int T, int H, int W, void* stream);

/* Joint video + text sequence (multimodal DiT blocks such as HunyuanVideo's, which attend over the
 * video tokens and the prompt's text tokens together).  The paper defines the stripe mask on the video
 * grid and is silent on the text tokens; the reading taken: the mask applies between video tokens,
 * every query attends every text key, and a text query attends every key.
 *   q, k, v, out  device bf16; every head holds L = T*H*W video tokens followed by n_text text tokens
 *                 (token index L .. L+n_text-1), element (head, token, c) at
 *                 head*stride_head + token*stride_token + c
 *   lse           device fp32 [n_heads][L + n_text]
 *   n_text        >= 0 (0 is psa_attn_fwd); at most 65535 * 128
 * Text keys travel as extra 128-token key slabs after the attended video slabs of every work item
 * (a ragged last slab is zero-filled and masked); text queries are extra work items that attend all
 * key blocks.  Everything else as psa_attn_fwd. */
int psa_attn_fwd_joint(const void* q, const void* k, const void* v, void* out, float* lse,
                       const psa_head_params* head_params, const psa_problem* prob, int64_t n_text,
                       int T, int H, int W, void* stream);

/* PSA-Search for ONE head (Appendix C, Algorithm 3).
 *
 * psa_search_losses: the inner loop -- Loss(M) = L2Loss(PSA(h, M), FullAttn(h)) for every candidate
 * mask M.  All n_cand candidates and full attention (an all-covering mask) run in one launch of the
 * stripe attention kernel on the same q, k, v; then loss[c] = mean over all L*128 output elements of
 * (out_c - out_full)^2 (the paper does not spell the loss out; mean squared difference is the reading
 * taken).  q, k, v: device bf16, ONE head, element (token, c) at token*stride_token + c (prob->n_heads
 * and stride_head are ignored; tile, scale, head_dim as for psa_attn_fwd).  candidates: host.
 * scratch: device, 256-byte aligned, psa_search_scratch_bytes(n_cand, T, H, W) bytes (holds every
 * candidate's output).  losses: device fp32 [n_cand].  Asynchronous on `stream`.
 *
 * psa_search_select: the selection -- sort by loss ascending (ties by index), start from the
 * lowest-loss candidate, and among candidates with loss <= alpha move to any strictly sparser one.
 * losses, sparsity: host arrays of n entries (sparsity = excluded fraction of block pairs, e.g. from
 * psa_mask_sizes).  Returns the chosen index (>= 0) or a negative psa_status (PSA_ERR_INVALID_ARG
 * when a loss is not finite or a sparsity is NaN).  Pure host code.
 *
 * psa_search_select_at_sparsity: the second interface of Section 3.3 -- for a target sparsity, the
 * candidate of minimal loss among those with sparsity >= target (ties by index); PSA_ERR_CAPACITY
 * when no candidate is that sparse.  Pure host code. */
int64_t psa_search_scratch_bytes(int n_cand, int T, int H, int W);
int psa_search_losses(const void* q, const void* k, const void* v, const psa_head_params* candidates, int n_cand,
                      const psa_problem* prob, int T, int H, int W, void* scratch, float* losses, void* stream);
int psa_search_select(const float* losses, const float* sparsity, int n, float alpha);
int psa_search_select_at_sparsity(const float* losses, const float* sparsity, int n, float target);

/* Synchronises the current device, then returns the status word the last psa_attn_fwd
 * on it left behind: PSA_OK, or PSA_ERR_TIMEOUT if a bounded wait inside the kernel
 * expired (outputs are then undefined).  *detail (optional, host) receives a
 * diagnostic code naming the wait that gave up. */
int psa_last_device_status(int32_t* detail);

/* Self-test of the bounded device-side waits (no counterpart in the paper): launches a
 * one-warp kernel that waits, with the same routine the attention kernel uses, on a barrier
 * nothing ever arrives on.  The wait gives up after limit_ms (1..1000) and the kernel
 * returns normally; psa_last_device_status() then reports PSA_ERR_TIMEOUT with detail
 * 0x7e57, and the context stays usable. */
int psa_selftest_wait_timeout(int limit_ms, void* stream);

/* Measurement hook: when both are non-NULL cudaEvent_t handles, every later psa_attn_fwd
 * records `start` on its stream just before the attention kernel and `stop` just after
 * it (the planning kernel stays outside the pair).  Pass NULL, NULL to switch it off. */
int psa_profile_events(void* start_event, void* stop_event);

/* Number of kernels the library has launched since load (all entry points). */
int64_t psa_launch_count(void);

/* Frees the per-device workspaces.  Safe to call more than once. */
int psa_shutdown(void);

const char* psa_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* PSA_H_ */
