// psa_attn_fwd for sm_100a: stripe-masked flash attention forward.
//
// One persistent CTA per SM draws work items from a global ticket; items are stored heaviest
// first (by the number of attended key blocks), head-major.  A work item is up to two query
// slabs (<= 128 rows each) of one query block (PSABlock); both slabs share the block's key
// list (GetKVBlocks, Algorithm 2), which the load warp enumerates in ascending block id straight
// from the six stripe parameters (Algorithm 1) -- no mask or index list is read from memory.
// A single-slab item runs in split-KV mode: both softmax warpgroups work on that one slab, on
// the even and the odd key slabs, and their partial results are merged in the epilogue.
//
// Roles (384 threads = 3 warpgroups):
//   warp  0    tcgen05.mma issue: S_i = Q_i K^T (SS form), O_i += P_i V (P read from TMEM).  Its
//              own instruction stream is on the critical path, so it probes two barriers per
//              shared-memory round trip and divides nothing inside the loop
//   warp  1    scheduler + TMA loads: Q slabs once per item, K and V slabs through a 5-slot ring
//              (V_j travels with K_{j+1} under one barrier)
//   warps 2-3  idle; they only exist so that the first warpgroup can hand its registers
//              to the softmax warpgroups (setmaxnreg)
//   warps 4-7  softmax / correction / epilogue of tile 0 = (S0, O0)   (TMEM lanes 0..127)
//   warps 8-11 the same for tile 1 = (S1, O1)
// TMEM (512 columns): S0 | S1 | O0 | O1, 128 fp32 columns each; the bf16 probabilities
// P_i overwrite the first columns of S_i.  A key slab has 128 keys, or 112/96/64 for the last
// slab of a block whose token count is not a multiple of 128.
// Every meeting point inside the kernel's loops is an mbarrier wait with a time limit (2 s of
// %globaltimer): producer / consumer hand-offs, the merge of a split-KV item, and the gathering
// of a staged output slab before its TMA store.  On expiry the waiter sets a CTA-wide abort
// flag; every other waiter sees the flag at its next poll and returns, all roles leave their
// loops, the load warp waits (bounded) for its TMA loads in flight, the MMA warp waits (bounded)
// for its MMAs in flight, all threads meet at the one __syncthreads of the teardown, TMEM is
// freed and the status word reports the timeout.  Not bounded by the kernel: the TMEM allocation
// at start-up, which blocks while another resident CTA holds tensor memory -- this kernel takes a
// whole SM (226 KB of shared memory, 512 TMEM columns), so a caller must not run other
// TMEM-using kernels on the same device concurrently with it.
// Build-time knob: PSA_EMU_PAIRS (share of exponentials computed by a polynomial on the FMA
// pipe, default 0).
#include <cuda.h>
#include <cuda_bf16.h>

#include "psa_common.cuh"

namespace psa {

constexpr int kThreads = 384;                       // 3 warpgroups; register budgets are re-split below
constexpr int kWarpMma = 0, kWarpLoad = 1, kUtilGroup = 0, kFirstSoftmaxWarp = 4;   // warp roles
constexpr int kNumSlots = 5;                       // K/V ring slots of one 128 x 128 bf16 slab
constexpr uint32_t kSlabBytes = 128 * 128 * 2;     // 32 KB
constexpr uint32_t kHalfBytes = kSlabBytes / 2;    // one 64-column swizzled half
// Register budgets after the re-split (setmaxnreg).  The CTA's pool is what it was launched with
// (kRegsAtLaunch per thread: the compiler's figure under the launch bound of 384 threads);
// setmaxnreg.inc blocks until the pool has room, so a split that does not fit would never start.
constexpr int kRegsAtLaunch = 168, kRegsUtil = 72, kRegsSoftmax = 216;
static_assert(128 * kRegsUtil + 256 * kRegsSoftmax <= kThreads * kRegsAtLaunch, "register re-split exceeds the CTA's pool");
constexpr int kMetaRing = 8;
constexpr float kRescaleThreshold = 8.0f;          // log2 units; lazy rescale of O
constexpr unsigned long long kTimeoutNs = 2000000000ull;

// shared memory map (offsets from a 1024-byte aligned base)
constexpr uint32_t kOffQ = 0;                                   // 2 slabs
constexpr uint32_t kOffRing = 2 * kSlabBytes;                   // kNumSlots slabs
constexpr uint32_t kOffBar = kOffRing + kNumSlots * kSlabBytes; // mbarriers
// One load barrier per ring slot: a barrier is armed again only after as many further tiles as
// there are slots have been issued, i.e. after the tiles of its previous phase were consumed
// (tiles that travel alone -- the first K and the last V of an item -- each take a barrier).
constexpr int kNumPairBars = kNumSlots;
constexpr int kBarQFull = 0, kBarQEmpty = 2, kBarPairFull = 4, kBarSlotEmpty = kBarPairFull + kNumPairBars,
              kBarSFull = kBarSlotEmpty + kNumSlots, kBarPHalf = kBarSFull + 2, kBarPReady = kBarPHalf + 2,
              kBarOFull = kBarPReady + 2, kBarOEmpty = kBarOFull + 2, kBarSchedFull = kBarOEmpty + 2,
              kBarSchedEmpty = kBarSchedFull + 2, kBarStage = kBarSchedEmpty + 2, kBarMerge = kBarStage + 2,
              kBarDrain = kBarMerge + 1, kNumBars = (kBarDrain + 1 + 1) & ~1;
constexpr uint32_t kOffMeta = kOffBar + kNumBars * 8;           // kMetaRing x 8 words
constexpr uint32_t kOffMaskT = kOffMeta + kMetaRing * 32;       // kMaxTp / 32 words
constexpr uint32_t kOffMaskS = kOffMaskT + (kMaxTp / 32) * 4;   // kMaxSp / 32 words
constexpr uint32_t kOffSched = kOffMaskS + (kMaxSp / 32) * 4;   // two published work items
constexpr uint32_t kOffMisc = kOffSched + 32;                   // tmem base, abort flag
constexpr uint32_t kOffXchg = kOffMisc + 16;                    // split-KV merge: (m, l) of 128 rows
constexpr uint32_t kSmemBytes = kOffXchg + 128 * 8;
constexpr uint32_t kSmemAlloc = kSmemBytes;                     // base alignment comes from the declaration
static_assert(kSmemAlloc <= 232448, "exceeds the 227 KB of shared memory a CTA may use");

// ----------------------------------------------------------------------------- PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false once the CTA-wide abort flag is set (by this or another
// waiter); `code` names the wait for the status word.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int code,
                                          unsigned long long limit_ns = kTimeoutNs) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  uint32_t n = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++n & 255u) == 0u) {
      if (*abort_flag != 0) return false;
      if (globaltimer_ns() - t0 > limit_ns) {
        atomicCAS((int*)abort_flag, 0, code);
        return false;
      }
    }
  }
  return true;
}
// warp-uniform variant: every lane waits, the warp agrees on the outcome
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag, int code) {
  const bool ok = mbar_wait(bar, parity, abort_flag, code);
  return __all_sync(0xffffffffu, ok);
}

// Two barriers at once: both probes are issued before either result is used, so a wait that is
// already satisfied costs one shared-memory round trip instead of two.
__device__ __forceinline__ bool mbar_wait2_warp(uint32_t bar_a, uint32_t par_a, uint32_t bar_b, uint32_t par_b,
                                                volatile int* abort_flag, int code_a, int code_b) {
  uint32_t ra, rb;
  asm volatile(
      "{\n\t.reg .pred pa, pb;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 pa, [%2], %3;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 pb, [%4], %5;\n\t"
      "selp.u32 %0, 1, 0, pa;\n\t"
      "selp.u32 %1, 1, 0, pb;\n\t}"
      : "=r"(ra), "=r"(rb) : "r"(bar_a), "r"(par_a), "r"(bar_b), "r"(par_b) : "memory");
  bool ok = true;
  if (!ra) ok = mbar_wait(bar_a, par_a, abort_flag, code_a);
  if (ok && !rb) ok = mbar_wait(bar_b, par_b, abort_flag, code_b);
  return __all_sync(0xffffffffu, ok);
}

// Waits on barrier a and, in the same shared-memory round trip, probes barrier b once;
// *b_done tells whether b's phase was already complete (warp-uniform).
__device__ __forceinline__ bool mbar_wait_probe_warp(uint32_t bar_a, uint32_t par_a, uint32_t bar_b, uint32_t par_b,
                                                     volatile int* abort_flag, int code_a, bool* b_done) {
  uint32_t ra, rb;
  asm volatile(
      "{\n\t.reg .pred pa, pb;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 pa, [%2], %3;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 pb, [%4], %5;\n\t"
      "selp.u32 %0, 1, 0, pa;\n\t"
      "selp.u32 %1, 1, 0, pb;\n\t}"
      : "=r"(ra), "=r"(rb) : "r"(bar_a), "r"(par_a), "r"(bar_b), "r"(par_b) : "memory");
  bool ok = true;
  if (!ra) ok = mbar_wait(bar_a, par_a, abort_flag, code_a);
  *b_done = __all_sync(0xffffffffu, rb != 0u);
  return __all_sync(0xffffffffu, ok);
}

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* tm, uint32_t bar,
                                            int c0, int c1, int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4) : "memory");
}
__device__ __forceinline__ void tma_store_5d(const CUtensorMap* tm, uint32_t src,
                                             int c0, int c1, int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5, %6}], [%1];"
      ::"l"(tm), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4) : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc]
__device__ __forceinline__ void tc_mma_ss(uint32_t d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc]
__device__ __forceinline__ void tc_mma_ts(uint32_t d, uint32_t a, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d), "r"(a), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t addr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(addr) : "memory");
}
__device__ __forceinline__ void tc_st32(uint32_t addr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t addr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(addr) : "memory");
}
__device__ __forceinline__ void tc_st8(uint32_t addr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
      ::"r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
      : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t addr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// packed fp32 pairs (one instruction for two lanes of work on sm_100)
__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
// 2^x for a pair on the FMA/ALU pipes: x = n + f with n = rint(x), f in [-0.5, 0.5];
// 2^f by a cubic (relative error < 8e-5, far below the bf16 rounding of the result), and
// 2^n by adding n to the exponent field.  x is clamped at -125 so the exponent cannot wrap.
__device__ __forceinline__ void exp2_poly_pair(uint64_t x2, float& p0, float& p1) {
  float x0, x1;
  unpack2(x2, x0, x1);
  x0 = fmaxf(x0, -125.f);
  x1 = fmaxf(x1, -125.f);
  const uint64_t xc = pack2(x0, x1);
  const uint64_t magic = pack2(12582912.f, 12582912.f);       // 1.5 * 2^23: rounds to integer
  const uint64_t t2 = add2(xc, magic);
  const uint64_t n2 = add2(t2, pack2(-12582912.f, -12582912.f));
  const uint64_t f2 = fma2(n2, pack2(-1.f, -1.f), xc);
  uint64_t q2 = fma2(f2, pack2(0.05508868396282196f, 0.05508868396282196f), pack2(0.24260404706001282f, 0.24260404706001282f));
  q2 = fma2(q2, f2, pack2(0.6932762265205383f, 0.6932762265205383f));
  q2 = fma2(q2, f2, pack2(0.9999289512634277f, 0.9999289512634277f));
  float q0, q1, t0, t1;
  unpack2(q2, q0, q1);
  unpack2(t2, t0, t1);
  p0 = __int_as_float(__float_as_int(q0) + (__float_as_int(t0) << 23));
  p1 = __int_as_float(__float_as_int(q1) + (__float_as_int(t1) << 23));
}
#ifndef PSA_EMU_PAIRS
#define PSA_EMU_PAIRS 0   // of every 4 pairs of probabilities, this many use exp2_poly_pair (0: all ex2.approx)
#endif


__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N columns (multiple of 16); A is K-major.
__host__ __device__ constexpr uint32_t instr_desc(bool b_mn_major, uint32_t n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}
// One elected lane of a converged warp (keeps the branch warp-uniform for the compiler).
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
  return pred != 0;
}

// Checked build (-DPSA_DEBUG_CHECKS; the stand-in for a memory checker): every global store index,
// TMA coordinate, ring / table index and TMEM column range computed by the kernel is verified before
// use.  A violation records PSA_ERR_INTERNAL with a code naming the site in the status word and the
// access is skipped -- nothing traps.  In the regular build the checks compile to `true`.
#ifdef PSA_DEBUG_CHECKS
__device__ __noinline__ bool dbg_fail(int* ws_header, int code) {
  if (atomicCAS(ws_header + kWsStatus, 0, (int)PSA_ERR_INTERNAL) == 0) ws_header[kWsDetail] = code;
  return false;
}
#define PSA_CHECKED(cond, code) ((cond) ? true : dbg_fail(prm.ws_header, (code)))
#else
#define PSA_CHECKED(cond, code) true
#endif

// ----------------------------------------------------------------------------- planning
// Work order: per head, query blocks ranked by attended key-block count (largest first),
// heads kept together so that concurrently running CTAs share K/V in L2.
__global__ void __launch_bounds__(256)
plan_kernel(const HeadParamsArray hp, const Geom g, int head0, int clear_status, int* __restrict__ ws_header,
            psa_head_params* __restrict__ hp_dev, WorkItem* __restrict__ items) {
  extern __shared__ int sm[];  // cntT[Tp], cntS[Sp], cnt[NB]
  int* cntT = sm;
  int* cntS = sm + g.Tp;
  int* cnt = cntS + g.Sp;
  const int h = blockIdx.x;
  const psa_head_params p = hp.p[head0 + h];
  // The scheduler ticket restarts with every launch; the status words are cleared only by the
  // first launch of an API call, so that a timeout recorded by an earlier launch of the same call
  // (a call may need several: more than 128 heads, chunks of a host-tensor call) survives.
  if (h == 0 && threadIdx.x < kWsHeaderWords && (clear_status || (threadIdx.x != kWsStatus && threadIdx.x != kWsDetail)))
    ws_header[threadIdx.x] = 0;
  if (threadIdx.x == 0) hp_dev[h] = p;
  for (int a = threadIdx.x; a < g.Tp + g.Sp; a += blockDim.x) {
    int c = 0;
    if (a < g.Tp) {
      for (int k = 0; k < g.Tp; ++k) c += axis_attends(k - a, p.Tw, p.To, p.Ts);
    } else {
      for (int k = 0; k < g.Sp; ++k) c += axis_attends(k - (a - g.Tp), p.Sw, p.So, p.Ss);
    }
    sm[a] = c;
  }
  __syncthreads();
  for (int qb = threadIdx.x; qb < g.NB; qb += blockDim.x) cnt[qb] = cntT[qb / g.Sp] * cntS[qb % g.Sp];
  __syncthreads();
  const int ipb = g.items_per_block;
  // Text-query items first: they attend every key block, so they are the heaviest of the head.
  // Two text slabs per item; a single one runs in split-KV mode.  Flag in bit 25.
  WorkItem* head_items = items + (size_t)h * g.items_per_head;
  for (int it = threadIdx.x; it < g.n_titems; it += blockDim.x) {
    const int sub0 = 2 * it;
    const int nq = (g.n_ts - sub0) >= 2 ? 2 : 1;
    head_items[it] = make_int4(h, 0, g.NB, sub0 | (nq << 16) | ((nq == 1 ? 1 : 0) << 24) | (1 << 25));
  }
  WorkItem* out = head_items + g.n_titems;
  for (int qb = threadIdx.x; qb < g.NB; qb += blockDim.x) {
    const int c = cnt[qb];
    int rank = 0;
    for (int j = 0; j < g.NB; ++j) {
      const int cj = cnt[j];
      rank += (cj > c) || (cj == c && j < qb);
    }
    // two-slab items first (heavier), then the odd single-slab items, each in rank order
    int pos = rank;
    for (int it = 0; it < ipb; ++it) {
      const int sub0 = 2 * it;
      const int nq = (g.n_sub - sub0) >= 2 ? 2 : 1;
      // A single-slab item runs in split-KV mode: both softmax warpgroups work on that one
      // query slab, one on the even and one on the odd key slabs (flag in bit 24).
      out[(size_t)it * g.NB + pos] = make_int4(h, qb, c, sub0 | (nq << 16) | ((nq == 1 ? 1 : 0) << 24));
    }
  }
}

// ----------------------------------------------------------------------------- attention
struct AttnParams {
  Geom g;
  const WorkItem* items;
  const psa_head_params* hp_dev;
  int* ws_header;
  float* lse;     // already offset to the first head of this launch
  int n_items;
  int shared_qkv; // 1: every head reads head 0 of q, k, v (candidate masks of one head, PSA-Search)
};

struct TensorMaps {
  CUtensorMap q[3], k[3], v[3], o[3];  // [0]: full 128-token slab box, [1]: a block's last slab, [2]: text slab
};

// Extents and token count of slab `sub` of a block; `last` selects the tensor-map set.
__device__ __forceinline__ void slab_shape(const Geom& g, int sub, int& et, int& eh, int& ew, int& ntok, int& last) {
  last = (sub == g.n_sub - 1) ? 1 : 0;
  et = g.ct; eh = g.ch; ew = g.cw;
  if (last) {
    if (g.sub_axis == 0) et = g.c_last;
    else if (g.sub_axis == 1) eh = g.c_last;
    else ew = g.c_last;
  }
  ntok = last ? g.n_last : kSlabTokens;
}

__device__ __forceinline__ void slab_origin(const Geom& g, int qb, int sub, int& t0, int& h0, int& w0) {
  const int tb = qb / g.Sp, sb = qb % g.Sp;
  t0 = tb * g.bt;
  h0 = (sb / g.Wp) * g.bh;
  w0 = (sb % g.Wp) * g.bw;
  if (g.sub_axis == 0) t0 += sub * g.ct;
  else if (g.sub_axis == 1) h0 += sub * g.ch;
  else w0 += sub * g.cw;
}

// Descriptor halves.  Only the low word (start address, leading byte offset) changes
// between MMAs; the high word (stride byte offset 1024, version, 128-byte swizzle) is fixed.
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr, uint32_t lbo_bytes) {
  return ((addr >> 4) & 0x3FFFu) | ((lbo_bytes >> 4) << 16);
}
__device__ __forceinline__ uint64_t make_desc(uint32_t lo) { return ((uint64_t)kDescHi << 32) | lo; }

// Online-softmax step of one query row (one thread) for one key slab of NK keys.
//   tS: TMEM address of the row's scores (fp32, NK columns); the bf16 probabilities are written
//       back over the first NK/2 columns.  tO: the row's output accumulator (128 fp32 columns).
//   meta: validity bits of the slab's keys (bit c of word c/32); all ones when nothing is padded.
//   m_ref / l: running reference maximum (scaled log2 domain) and running sum.
// The reference maximum is lazy: it moves only when the slab's maximum exceeds it by more than
// kRescaleThreshold, so exponentials stay below 2^threshold and O is rarely rescaled.
template <int NK>
__device__ __forceinline__ void softmax_slab(uint32_t tS, uint32_t tO, const uint4 meta, bool first,
                                             float scale_log2, float& m_ref, float& l, uint32_t bar_half,
                                             uint32_t bar_ready) {
  constexpr int NFULL = NK / 32, REM = NK % 32;
  static_assert(NK % 16 == 0 && NK >= 64 && NK <= 128 && (REM == 0 || REM == 16), "unsupported slab width");
  const float neg_inf = __int_as_float(0xff800000);
  uint32_t s[NK];  // raw scores of this row (fp32 bit patterns), kept in registers
#pragma unroll
  for (int c4 = 0; c4 < NFULL; ++c4) tc_ld32(tS + c4 * 32, s + c4 * 32);
  if (REM) tc_ld16(tS + NFULL * 32, s + NFULL * 32);
  tc_wait_ld();
  if ((meta.x & meta.y & meta.z & meta.w) != 0xffffffffu) {  // 3D-padding: padded key positions score -inf
    const uint32_t v[4] = {meta.x, meta.y, meta.z, meta.w};
#pragma unroll
    for (int c = 0; c < NK; ++c)
      if (!((v[c >> 5] >> (c & 31)) & 1u)) s[c] = 0xff800000u;
  }
  // eight independent chains (NK is a multiple of 16): shorter dependency depth
  float a[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) a[i] = fmaxf(__uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1]));
#pragma unroll
  for (int c = 16; c < NK; c += 16) {
#pragma unroll
    for (int i = 0; i < 8; ++i) a[i] = max3(a[i], __uint_as_float(s[c + 2 * i]), __uint_as_float(s[c + 2 * i + 1]));
  }
  const float ms = fmaxf(fmaxf(max3(a[0], a[1], a[2]), max3(a[3], a[4], a[5])), fmaxf(a[6], a[7])) * scale_log2;
  if (first) {
    m_ref = ms;  // first slab of the item: nothing accumulated yet
  } else {
    float alpha = 1.f;
    const bool grow = ms > m_ref + kRescaleThreshold;  // also true when m_ref == -inf
    if (grow) {
      alpha = fast_exp2(m_ref - ms);  // 0 when m_ref == -inf
      m_ref = ms;
    }
    if (__any_sync(0xffffffffu, grow)) {
      l *= alpha;
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) {
        uint32_t o[32];
        tc_ld32(tO + c4 * 32, o);
        tc_wait_ld();
#pragma unroll
        for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
        tc_st32(tO + c4 * 32, o);
      }
    }
  }
  const float m_use = (m_ref == neg_inf) ? 0.f : m_ref;
  const uint64_t sc2 = pack2(scale_log2, scale_log2), negm2 = pack2(-m_use, -m_use);
  uint64_t sum2 = pack2(0.f, 0.f);
  // probabilities exp2(scale*s - m_use), bf16, written over the scores in chunks of 32 keys
  auto exp_chunk = [&](int base, int npairs, uint32_t* pk) {
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      if (c >= npairs) break;
      const uint64_t x2 = fma2(pack2(__uint_as_float(s[base + 2 * c]), __uint_as_float(s[base + 2 * c + 1])), sc2, negm2);
      float p0, p1;
      if ((c & 3) < PSA_EMU_PAIRS) {
        exp2_poly_pair(x2, p0, p1);
      } else {
        float x0, x1;
        unpack2(x2, x0, x1);
        p0 = fast_exp2(x0);
        p1 = fast_exp2(x1);
      }
      sum2 = add2(sum2, pack2(p0, p1));
      pk[c] = pack_bf16(p0, p1);
    }
  };
#pragma unroll
  for (int c4 = 0; c4 < NFULL; ++c4) {
    uint32_t pk[16];
    exp_chunk(c4 * 32, 16, pk);
    tc_st16(tS + c4 * 16, pk);
    if (c4 == 1) {  // the first 64 keys are final: their P V MMAs may start
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(bar_half);
    }
  }
  if (REM) {
    uint32_t pk[16];
    exp_chunk(NFULL * 32, 8, pk);
    tc_st8(tS + NFULL * 16, pk);
  }
  float sum0, sum1;
  unpack2(sum2, sum0, sum1);
  l += sum0 + sum1;
  tc_wait_st();
  tc_fence_before();
  mbar_arrive(bar_ready);
}

__global__ void __launch_bounds__(kThreads, 1)
attn_fwd_kernel(const __grid_constant__ TensorMaps tms, const AttnParams prm) {
  // 128-byte swizzled slabs need a 1024-byte aligned base; the declaration asks for it and the
  // kernel checks it (a misaligned base is reported through the status word, no work is done).
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = smem_raw;
  const uint32_t sbase = smem_u32(smem);
  const Geom& g = prm.g;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  auto bar = [&](int idx) -> uint32_t { return sbase + kOffBar + 8u * (uint32_t)idx; };
  uint32_t* meta = reinterpret_cast<uint32_t*>(smem + kOffMeta);
  uint32_t* maskT = reinterpret_cast<uint32_t*>(smem + kOffMaskT);
  uint32_t* maskS = reinterpret_cast<uint32_t*>(smem + kOffMaskS);
  volatile int4* sched = reinterpret_cast<volatile int4*>(smem + kOffSched);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kOffMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffMisc + 4);

  // A short query slab leaves its last rows of the Q buffer unwritten; keep them finite.
  for (uint32_t off = threadIdx.x * 16u; off < 2u * kSlabBytes; off += kThreads * 16u)
    *reinterpret_cast<uint4*>(smem + kOffQ + off) = make_uint4(0u, 0u, 0u, 0u);
  fence_async_smem();
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(kBarQFull + i), 1);
      mbar_init(bar(kBarQEmpty + i), 1);
      mbar_init(bar(kBarSFull + i), 1);
      mbar_init(bar(kBarPHalf + i), 128);
      mbar_init(bar(kBarPReady + i), 128);
      mbar_init(bar(kBarOFull + i), 1);
      mbar_init(bar(kBarOEmpty + i), 128);
      mbar_init(bar(kBarStage + i), 128);
      mbar_init(bar(kBarSchedFull + i), 1);
      mbar_init(bar(kBarSchedEmpty + i), 9);  // the MMA warp and the eight softmax warps
    }
    mbar_init(bar(kBarMerge), 128);
    mbar_init(bar(kBarDrain), 1);
    for (int s = 0; s < kNumPairBars; ++s) mbar_init(bar(kBarPairFull + s), 1);
    for (int s = 0; s < kNumSlots; ++s) mbar_init(bar(kBarSlotEmpty + s), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kWarpMma) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + kOffMisc), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // The CTA owns all 512 TMEM columns, so the allocation starts at column 0, lane 0; using
  // the constant keeps every TMEM address of the MMA stream in uniform registers.  Checked:
  // any other base is reported through the status word and the CTA does no work.
  constexpr uint32_t tmem = 0u;
  const bool tmem_ok = (*tmem_slot == 0u) && ((sbase & 1023u) == 0u);
  if (!tmem_ok && threadIdx.x == 0) atomicCAS((int*)abort_flag, 0, (*tmem_slot == 0u) ? 0x501 : 0x500);

  // Work items are handed out through a two-entry ring: the load warp draws a ticket from
  // a global counter (items are stored heaviest first), publishes the item, and the other
  // roles pick it up.  A negative head ends the kernel.
  auto next_item = [&](uint32_t n, WorkItem& wi) -> bool {
    const uint32_t slot = n & 1u;
    if (!tmem_ok) return false;
    if (!mbar_wait_warp(bar(kBarSchedFull + slot), (n >> 1) & 1u, abort_flag, 0x400)) return false;
    // broadcast from lane 0 so that the compiler knows the item (and every loop bound
    // derived from it) is warp-uniform
    wi.x = __shfl_sync(0xffffffffu, sched[slot].x, 0);
    wi.y = __shfl_sync(0xffffffffu, sched[slot].y, 0);
    wi.z = __shfl_sync(0xffffffffu, sched[slot].z, 0);
    wi.w = __shfl_sync(0xffffffffu, sched[slot].w, 0);
    __syncwarp();
    if (lane == 0) mbar_arrive(bar(kBarSchedEmpty + slot));
    return wi.x >= 0;
  };

  if ((warp >> 2) == kUtilGroup) {
  // Utility warpgroup: give registers away (the budget is re-split per warpgroup).
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsUtil));
  if (warp == kWarpLoad) {
    // ======================================================================= load warp
    // Ring tiles are issued in the order K_0, V_0, K_1, V_1, ...; the MMA warp needs V_j and
    // K_{j+1} at the same moment, so those two travel under one "pair" barrier
    // (K_0 and the last V of an item travel alone).
    uint32_t tile_g = 0;       // ring tiles issued so far
    uint32_t pair_g = 0;       // pair barriers armed so far
    uint32_t kv_g = 0;         // key slabs issued so far
    uint32_t it_q0 = 0, it_q1 = 0; // items in which query slab i was active
    bool ok = tmem_ok;
    for (uint32_t n = 0; ok; ++n) {
      const uint32_t sslot = n & 1u;
      ok = mbar_wait_warp(bar(kBarSchedEmpty + sslot), ((n >> 1) & 1u) ^ 1u, abort_flag, 0x401);
      if (!ok) break;
      WorkItem wi = make_int4(-1, 0, 0, 0);
      if (lane == 0) {
        const int ticket = atomicAdd(prm.ws_header + kWsCounter, 1);
        if (ticket < prm.n_items) wi = prm.items[ticket];
        sched[sslot].x = wi.x; sched[sslot].y = wi.y; sched[sslot].z = wi.z; sched[sslot].w = wi.w;
        mbar_arrive(bar(kBarSchedFull + sslot));
      }
      wi.x = __shfl_sync(0xffffffffu, wi.x, 0);
      wi.y = __shfl_sync(0xffffffffu, wi.y, 0);
      wi.w = __shfl_sync(0xffffffffu, wi.w, 0);
      if (wi.x < 0) break;
      const int head = wi.x, qb = wi.y, sub0 = wi.w & 0xffff, nq = (wi.w >> 16) & 0xff;
      if (!PSA_CHECKED(head < g.n_heads && qb >= 0 && qb <= g.NB && nq >= 1 && nq <= 2 &&
                       sub0 + nq <= ((wi.w >> 25) & 1 ? g.n_ts : g.n_sub), 0xD04)) {
        if (lane == 0) atomicCAS((int*)abort_flag, 0, 0xD04);   // a malformed item: stop this CTA through the abort path
        ok = false;
        break;
      }
      const int lag = ((wi.w >> 24) & 1) ? 2 : 1;   // V_j travels with K_{j+lag} (2 in split-KV mode)
      const bool textq = ((wi.w >> 25) & 1) != 0;   // the queries are text tokens: every key is attended
      const int head_ld = prm.shared_qkv ? 0 : head;   // head coordinate of the q, k, v loads
      const psa_head_params p = prm.hp_dev[head];
      const int tq = qb / g.Sp, sq = qb % g.Sp;
      // attended key-block coordinates of this query block, one bit per block coordinate
      for (int b = 0; b < g.Tp; b += 32) {
        const int tk = b + lane;
        const unsigned m = __ballot_sync(0xffffffffu, tk < g.Tp && (textq || axis_attends(tk - tq, p.Tw, p.To, p.Ts)));
        if (lane == 0) maskT[b >> 5] = m;
      }
      for (int b = 0; b < g.Sp; b += 32) {
        const int sk = b + lane;
        const unsigned m = __ballot_sync(0xffffffffu, sk < g.Sp && (textq || axis_attends(sk - sq, p.Sw, p.So, p.Ss)));
        if (lane == 0) maskS[b >> 5] = m;
      }
      __syncwarp();
      // query slabs
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        if (i >= nq) break;
        const uint32_t itq = i == 0 ? it_q0 : it_q1;
        ok = mbar_wait_warp(bar(kBarQEmpty + i), (itq & 1u) ^ 1u, abort_flag, 0x100 + i);
        if (!ok) break;
        if (lane == 0) {
          int t0, h0, w0, et, eh, ew, ntok, last;
          if (textq) {   // text slab: 128 tokens from the text map, token index in the second coordinate
            t0 = 0; h0 = 0; w0 = (sub0 + i) * kSlabTokens; ntok = kSlabTokens; last = 2;
          } else {
            slab_origin(g, qb, sub0 + i, t0, h0, w0);
            slab_shape(g, sub0 + i, et, eh, ew, ntok, last);
          }
          const uint32_t dst = sbase + kOffQ + (uint32_t)i * kSlabBytes;
          if (PSA_CHECKED(w0 >= 0 && h0 >= 0 && t0 >= 0 && head_ld >= 0 && head_ld < g.n_heads && last >= 0 && last <= 2 &&
                          ntok > 0 && ntok <= kSlabTokens &&
                          (textq || (w0 < g.Wp * g.bw && h0 < g.Hp * g.bh && t0 < g.Tp * g.bt)), 0xD01)) {   // inside the padded grid
            mbar_expect_tx(bar(kBarQFull + i), (uint32_t)ntok * 256u);
            tma_load_5d(dst, &tms.q[last], bar(kBarQFull + i), 0, w0, h0, t0, head_ld);
            tma_load_5d(dst + kHalfBytes, &tms.q[last], bar(kBarQFull + i), 64, w0, h0, t0, head_ld);
          }
        }
        if (i == 0) ++it_q0; else ++it_q1;
      }
      if (!ok) break;
      // key / value slabs in ascending key-block id.  Up to `lag` slabs wait for their V load.
      int npend = 0;
      int at0 = 0, ah0 = 0, aw0 = 0, alast = 0, antok = kSlabTokens;  // oldest pending slab
      int bt0 = 0, bh0 = 0, bw0 = 0, blast = 0, bntok = kSlabTokens;  // newer pending slab (lag 2)
      // One key slab: K now, V of the slab issued `lag` slabs earlier under the same barrier.
      auto issue_slab = [&](int t0, int h0, int w0, int last, int ntok, uint32_t vw0, uint32_t vw1, uint32_t vw2,
                            uint32_t vw3) {
        // slots: [V of the oldest pending slab,] K of this slab
        const bool with_v = (npend == lag);
        const uint32_t v_slot = tile_g % kNumSlots, v_use = tile_g / kNumSlots;
        const uint32_t k_tile = tile_g + (with_v ? 1u : 0u);
        const uint32_t k_slot = k_tile % kNumSlots, k_use = k_tile / kNumSlots;
        if (with_v) {
          ok = mbar_wait_warp(bar(kBarSlotEmpty + v_slot), (v_use & 1u) ^ 1u, abort_flag, 0x111);
          if (!ok) return;
        }
        ok = mbar_wait_warp(bar(kBarSlotEmpty + k_slot), (k_use & 1u) ^ 1u, abort_flag, 0x110);
        if (!ok) return;
        if (lane == 0 && PSA_CHECKED(v_slot < (uint32_t)kNumSlots && k_slot < (uint32_t)kNumSlots && t0 >= 0 && h0 >= 0 && w0 >= 0 &&
                                     last >= 0 && last <= 2 && ntok > 0 && ntok <= kSlabTokens &&
                                     (!with_v || (at0 >= 0 && ah0 >= 0 && aw0 >= 0 && alast >= 0 && alast <= 2)), 0xD02)) {
          uint32_t* m = meta + (kv_g % kMetaRing) * 8;
          m[0] = vw0; m[1] = vw1; m[2] = vw2; m[3] = vw3;
          const uint32_t pb = bar(kBarPairFull + pair_g % kNumPairBars);
          mbar_expect_tx(pb, (uint32_t)((with_v ? antok : 0) + ntok) * 256u);
          if (with_v) {
            const uint32_t dv = sbase + kOffRing + v_slot * kSlabBytes;
            tma_load_5d(dv, &tms.v[alast], pb, 0, aw0, ah0, at0, head_ld);
            tma_load_5d(dv + kHalfBytes, &tms.v[alast], pb, 64, aw0, ah0, at0, head_ld);
          }
          const uint32_t dk = sbase + kOffRing + k_slot * kSlabBytes;
          tma_load_5d(dk, &tms.k[last], pb, 0, w0, h0, t0, head_ld);
          tma_load_5d(dk + kHalfBytes, &tms.k[last], pb, 64, w0, h0, t0, head_ld);
        }
        tile_g = k_tile + 1;
        ++pair_g;
        ++kv_g;
        // queue this slab's V
        if (with_v) {
          if (lag == 2) { at0 = bt0; ah0 = bh0; aw0 = bw0; alast = blast; antok = bntok; }
          --npend;
        }
        if (npend == 0) { at0 = t0; ah0 = h0; aw0 = w0; alast = last; antok = ntok; }
        else { bt0 = t0; bh0 = h0; bw0 = w0; blast = last; bntok = ntok; }
        ++npend;
      };
      for (int tw = 0; ok && tw < g.Tp; tw += 32) {
        uint32_t mt = maskT[tw >> 5];
        while (ok && mt) {
          const int tk = tw + __ffs(mt) - 1;
          mt &= mt - 1;
          for (int sw = 0; ok && sw < g.Sp; sw += 32) {
            uint32_t ms = maskS[sw >> 5];
            while (ok && ms) {
              const int sk = sw + __ffs(ms) - 1;
              ms &= ms - 1;
              const int kb = tk * g.Sp + sk;
              for (int sub = 0; ok && sub < g.n_sub; ++sub) {
                int t0, h0, w0, et, eh, ew, ntok, last;
                slab_origin(g, kb, sub, t0, h0, w0);
                slab_shape(g, sub, et, eh, ew, ntok, last);
                // validity of the slab's key positions (3D-padding): bit c of word c/32
                const bool edge = (t0 + et > g.T) || (h0 + eh > g.H) || (w0 + ew > g.W);
                uint32_t vw0 = 0xffffffffu, vw1 = 0xffffffffu, vw2 = 0xffffffffu, vw3 = 0xffffffffu;
                if (edge) {
                  const int ehw = ew * eh;
                  int c = lane;
                  vw0 = __ballot_sync(0xffffffffu, (t0 + c / ehw < g.T) && (h0 + (c / ew) % eh < g.H) && (w0 + c % ew < g.W));
                  c += 32;
                  vw1 = __ballot_sync(0xffffffffu, (t0 + c / ehw < g.T) && (h0 + (c / ew) % eh < g.H) && (w0 + c % ew < g.W));
                  c += 32;
                  vw2 = __ballot_sync(0xffffffffu, (t0 + c / ehw < g.T) && (h0 + (c / ew) % eh < g.H) && (w0 + c % ew < g.W));
                  c += 32;
                  vw3 = __ballot_sync(0xffffffffu, (t0 + c / ehw < g.T) && (h0 + (c / ew) % eh < g.H) && (w0 + c % ew < g.W));
                }
                issue_slab(t0, h0, w0, last, ntok, vw0, vw1, vw2, vw3);
              }
            }
          }
        }
      }
      // text key slabs: attended by every query; tokens beyond n_text are zero-filled and masked
      for (int ts = 0; ok && ts < g.n_ts; ++ts) {
        const int tok0 = ts * kSlabTokens;
        const int nvalid = g.n_text - tok0;   // >= 1
        const uint32_t vw0 = nvalid >= 32 ? 0xffffffffu : ((1u << nvalid) - 1u);
        const uint32_t vw1 = nvalid >= 64 ? 0xffffffffu : (nvalid <= 32 ? 0u : ((1u << (nvalid - 32)) - 1u));
        const uint32_t vw2 = nvalid >= 96 ? 0xffffffffu : (nvalid <= 64 ? 0u : ((1u << (nvalid - 64)) - 1u));
        const uint32_t vw3 = nvalid >= 128 ? 0xffffffffu : (nvalid <= 96 ? 0u : ((1u << (nvalid - 96)) - 1u));
        issue_slab(0, 0, tok0, 2, kSlabTokens, vw0, vw1, vw2, vw3);
      }
      while (ok && npend > 0) {  // V of the item's last slab(s), one pair barrier each
        const uint32_t v_slot = tile_g % kNumSlots, v_use = tile_g / kNumSlots;
        ok = mbar_wait_warp(bar(kBarSlotEmpty + v_slot), (v_use & 1u) ^ 1u, abort_flag, 0x112);
        if (!ok) break;
        if (lane == 0 && PSA_CHECKED(v_slot < (uint32_t)kNumSlots && at0 >= 0 && ah0 >= 0 && aw0 >= 0 && alast >= 0 && alast <= 2 &&
                                     antok > 0 && antok <= kSlabTokens, 0xD03)) {
          const uint32_t pb = bar(kBarPairFull + pair_g % kNumPairBars);
          mbar_expect_tx(pb, (uint32_t)antok * 256u);
          const uint32_t dv = sbase + kOffRing + v_slot * kSlabBytes;
          tma_load_5d(dv, &tms.v[alast], pb, 0, aw0, ah0, at0, head_ld);
          tma_load_5d(dv + kHalfBytes, &tms.v[alast], pb, 64, aw0, ah0, at0, head_ld);
        }
        ++tile_g;
        ++pair_g;
        at0 = bt0; ah0 = bh0; aw0 = bw0; alast = blast; antok = bntok;
        --npend;
      }
      if (!ok) break;
    }
    // Let every load that was issued land before the CTA retires: wait for the last armed
    // phase of each pair barrier and of the Q barriers (bounded; the abort flag no longer
    // cuts these short).
    if (lane == 0) {
      for (uint32_t back = 0; back < (uint32_t)kNumPairBars && back < pair_g; ++back) {
        const uint32_t pg = pair_g - 1 - back;
        const unsigned long long t0 = globaltimer_ns();
        while (!mbar_try_wait(bar(kBarPairFull + pg % kNumPairBars), (pg / kNumPairBars) & 1u)) {
          if (globaltimer_ns() - t0 > kTimeoutNs) break;
        }
      }
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const uint32_t itq = i == 0 ? it_q0 : it_q1;
        if (itq == 0) continue;
        const unsigned long long t0 = globaltimer_ns();
        while (!mbar_try_wait(bar(kBarQFull + i), (itq - 1) & 1u)) {
          if (globaltimer_ns() - t0 > kTimeoutNs) break;
        }
      }
    }
    __syncwarp();
  } else if (warp == kWarpMma) {
    // ======================================================================= MMA warp
    constexpr uint32_t kIdescPV = instr_desc(true, 128);  // N = head_dim
    // ring slot of the next tile and pair barrier of the next arrival: wrapping index + phase bit
    uint32_t slot_i = 0, pair_i = 0, pair_ph = 0;
    auto slot_next = [&](uint32_t sl) -> uint32_t { return sl + 1u == (uint32_t)kNumSlots ? 0u : sl + 1u; };
    auto pair_adv = [&]() { if (++pair_i == (uint32_t)kNumPairBars) { pair_i = 0; pair_ph ^= 1u; } };
    uint32_t it_q0 = 0, it_q1 = 0;
    uint32_t cnt_s0 = 0, cnt_s1 = 0;  // P_i tiles consumed so far
    bool ok = true;
    const uint32_t q_lo = desc_lo(sbase + kOffQ, 16);
    const uint32_t ring_lo_k = desc_lo(sbase + kOffRing, 16);
    const uint32_t ring_lo_v = desc_lo(sbase + kOffRing, kHalfBytes);
    constexpr uint32_t kSlabStep = kSlabBytes >> 4;  // descriptor address units per slab

    // S_i = Q_i K^T over head_dim = 128: 8 MMAs of K = 16; both operands K-major, SW128.
    // nk = keys of the slab (N of the instruction): 128, or fewer for a block's last slab.
    // iq: Q buffer; it: S tile written (they differ only in split-KV items).
    auto issue_qk = [&](int iq, uint32_t kslot, int nk, int it) {
      if (!PSA_CHECKED(iq >= 0 && iq < 2 && it >= 0 && it < 2 && kslot < (uint32_t)kNumSlots && nk >= 16 && nk <= 128 && (nk & 15) == 0, 0xD20))
        return;
      const uint32_t a0 = q_lo + (uint32_t)iq * kSlabStep, b0 = ring_lo_k + kslot * kSlabStep;
      const uint32_t idesc = instr_desc(false, (uint32_t)nk);
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        const uint32_t off = (uint32_t)(kk >> 2) * (kHalfBytes >> 4) + (uint32_t)(kk & 3) * 2u;
        tc_mma_ss(tmem + (uint32_t)it * 128u, make_desc(a0 + off), make_desc(b0 + off), idesc, kk > 0 ? 1u : 0u);
      }
    };
    // O_i (+)= P_i V over 128 keys: 8 MMAs of K = 16; A = bf16 P in TMEM (8 columns per
    // step), B = V slab as loaded (keys x head_dim, head_dim contiguous) = MN-major SW128:
    // 16 keys advance 2048 bytes, the second 64 columns of head_dim sit one half slab
    // further (leading byte offset).
    auto issue_pv_half = [&](int i, uint32_t vslot, int half, bool accumulate, int nk) {
      if (!PSA_CHECKED(i >= 0 && i < 2 && half >= 0 && half < 2 && vslot < (uint32_t)kNumSlots && nk >= 16 && nk <= 128, 0xD21)) return;
      const uint32_t b0 = ring_lo_v + vslot * kSlabStep;
#pragma unroll
      for (int k4 = 0; k4 < 4; ++k4) {
        const int kk = half * 4 + k4;
        if (kk * 16 >= nk) break;   // a short slab has fewer 16-key steps
        tc_mma_ts(tmem + 256u + (uint32_t)i * 128u, tmem + (uint32_t)i * 128u + (uint32_t)kk * 8u,
                  make_desc(b0 + (uint32_t)kk * (2048u >> 4)), kIdescPV, (accumulate || kk > 0) ? 1u : 0u);
      }
    };

    uint32_t it_o0 = 0, it_o1 = 0;    // items in which accumulator O_i was used
    // keys of a slab from its index within its block (r = j mod n_sub, carried along: no division)
    const int r_last = g.n_sub - 1;
    auto nk_at = [&](int r) -> int { return r == r_last ? g.n_last : kSlabTokens; };
    auto r_inc = [&](int r) -> int { return r == r_last ? 0 : r + 1; };

    for (uint32_t n = 0; ok; ++n) {
      WorkItem wi;
      if (!next_item(n, wi)) break;
      const int nq = (wi.w >> 16) & 0xff;
      const bool split = ((wi.w >> 24) & 1) != 0;
      const int n_vid = wi.z * g.n_sub;          // video key slabs, then the text slabs (always 128 wide)
      const int n_kv = n_vid + g.n_ts;
      auto nk_j = [&](int j, int r) -> int { return j >= n_vid ? kSlabTokens : nk_at(r); };
      // which accumulators this item uses: both for a two-slab item, and for a split-KV item
      // with at least two key slabs (even slabs -> O_0, odd slabs -> O_1)
      const bool use_o1 = (nq > 1) || (split && n_kv > 1);
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        if (i < nq) {
          const uint32_t itq = i == 0 ? it_q0 : it_q1;
          ok = mbar_wait_warp(bar(kBarQFull + i), itq & 1u, abort_flag, 0x200 + i);
          if (!ok) break;
        }
        if (i == 0 || use_o1) {
          // the epilogue of the previous item must have drained O_i before it is overwritten
          const uint32_t ito = i == 0 ? it_o0 : it_o1;
          ok = mbar_wait_warp(bar(kBarOEmpty + i), (ito & 1u) ^ 1u, abort_flag, 0x202 + i);
          if (!ok) break;
        }
      }
      if (!ok) break;
      if (n_kv > 0 && split) {
        // ---- split-KV item: one query slab (Q buffer 0); key slab j feeds tile (j & 1).
        // Ring order (see the load warp): K_0, K_1, (V_0, K_2), (V_1, K_3), ..., V_{n-2}, V_{n-1}.
        int r0 = 0;   // residue of the slab whose scores are issued next
        for (int j = 0; ok && j < 2 && j < n_kv; ++j) {
          ok = mbar_wait_warp(bar(kBarPairFull + pair_i), pair_ph, abort_flag, 0x230);
          if (!ok) break;
          pair_adv();
          const uint32_t slot = slot_i;
          slot_i = slot_next(slot_i);
          tc_fence_after();
          if (elect_one()) {
            issue_qk(0, slot, nk_j(j, r0), j);
            tc_commit(bar(kBarSFull + j));
            tc_commit(bar(kBarSlotEmpty + slot));
          }
          __syncwarp();
          r0 = r_inc(r0);
        }
        int rj = 0;   // residue of slab j; r0 is that of slab j + 2 from here on
        for (int j = 0; ok && j < n_kv; ++j) {
          const int i = j & 1;
          const uint32_t cs = i == 0 ? cnt_s0 : cnt_s1;
          ok = mbar_wait2_warp(bar(kBarPairFull + pair_i), pair_ph, bar(kBarPHalf + i), cs & 1u, abort_flag, 0x231, 0x234 + i);
          if (!ok) break;
          pair_adv();
          const bool more = (j + 2 < n_kv);
          const uint32_t vslot = slot_i;
          const uint32_t kslot = slot_next(slot_i);
          slot_i = more ? slot_next(kslot) : kslot;
          const int nk_cur = nk_j(j, rj);
          rj = r_inc(rj);
          tc_fence_after();
          if (elect_one()) issue_pv_half(i, vslot, 0, j > 1, nk_cur);
          ok = mbar_wait_warp(bar(kBarPReady + i), cs & 1u, abort_flag, 0x232 + i);
          if (!ok) break;
          if (i == 0) ++cnt_s0; else ++cnt_s1;
          tc_fence_after();
          if (elect_one()) {
            issue_pv_half(i, vslot, 1, true, nk_cur);
            tc_commit(bar(kBarSlotEmpty + vslot));
            if (more) {
              issue_qk(0, kslot, nk_j(j + 2, r0), i);
              r0 = r_inc(r0);
              tc_commit(bar(kBarSFull + i));
              tc_commit(bar(kBarSlotEmpty + kslot));
            } else {
              tc_commit(bar(kBarOFull + i));
            }
          }
          __syncwarp();
        }
        if (!ok) break;
      } else if (n_kv > 0) {
        // first key slab: both S tiles (a two-slab item: nq == 2)
        {
          ok = mbar_wait_warp(bar(kBarPairFull + pair_i), pair_ph, abort_flag, 0x210);
          if (!ok) break;
          pair_adv();
          const uint32_t slot = slot_i;
          slot_i = slot_next(slot_i);
          tc_fence_after();
          if (elect_one()) {
            issue_qk(0, slot, nk_j(0, 0), 0);
            tc_commit(bar(kBarSFull + 0));
            issue_qk(1, slot, nk_j(0, 0), 1);
            tc_commit(bar(kBarSFull + 1));
            tc_commit(bar(kBarSlotEmpty + slot));
          }
          __syncwarp();
        }
        // Per key slab j: P_0's first half -> P V (4 MMAs); all of P_0 -> the other 4 + next scores of
        // tile 0; the same for tile 1.  The barrier of V_j / K_{j+1} (loaded long before) is waited for
        // together with another wait, never on its own, and the bookkeeping for the next slab runs
        // while the queued MMAs drain.
        int rj = 0;
        bool pair_seen = false;   // V_j / K_{j+1} already known to have arrived
        for (int j = 0; ok && j < n_kv; ++j) {
          const int nk_cur = nk_j(j, rj);
          rj = r_inc(rj);
          const int nk_next = nk_j(j + 1, rj);
          const bool more = (j + 1 < n_kv);
          const uint32_t vslot = slot_i;
          const uint32_t kslot = slot_next(slot_i);
          slot_i = more ? slot_next(kslot) : kslot;
          if (pair_seen) ok = mbar_wait_warp(bar(kBarPHalf + 0), cnt_s0 & 1u, abort_flag, 0x224);
          else ok = mbar_wait2_warp(bar(kBarPairFull + pair_i), pair_ph, bar(kBarPHalf + 0), cnt_s0 & 1u, abort_flag, 0x211, 0x224);
          if (!ok) break;
          pair_adv();
          tc_fence_after();
          if (elect_one()) issue_pv_half(0, vslot, 0, j > 0, nk_cur);
          bool half1_done = false;   // first half of P_1 already seen complete
          ok = mbar_wait_probe_warp(bar(kBarPReady + 0), cnt_s0 & 1u, bar(kBarPHalf + 1), cnt_s1 & 1u, abort_flag, 0x220,
                                    &half1_done);
          if (!ok) break;
          ++cnt_s0;
          tc_fence_after();
          if (elect_one()) {
            issue_pv_half(0, vslot, 1, true, nk_cur);
            if (more) {
              issue_qk(0, kslot, nk_next, 0);
              tc_commit(bar(kBarSFull + 0));
            } else {
              tc_commit(bar(kBarOFull + 0));
            }
          }
          __syncwarp();
          if (!half1_done) {
            ok = mbar_wait_warp(bar(kBarPHalf + 1), cnt_s1 & 1u, abort_flag, 0x225);
            if (!ok) break;
          }
          tc_fence_after();
          if (elect_one()) issue_pv_half(1, vslot, 0, j > 0, nk_cur);
          // all of P_1, and (one round trip) the loads of the next slab
          pair_seen = false;
          if (more) {
            ok = mbar_wait_probe_warp(bar(kBarPReady + 1), cnt_s1 & 1u, bar(kBarPairFull + pair_i), pair_ph, abort_flag, 0x221,
                                      &pair_seen);
          } else {
            ok = mbar_wait_warp(bar(kBarPReady + 1), cnt_s1 & 1u, abort_flag, 0x221);
          }
          if (!ok) break;
          ++cnt_s1;
          tc_fence_after();
          if (elect_one()) {
            issue_pv_half(1, vslot, 1, true, nk_cur);
            tc_commit(bar(kBarSlotEmpty + vslot));
            if (more) {
              issue_qk(1, kslot, nk_next, 1);
              tc_commit(bar(kBarSFull + 1));
              tc_commit(bar(kBarSlotEmpty + kslot));
            } else {
              tc_commit(bar(kBarOFull + 1));
            }
          }
          __syncwarp();
        }
        if (!ok) break;
      } else {
        if (elect_one()) {
          tc_commit(bar(kBarOFull + 0));
          if (nq > 1) tc_commit(bar(kBarOFull + 1));
        }
        __syncwarp();
      }
      ++it_q0;
      if (nq > 1) ++it_q1;
      ++it_o0;
      if (use_o1) ++it_o1;
    }
    // Every MMA issued so far must have completed before the TMEM allocation is released (after
    // a timeout some may still be in flight): one more commit, awaited with a bound of its own.
    if (elect_one()) {
      tc_commit(bar(kBarDrain));
      const unsigned long long t0 = globaltimer_ns();
      while (!mbar_try_wait(bar(kBarDrain), 0u)) {
        if (globaltimer_ns() - t0 > kTimeoutNs) break;
      }
    }
    __syncwarp();
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
    // ======================================================================= softmax warps
    const int qi = (warp - kFirstSoftmaxWarp) >> 2;   // tile (S_i, O_i) handled by this warpgroup
    const int row = (warp & 3) * 32 + lane;       // row of the slab == TMEM lane
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_addr + (uint32_t)qi * 128u;
    const uint32_t tO = tmem + lane_addr + 256u + (uint32_t)qi * 128u;
    uint32_t it_o0 = 0, it_o1 = 0, cnt_s = 0, kv_g = 0;
    uint32_t n_stage = 0;   // output slabs staged by this warpgroup so far
    uint32_t n_merge = 0;   // split-KV merges so far
    bool ok = true;
    const float neg_inf = __int_as_float(0xff800000);
    float2* xchg = reinterpret_cast<float2*>(smem + kOffXchg);

    for (uint32_t n = 0; ok; ++n) {
      WorkItem wi;
      if (!next_item(n, wi)) break;
      const int head = wi.x, qb = wi.y, sub0 = wi.w & 0xffff, nq = (wi.w >> 16) & 0xff;
      const bool split = ((wi.w >> 24) & 1) != 0;
      const bool textq = ((wi.w >> 25) & 1) != 0;
      const int n_vid = wi.z * g.n_sub;          // video key slabs, then the text slabs (always 128 wide)
      const int n_kv = n_vid + g.n_ts;
      const bool use_o1 = (nq > 1) || (split && n_kv > 1);
      const bool active = (qi == 0) || use_o1;
      float m_ref = neg_inf;  // running reference maximum, scaled log2 domain
      float l = 0.f;          // running sum of exp2(s - m_ref)
      if (active) {
        // key slabs of this tile: all of them, or every second one in a split-KV item
        const int j0 = split ? qi : 0, dj = split ? 2 : 1;
        const int r_last = g.n_sub - 1;
        int rj = (j0 > r_last) ? 0 : j0;   // j mod n_sub, carried along (no division in the loop)
        for (int j = j0; ok && j < n_kv; j += dj) {
          const int nk = (rj == r_last && j < n_vid) ? g.n_last : kSlabTokens;
          rj = (rj == r_last) ? 0 : rj + 1;
          if (dj == 2) rj = (rj == r_last) ? 0 : rj + 1;
          ok = mbar_wait_warp(bar(kBarSFull + qi), cnt_s & 1u, abort_flag, 0x300 + qi);
          if (!ok) break;
          ++cnt_s;
          tc_fence_after();
          // Read the slab's validity words first: shared memory is busy feeding the tensor core,
          // so the load's latency is overlapped with the TMEM loads that follow.
          const uint4 m = *reinterpret_cast<const uint4*>(meta + ((kv_g + (uint32_t)j) % kMetaRing) * 8);
          const uint32_t bh = bar(kBarPHalf + qi), br = bar(kBarPReady + qi);
          const bool first = (j == j0);
          if (nk == 128) softmax_slab<128>(tS, tO, m, first, g.scale_log2, m_ref, l, bh, br);
          else if (nk == 112) softmax_slab<112>(tS, tO, m, first, g.scale_log2, m_ref, l, bh, br);
          else if (nk == 96) softmax_slab<96>(tS, tO, m, first, g.scale_log2, m_ref, l, bh, br);
          else softmax_slab<64>(tS, tO, m, first, g.scale_log2, m_ref, l, bh, br);
        }
      }
      kv_g += (uint32_t)n_kv;
      if (!ok) break;
      const uint32_t par_o0 = it_o0 & 1u, par_o1 = it_o1 & 1u;
      ++it_o0;
      if (use_o1) ++it_o1;
      if (!active) continue;

      // ---- epilogue: out = O / l, lse = ln2 * (m_ref + log2 l).  In a split-KV item the two
      // partial results (even / odd key slabs) of each row are merged by warpgroup 0, which can
      // read both accumulators because they sit in the same TMEM lanes.
      float scale0 = 1.f, scale1 = 0.f;   // weights of O_0 and O_1 in the merged output
      if (split && qi == 1) {
        // hand (m, l) of the odd key slabs to warpgroup 0 (release / acquire through the barrier)
        xchg[row] = make_float2(m_ref, l);
        mbar_arrive(bar(kBarMerge));
        continue;
      }
      ok = mbar_wait_warp(bar(kBarOFull + qi), (qi == 0 ? par_o0 : par_o1), abort_flag, 0x310 + qi);
      if (!ok) break;
      if (split && use_o1) {
        ok = mbar_wait_warp(bar(kBarOFull + 1), par_o1, abort_flag, 0x312);
        if (!ok) break;
        ok = mbar_wait_warp(bar(kBarMerge), n_merge & 1u, abort_flag, 0x313);
        if (!ok) break;
        ++n_merge;
        const float2 other = xchg[row];
        const float m_all = fmaxf(m_ref, other.x);
        scale0 = (m_ref == neg_inf) ? 0.f : fast_exp2(m_ref - m_all);
        scale1 = (other.x == neg_inf) ? 0.f : fast_exp2(other.x - m_all);
        l = scale0 * l + scale1 * other.y;
        m_ref = m_all;
      }
      tc_fence_after();
      const bool empty = (n_kv == 0) || !(l > 0.f);
      const float inv = empty ? 0.f : 1.f / l;
      scale0 *= inv;
      scale1 *= inv;
      uint8_t* stage = smem + kOffQ + (uint32_t)qi * kSlabBytes;
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) {
        uint32_t o[32];
        if (n_kv > 0) {
          tc_ld32(tO + c4 * 32, o);
          tc_wait_ld();
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c) o[c] = 0u;
        }
        if (split && use_o1) {   // qi == 0 here: add the odd-slab accumulator
          uint32_t o1[32];
          tc_ld32(tO + 128u + c4 * 32, o1);
          tc_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; ++c)
            o[c] = __float_as_uint(__uint_as_float(o[c]) * scale0 + __uint_as_float(o1[c]) * scale1);
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * scale0);
        }
#pragma unroll
        for (int c8 = 0; c8 < 4; ++c8) {
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float a = empty ? 0.f : __uint_as_float(o[c8 * 8 + 2 * e]);
            const float b = empty ? 0.f : __uint_as_float(o[c8 * 8 + 2 * e + 1]);
            w[e] = pack_bf16(a, b);
          }
          // 128-byte swizzle of the staging slab: 16-byte chunk index xor (row mod 8)
          const int col = c4 * 32 + c8 * 8;
          const int half = col >> 6, chunk = (col & 63) >> 3;
          uint8_t* dst = stage + half * kHalfBytes + row * 128 + ((chunk ^ (row & 7)) << 4);
          if (PSA_CHECKED(dst >= smem + kOffQ && dst + 16 <= smem + kOffQ + 2u * kSlabBytes &&
                          (reinterpret_cast<uintptr_t>(dst) & 15u) == 0u, 0xD12))
            *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
      tc_fence_before();
      mbar_arrive(bar(kBarOEmpty + qi));
      if (split && use_o1) mbar_arrive(bar(kBarOEmpty + 1));
      int t0, h0, w0, et, eh, ew, ntok, last;
      const float lse_row = empty ? neg_inf : (m_ref + log2f(l)) * 0.6931471805599453f;
      if (textq) {   // text slab: rows are consecutive text tokens; they follow the L video tokens
        t0 = 0; h0 = 0; w0 = (sub0 + qi) * kSlabTokens; last = 2;
        if (w0 + row < g.n_text && PSA_CHECKED(head >= 0 && head < g.n_heads && w0 >= 0, 0xD10))
          prm.lse[(long long)head * g.Lt + g.L + w0 + row] = lse_row;
      } else {
        slab_origin(g, qb, sub0 + qi, t0, h0, w0);
        slab_shape(g, sub0 + qi, et, eh, ew, ntok, last);
        const int wi_ = row % ew, hi_ = (row / ew) % eh, ti_ = row / (ew * eh);
        const int t = t0 + ti_, hh = h0 + hi_, ww = w0 + wi_;
        if (row < ntok && t < g.T && hh < g.H && ww < g.W) {
          const long long tok = ((long long)t * g.H + hh) * g.W + ww;
          if (PSA_CHECKED(head >= 0 && head < g.n_heads && tok >= 0 && tok < g.L, 0xD11)) prm.lse[(long long)head * g.Lt + tok] = lse_row;
        }
      }
      // Every thread's staged row is made visible to the TMA engine; the warpgroup's first warp
      // waits for all 128 rows (a bounded wait, like every other one) and stores the slab.
      fence_async_smem();
      mbar_arrive(bar(kBarStage + qi));
      if ((warp & 3) == 0) {
        ok = mbar_wait_warp(bar(kBarStage + qi), n_stage & 1u, abort_flag, 0x320 + qi);
        if (!ok) break;
        if (lane == 0) {
          const uint32_t src = sbase + kOffQ + (uint32_t)qi * kSlabBytes;
          if (PSA_CHECKED(w0 >= 0 && h0 >= 0 && t0 >= 0 && head >= 0 && head < g.n_heads && last >= 0 && last <= 2, 0xD13)) {
            tma_store_5d(&tms.o[last], src, 0, w0, h0, t0, head);
            tma_store_5d(&tms.o[last], src + kHalfBytes, 64, w0, h0, t0, head);
          }
          tma_store_commit();
          tma_store_wait_read();
          mbar_arrive(bar(kBarQEmpty + qi));
        }
        __syncwarp();
      }
      ++n_stage;
    }
    if ((warp & 3) == 0 && lane == 0) tma_store_wait_all();
  }

  // ------------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag != 0) {
    if (atomicCAS(prm.ws_header + kWsStatus, 0, (int)PSA_ERR_TIMEOUT) == 0) prm.ws_header[kWsDetail] = *abort_flag;
  }
  if (warp == kWarpMma) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(*tmem_slot), "r"(512) : "memory");
  }
}

// One warp waits, with the kernel's own bounded wait, on a barrier that nothing arrives on.
// The wait must give up after limit_ns, record PSA_ERR_TIMEOUT and return normally.
__global__ void wait_probe_kernel(int* ws_header, unsigned long long limit_ns) {
  __shared__ __align__(8) unsigned long long probe_bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&probe_bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  const bool ok = mbar_wait(smem_u32(&probe_bar), 0, &abort_flag, 0x7e57, limit_ns);
  __syncwarp();
  if (threadIdx.x == 0 && !ok) {
    if (atomicCAS(ws_header + kWsStatus, 0, (int)PSA_ERR_TIMEOUT) == 0) ws_header[kWsDetail] = abort_flag;
  }
}

cudaError_t launch_wait_probe(int* ws_header, unsigned long long limit_ns, cudaStream_t stream) {
  wait_probe_kernel<<<1, 32, 0, stream>>>(ws_header, limit_ns);
  return cudaGetLastError();
}

// ----------------------------------------------------------------------------- launchers
size_t plan_smem_bytes(const Geom& g) { return sizeof(int) * (size_t)(g.Tp + g.Sp + g.NB); }

cudaError_t launch_plan(const HeadParamsArray& hp, const Geom& g, int head0, int n_heads_here, bool clear_status,
                        int* ws_header, psa_head_params* hp_dev, WorkItem* items, cudaStream_t stream) {
  const size_t smem = plan_smem_bytes(g);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  plan_kernel<<<n_heads_here, 256, smem, stream>>>(hp, g, head0, clear_status ? 1 : 0, ws_header, hp_dev, items);
  return cudaGetLastError();
}

cudaError_t launch_attn(const TensorMaps& tm, const Geom& g, const WorkItem* items, const psa_head_params* hp_dev,
                        int* ws_header, float* lse, int n_items, int n_sms, bool shared_qkv, cudaStream_t stream) {
  {  // per device, cheap: set on every call
    cudaError_t e = cudaFuncSetAttribute(attn_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemAlloc);
    if (e != cudaSuccess) return e;
  }
  AttnParams prm;
  prm.g = g;
  prm.items = items;
  prm.hp_dev = hp_dev;
  prm.ws_header = ws_header;
  prm.lse = lse;
  prm.n_items = n_items;
  prm.shared_qkv = shared_qkv ? 1 : 0;
  const int grid = n_items < n_sms ? n_items : n_sms;
  if (grid <= 0) return cudaSuccess;
  attn_fwd_kernel<<<grid, kThreads, kSmemAlloc, stream>>>(tm, prm);
  return cudaGetLastError();
}

}  // namespace psa

