// Stage 4: grouped SwiGLU expert FFN over the activated experts with weighted combine,
//   y_t = sum_e w_{t,e} * W_down_e ( silu(W_gate_e x_t) * (W_up_e x_t) ),
// the step whose cost is the number of distinct expert weights touched (Section 1; Section 3.1).
//
// bf16 path (sm_100a): one persistent kernel, one CTA per SM, eight specialised warps:
//   warp 0      weight producer: one TMA copy per operand and stage (32 KB of weights = 128 rows x 128 K
//               in two 128-byte-swizzled atoms, plus the x chunk of gate/up stages) into a 3-stage ring
//   warp 1      issues tcgen05.mma (M=128 weight rows, N=node columns, fp32 accumulators in TMEM)
//   warps 2..5  epilogue: tcgen05.ld, SwiGLU / combine; only TMEM and shared memory are touched here
//   warp 6      helper: waits for other CTAs' partial sums and copies them into shared memory ahead of
//               need; adds the activation chunk to down stages once their experts are complete
//   warp 7      publisher: moves staged fragments / activation tiles to global memory (bulk reduce-add,
//               TMA store), waits for completion, then raises the counter other CTAs wait on
// The weights are the M operand ("swap-AB"): every activated expert's weights are read from HBM
// exactly once for all nodes of the block.  Work plan of a launch (plan_lane):
//   gate/up  tile = 64 gate rows + the 64 matching up rows of one expert, K = hidden.  The
//            n_tiles mod grid leftover tiles come first, cut into equal contiguous ranges of (tile,
//            K-chunk) units over all CTAs; the CTA that owns a tile's last chunk receives the others'
//            partial sums (added into its pre-zeroed global buffer), applies w * silu(g) * u and
//            stores the activation tile.  Then whole tiles, one per CTA and round.
//   down     tile = 128 output rows, K = (activated expert, intermediate) concatenated, cut evenly;
//            experts complete early first.  Partial tiles are added to the output with fp32
//            reductions in L2 (the caller zeroes the output).
// The down phase reads activations written by other CTAs in the gate/up phase; one finished-tile counter
// per expert orders them (a CTA waits for the experts its share of the K range reads).  Every wait is
// bounded; on expiry the kernel raises a status and drains.
//
// f32 path: plain FMA kernels (the fp32 toy configuration is a few MFLOP).
#include <cuda_bf16.h>

#include <mutex>

#include "acm_internal.h"
#include "ffn_plan.h"

namespace acm {
namespace {

#ifndef ACM_FFN_MX
#define ACM_FFN_MX 0
#endif
constexpr int kMaxStages = 3;                            // pipeline stages of the weight ring (see Geo)
constexpr int kAcc = 4;                                  // TMEM accumulators in flight (power of two)
constexpr int kBK = 64;                                  // K elements of one 128-byte swizzle atom
constexpr int kAtoms = 2;                                // atoms per pipeline stage: a stage covers 128 K
constexpr int kTileM = 128;
constexpr int kAtomABytes = kTileM * kBK * 2;            // 16 KB: 128 weight rows x one atom
constexpr int kABytes = kAtoms * kAtomABytes;            // 32 KB weight tile, one TMA copy
// The epilogue handles node columns kMaxNodes = 64 at a time: one fragment, one activation tile.  A wide tile (a
// batch of blocks with more than 64 nodes in all, up to kWideNodes = 128 accumulator columns) goes in two halves.
constexpr int kOutStageBytes = kTileM * kMaxNodes * 4;   // 32 KB: outgoing fragment (also the gate/up exchange buffer)
constexpr int kHStageBytes = kMaxNodes * 64 * 2;         // 8 KB: one finished activation tile (64 features x 64 nodes)
constexpr int kMxACols = 64;                             // MXFP4: one expanded weight stage in tensor memory = 128 K bf16 per row
static_assert(kAcc * kMaxNodes + kMaxStages * kMxACols <= 512, "tensor memory: accumulators + expanded weight stages");
// ACM_FFN_MX = 1 (set by ffn_mx.cu, which includes this file) builds the same kernel for MXFP4 expert
// weights: a pipeline stage of a weight tile arrives as 128 rows x 64 bytes of E2M1 codes + 128 x 4 E8M0
// scale bytes (one contiguous 8704-byte copy into the stage's weight area), and four more warps expand it
// there to the 32 KB bf16 tile the MMAs read -- every MXFP4 value is a bf16, so the arithmetic is the
// bf16 path's.
constexpr int kThreads = ACM_FFN_MX ? 384 : 256;         // producer, MMA, 4 epilogue warps, helper, publisher (+ 4 expanding warps)
constexpr int kMxCodeBytes = kTileM * 64;                // 128 rows x 128 four-bit codes
[[maybe_unused]] constexpr int kMxStageBytes = kMxCodeBytes + kTileM * 4; // + one scale byte per row and 32 K
constexpr int kFragBytes = kTileM * kMaxNodes * 4;       // contributor fragments pre-summed in shared memory
constexpr int kFragFloats = kTileM * kMaxNodes;

using plan::FastDiv;
using plan::make_fastdiv;
using plan::fdiv;
using plan::Segment;
using plan::SegRange;
using plan::Plan;
using plan::Sched;
using plan::make_range;
using plan::cut_begin;
using plan::plan_lane;

// Every wait in this kernel is bounded.  What a role needs when one runs out lives in shared memory (GiveUp,
// touched on slow paths only): the limit, where to raise the status, and this CTA's diagnostic word, which
// names the wait that gave up first (acm_wait_report reads it).
enum WaitSite : int {
  kSiteNone = 0,
  kSiteAnchorWords = 1,     // prologue: the anchors' tagged words (router kernel's root CTAs)
  kSiteEligibleWords = 2,   // prologue / helper: the eligible set's tagged words (selection kernel)
  kSiteStageEmpty = 3,      // weight producer: a ring stage the MMAs have not released
  kSiteAccEmpty = 4,        // MMA issuer: an accumulator the epilogue has not drained
  kSiteStageFull = 5,       // MMA issuer: a stage whose copies have not landed
  kSiteFragFree = 6,        // helper: the fragment buffer in shared memory is still being read
  kSiteFragArrivals = 7,    // helper: other CTAs' partial sums of a cut tile
  kSiteFragCopy = 8,        // helper: its own bulk copy of the summed fragment
  kSiteExpertReady = 9,     // helper: finished-tile counters of the experts a down stage reads
  kSiteStageArmed = 10,     // helper: the weight producer has not armed the stage
  kSiteOutStaged = 11,      // publisher: an outgoing fragment from the epilogue
  kSiteActStaged = 12,      // publisher: a finished activation tile from the epilogue
  kSiteAccFull = 13,        // epilogue: an accumulator's MMAs
  kSiteOutFree = 14,        // epilogue: the outgoing-fragment buffer
  kSiteFragFull = 15,       // epilogue: the summed fragments of a cut tile
  kSiteActFree = 16,        // epilogue: an activation staging buffer
  kSitePlanReady = 17,      // any role: the rest of the plan (anchor start)
  kSitePackedStage = 18     // MXFP4 expanding warps: the packed weight stage
};
struct GiveUp {
  volatile int flag;             // set once this CTA has given up: every role then leaves at its next slow path
  unsigned long long limit_ns;   // the longest any single wait may last
  int32_t* status;               // the context's sticky status word
  int32_t* where;                // this CTA's diagnostic word: (launch number << 8) | WaitSite
  int32_t tag;                   // launch number << 8
};

template <int kN>
struct __align__(8) BarriersT {
  unsigned long long full[kMaxStages];
  unsigned long long empty[kMaxStages];
  unsigned long long tfull[kAcc];
  unsigned long long tempty[kAcc];
  unsigned long long drained;
  unsigned long long frag_full;      // helper -> epilogue: the pre-summed fragments of the next cut tile (half) are in smem
  unsigned long long frag_free;      // epilogue -> helper: the fragment buffer may be overwritten
  unsigned long long helper;         // completion of the helper warp's bulk copy
  unsigned long long ost_full, ost_free;   // epilogue <-> publisher: outgoing fragment staged / copied out
  unsigned long long hst_full[2], hst_free[2];   // epilogue <-> publisher: activation tile staged / stored
#if ACM_FFN_MX
  unsigned long long raw[kMaxStages];   // the packed weight stage has landed (producer's copy -> expanding warps)
#endif
  volatile uint32_t armed;           // stages whose barrier the weight producer has armed so far
  volatile int32_t n_routed_slots;   // routed experts in this launch's work list (known with the complete list)
  uint32_t tmem_base;
  GiveUp give_up;
  float wd[kN];                 // combine weights of the expert being finalised
  int32_t entry[kMaxSlots];     // this launch's work list: make_entry(source, index) of every activated slot
  int16_t expert[kMaxSlots];    // routed expert id of the slot (-1: shared expert)
  uint32_t sel_half[4 * kMaskWords];   // early start: the eligible mask in 16-bit pieces (second half: blocks 4..7 of a batch)
  Plan plan;                    // this launch's work plan
  unsigned long long plan_ready;     // anchors' pre-segment: the rest of the plan and of the work list is in place
  uint32_t anc_part[4 * kMaskWords];   // early start on the anchors: their mask in 16-bit pieces (by the two polling warps)
};

// Geometry of the kernel for accumulator tiles of kN node columns: 64 (one block, three 48 KB stages) or 128 (a
// batch, two 64 KB stages -- as many bytes in flight -- and all of tensor memory).
template <int kN>
struct Geo {
  static constexpr int kStages = kN > kMaxNodes ? 2 : 3;
  static constexpr int kBBytes = kAtoms * kN * kBK * 2;          // activation chunk of a stage, one TMA copy
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kTmemCols = ACM_FFN_MX ? 512 : kAcc * kN;    // MXFP4: accumulators, then the expanded weight stages
  static constexpr size_t kSmemBytes =
      1024 + static_cast<size_t>(kStages) * kStageBytes + kOutStageBytes + kFragBytes + 2 * kHStageBytes + sizeof(BarriersT<kN>);
  static_assert(kSmemBytes <= 232448, "shared memory: ring + staging buffers + control block exceed 227 KB");
  static_assert(kStages <= kMaxStages, "barrier arrays");
};

// ---------------------------------------------------------------------------------- PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ unsigned long long global_timer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}\n"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Has a wait that began at t0 outlasted the limit?  The clock is read twice before the answer is yes: a single
// reading that lies outside [t0, t0 + limit] (a value caught while the counter's halves roll over would) must
// not end a healthy launch.
__device__ __forceinline__ bool limit_passed(unsigned long long t0, unsigned long long limit_ns) {
  const long long d1 = static_cast<long long>(global_timer() - t0);
  if (d1 >= 0 && static_cast<unsigned long long>(d1) <= limit_ns) return false;
  const long long d2 = static_cast<long long>(global_timer() - t0);
  return d2 < 0 ? false : static_cast<unsigned long long>(d2) > limit_ns;
}
__device__ __noinline__ void give_up(GiveUp* g, int site) {
  if (atomicExch(const_cast<int*>(&g->flag), 1) == 0 && g->where) *g->where = g->tag | site;
  atomicCAS(g->status, 0, static_cast<int32_t>(ACM_ERR_TIMEOUT));
}
// Returns false if the limit ran out (the status is raised once) or the CTA has already given up; callers
// then skip the rest of their work.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, GiveUp* g, int site) {
  if (g->flag) return false;
  for (int i = 0; i < 1024; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_timer();
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (g->flag) return false;
    if (limit_passed(t0, g->limit_ns)) {
      give_up(g, site);
      return false;
    }
  }
}
// One inlined poll for the common case (the phase is already complete), the bounded loop out of line: the
// single-thread roles pay every instruction of their per-stage loop.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, GiveUp* g, int site) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, g, site);
}
__device__ __forceinline__ int ld_acquire(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_add(int32_t* p, int v) {
  asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Bounded wait until *p >= target (p written by other CTAs with release semantics).
__device__ bool flag_wait_ge(const int32_t* p, int target, GiveUp* g, int site) {
  if (g->flag) return false;
  for (int i = 0; i < 256; ++i)
    if (ld_acquire(p) >= target) return true;
  const unsigned long long t0 = global_timer();
  for (;;) {
    for (int i = 0; i < 16; ++i) {
      if (ld_acquire(p) >= target) return true;
      __nanosleep(64);
    }
    if (g->flag) return false;
    if (limit_passed(t0, g->limit_ns)) {
      give_up(g, site);
      return false;
    }
  }
}
// Bounded poll of one self-validating word (16 payload bits under a 16-bit tag) written by an earlier kernel
// of the same stream: returns the payload, or sets `seen` to false when the limit ran out.
__device__ __forceinline__ uint32_t poll_tagged_word(const uint32_t* word, uint32_t tag, unsigned long long limit_ns, bool& seen) {
  uint32_t v = 0;
  const unsigned long long t0 = global_timer();
  do {
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(word) : "memory");
    seen = (v >> 16) == tag;
  } while (!seen && !limit_passed(t0, limit_ns));
  return seen ? (v & 0xffffu) : 0u;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
#if ACM_FFN_MX
__device__ __forceinline__ void bulk_load_hint(uint32_t smem_dst, const void* gmem_src, uint32_t bytes, uint32_t bar, uint64_t policy) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
               ::"r"(smem_dst), "l"(gmem_src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
}
#endif
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

// Barrier over the 128 epilogue threads that also ANDs a predicate, so that all of them take the
// same decision after a bounded wait (a thread that left alone would strand the others at a barrier).
__device__ __forceinline__ bool epi_vote_all(bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %1, 0;\n\t"
      "bar.red.and.pred q, 1, 128, p;\n\tselp.u32 %0, 1, 0, q;\n\t}\n"
      : "=r"(r) : "r"(static_cast<uint32_t>(pred)) : "memory");
  return r != 0;
}

__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3, %4}], [%5], %6;"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2, int c3, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3, %4, %5}], [%6], %7;"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2, int c3, int c4, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3, %4, %5, %6}], [%7], %8;"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}\n"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, rows of 128 bytes, 128-byte swizzle, groups of
// 8 rows 1024 bytes apart.  The tile base is 1024-byte aligned; stepping K by 16 elements adds 32 bytes.
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3ffffu) >> 4);       // start address
  d |= static_cast<uint64_t>(1) << 16;                           // leading byte offset (unused here)
  d |= static_cast<uint64_t>(1024 >> 4) << 32;                   // stride byte offset
  d |= static_cast<uint64_t>(1) << 46;                           // descriptor version
  d |= static_cast<uint64_t>(2) << 61;                           // 128-byte swizzle
  return d;
}
#if ACM_FFN_MX
// The same MMA with the A operand (128 rows x 16 K bf16) in tensor memory: row = lane, two K elements per column.
__device__ __forceinline__ void umma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}\n"
      ::"r"(tmem_d), "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}
// 16 consecutive columns of this thread's lane
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
        "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
#endif
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t umma_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(kTileM >> 4) << 24);
}

// Optional time stamps (acm_stage_timing): per CTA, slot 0 = the roles start, 10 / 11 = its last gate/up / down tile is done.
#define ACM_STAMP(slot) do { if (p.trace) p.trace[static_cast<size_t>(blockIdx.x) * 32 + (slot)] = global_timer(); } while (0)

struct FfnArgs {
  int T, H, I, n_pad;
  FastDiv d_grid, d_kc1, d_tpe, d_kpe;   // reciprocals of the grid size and of the per-tile / per-expert chunk counts
  const uint32_t* act_mask;
  const uint32_t* resident;
  int li, n_shared;
  uint32_t only[4];
  const int32_t* slot_of;
  const float* wtab;
  acm_block_stats* stats;
  __nv_bfloat16* hbuf;
  int32_t* ready;
  float* frag;
  int32_t* frag_flag;
  const uint32_t* sel_flag;
  int32_t sel_epoch;
  int sel_blocks;
  const uint32_t* anc_flag;    // non-null: eight tagged words with the anchor experts (Eq. 5), published before sel_flag
  float* out;
  int32_t* status;
  unsigned long long wait_limit_ns;   // the longest any single device-side wait may last
  int32_t* wait_diag;          // [grid] per-CTA diagnostic words (see GiveUp) or null
  int32_t launch_tag;          // launch number << 8
  unsigned long long* trace;   // optional [grid][32] time stamps (acm_stage_timing) or null
#if ACM_FFN_MX
  const unsigned char* mx_gate_up;   // [E][I/64][H/128][8704]
  const unsigned char* mx_down;      // [E][H/128][I/128][8704]
#endif
};

__device__ __forceinline__ const CUtensorMap* pick_map(int src, const CUtensorMap* routed, const CUtensorMap* shared,
                                                       const CUtensorMap* staged) {
  return src == kSrcRouted ? routed : src == kSrcShared ? shared : staged;
}

// The plan (ffn_plan.h) lives in shared memory: a private copy indexed at run time would live in local memory,
// whose first touch costs every role a trip to DRAM at the start of the kernel.
#if ACM_FFN_MX
#define ACM_FFN_KERNEL k_ffn_mxfp4
#else
#define ACM_FFN_KERNEL k_ffn_bf16
#endif
// One kernel for both starts (on the anchors' pre-segment, or with the whole work list at hand): a launch bracketed
// by events then runs the same code as the launches around it, which keeps its instructions warm in the caches.
// kN = node columns of an accumulator tile (see Geo).
template <int kN>
__global__ void __launch_bounds__(kThreads, 1)
ACM_FFN_KERNEL(const __grid_constant__ FfnMaps maps, const __grid_constant__ CUtensorMap x_map,
           const __grid_constant__ CUtensorMap h_map, const __grid_constant__ CUtensorMap hs_map,
           const FfnArgs p) {
  constexpr int kStages = Geo<kN>::kStages, kStageBytes = Geo<kN>::kStageBytes, kAccCols = kN, kTmemCols = Geo<kN>::kTmemCols;
  using Barriers = BarriersT<kN>;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  unsigned char* stage_base = smem;
  unsigned char* after_ring = smem + static_cast<size_t>(kStages) * kStageBytes;
  float* ostage = reinterpret_cast<float*>(after_ring);           // outgoing fragment [node][128 rows]
  float* ex = ostage;                                             // gate/up exchange aliases it (never used at once)
  float* sfrag = reinterpret_cast<float*>(after_ring + kOutStageBytes);
  unsigned char* hstage = after_ring + kOutStageBytes + kFragBytes;   // 2 x [node][64 features] bf16, swizzled
  Barriers* bars = reinterpret_cast<Barriers*>(after_ring + kOutStageBytes + kFragBytes + 2 * kHStageBytes);
  GiveUp* const quit = &bars->give_up;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, G = gridDim.x;
  griddep_launch_dependents();
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&bars->full[s]), ACM_FFN_MX ? 5 : 1);   // MXFP4: + one arrival per expanding warp
      mbar_init(smem_u32(&bars->empty[s]), 1);
#if ACM_FFN_MX
      mbar_init(smem_u32(&bars->raw[s]), 1);
#endif
    }
    for (int b = 0; b < kAcc; ++b) {
      mbar_init(smem_u32(&bars->tfull[b]), 1);
      mbar_init(smem_u32(&bars->tempty[b]), 128);
    }
    mbar_init(smem_u32(&bars->drained), 1);
    mbar_init(smem_u32(&bars->plan_ready), 1);
    mbar_init(smem_u32(&bars->frag_full), 1);
    mbar_init(smem_u32(&bars->frag_free), 128);
    mbar_init(smem_u32(&bars->helper), 1);
    mbar_init(smem_u32(&bars->ost_full), 128);
    mbar_init(smem_u32(&bars->ost_free), 1);
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars->hst_full[b]), 128);
      mbar_init(smem_u32(&bars->hst_free[b]), 1);
    }
    bars->give_up.flag = 0;
    bars->give_up.limit_ns = p.wait_limit_ns;
    bars->give_up.status = p.status;
    bars->give_up.where = p.wait_diag ? p.wait_diag + blockIdx.x : nullptr;
    bars->give_up.tag = p.launch_tag;
    if (p.wait_diag) p.wait_diag[blockIdx.x] = p.launch_tag;      // "this CTA of that launch has started"
    bars->armed = 0;
    fence_barrier_init();
  }
  if (warp == 0 && lane == 0) {
#if !ACM_FFN_MX
    prefetch_tensormap(&maps.gate_up);
    prefetch_tensormap(&maps.down);
#endif
    prefetch_tensormap(&x_map);
    prefetch_tensormap(&h_map);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&bars->tmem_base), kTmemCols);
    tmem_relinquish();
  }
  // Everything above touched only this CTA's own resources; global memory written by the kernels
  // before this one is read only from here on.  Early start: wait for the eligible set only.
  const bool early = p.sel_flag != nullptr;
  // Early start on the ANCHORS (Eq. 5: the root's natural top-k, always eligible): the router kernel publishes
  // them microseconds before the selection is done.  Their gate/up tiles become segment 0 of the plan, one
  // whole tile per CTA, and the roles start on it at once; the helper warp meanwhile waits for the eligible
  // set, completes the work list (the pre-streamed experts keep the first slots) and the plan, and opens
  // `plan_ready`, which every other role passes before its second segment.
  const bool pre = p.anc_flag != nullptr && p.sel_flag != nullptr;
  if (pre || early) {
    // Eight tagged words per block (16 mask bits under the 16-bit tag of this call; a batch has eight per block
    // and takes their union), each polled by its own thread of warps 2 and 3 -- four blocks per warp -- which have
    // nothing else to do yet, so that the poll runs beside the set-up above.  With the anchor start these are the
    // anchors' words, else the eligible set's.
    bool timed_out = false;
    if (threadIdx.x >= 64 && threadIdx.x < 128) {
      const int j = threadIdx.x - 64;
      const uint32_t* words = pre ? p.anc_flag : p.sel_flag;
      bool seen = true;
      uint32_t bits = 0u;
      if (j < 2 * kMaskWords * p.sel_blocks)
        bits = poll_tagged_word(words + j, static_cast<uint32_t>(p.sel_epoch) & 0xffffu, p.wait_limit_ns, seen);
      timed_out = !seen;
      bits |= __shfl_xor_sync(0xffffffffu, bits, 8);
      bits |= __shfl_xor_sync(0xffffffffu, bits, 16);
      if (lane < 2 * kMaskWords) (pre ? bars->anc_part : bars->sel_half)[(j >> 5) * 2 * kMaskWords + lane] = bits;
    }
    __syncthreads();
    if (timed_out) give_up(quit, pre ? kSiteAnchorWords : kSiteEligibleWords);
  } else {
    griddep_wait();
  }
  // The work list of this launch: slot a = the a-th activated expert of this list in ascending id
  // order (list 0: the resident ones, then the shared experts; list 1: the non-resident ones, which
  // the host has copied into staging slot a).
  uint32_t am[kMaskWords];
  int n_routed = 0;
#pragma unroll
  for (int wd = 0; wd < kMaskWords; ++wd) {
    uint32_t act;
    if (pre) {
      act = (bars->anc_part[2 * wd] | bars->anc_part[2 * kMaskWords + 2 * wd]) |
            ((bars->anc_part[2 * wd + 1] | bars->anc_part[2 * kMaskWords + 2 * wd + 1]) << 16);      // for now: the anchors only
    } else if (early) {
      act = (bars->sel_half[2 * wd] | bars->sel_half[2 * kMaskWords + 2 * wd]) |
            ((bars->sel_half[2 * wd + 1] | bars->sel_half[2 * kMaskWords + 2 * wd + 1]) << 16);
    } else {
      act = p.act_mask[wd];
    }
    const uint32_t res = p.resident ? p.resident[wd] : 0xffffffffu;
    am[wd] = (p.li == 0 ? act & res : act & ~res) & p.only[wd];
    n_routed += __popc(am[wd]);
  }
  const int tpe = p.I / 64;          // gate/up tiles per expert = K-chunks per expert in the down phase
  const int n_halves = (kN > kMaxNodes && p.n_pad > kMaxNodes) ? 2 : 1;   // the epilogue takes 64 node columns at a time
  // pre-segment: as many of the anchors (in ascending id) as give every CTA at most one whole tile
  const int n_pre = pre ? min(n_routed, static_cast<int>(fdiv(static_cast<unsigned>(G), p.d_tpe))) : 0;
  if (pre) {
    // keep the first n_pre anchors only
    int left = n_pre;
#pragma unroll
    for (int wd = 0; wd < kMaskWords; ++wd) {
      uint32_t m = am[wd], kept = 0u;
      while (m && left > 0) {
        const uint32_t bit = m & (0u - m);
        kept |= bit;
        m ^= bit;
        --left;
      }
      am[wd] = kept;
    }
    n_routed = n_pre;
  }
  const int n_act = n_routed + ((p.li == 0 && !pre) ? p.n_shared : 0);
  const int kc1 = p.H / (kBK * kAtoms);   // K-chunks (stages) of a gate/up tile
  const int kpe = (tpe + kAtoms - 1) / kAtoms;   // K-chunks (stages) per expert in the down phase
  const int h_tiles = p.H / kTileM;  // output tiles of the down phase
  const uint32_t b_atom_bytes = static_cast<uint32_t>(p.n_pad) * kBK * 2;   // one atom of the activation chunk
  const uint32_t b_bytes = kAtoms * b_atom_bytes;
  if (pre) {
    if (threadIdx.x == kThreads - 32) {            // segment 0: the pre-streamed experts' tiles, one whole tile per CTA
      Segment sg0 = Segment{1, 1, 0, n_pre * tpe, 0, 0, 0, p.d_kc1, 0};
      bars->plan.seg[0] = sg0;
      bars->plan.range[0] = make_range(sg0, cta, p.d_grid, h_tiles);
      bars->plan.n_pre = n_pre;
      bars->plan.n_seg = 1;
    }
  } else if (warp == kThreads / 32 - 1 && lane < 4) {      // (the publisher warp has nothing else to do yet)
    if (lane == 0) bars->n_routed_slots = n_routed;
    plan_lane(bars->plan, lane, cta, n_act, tpe, G, p.d_kc1, kpe, p.d_grid, p.d_tpe, h_tiles);
  }
  int32_t* s_entry = bars->entry;
  if (threadIdx.x < kMaxExperts) {
    const int e = threadIdx.x, wd = e >> 5;
    const uint32_t mine = wd == 0 ? am[0] : wd == 1 ? am[1] : wd == 2 ? am[2] : am[3];
    if ((mine >> (e & 31)) & 1u) {
      int slot = __popc(mine & ((1u << (e & 31)) - 1u));
#pragma unroll
      for (int v = 0; v < kMaskWords; ++v) slot += v < wd ? __popc(am[v]) : 0;
      // where the expert's weights are: the layer's own tensors (resident), staging slot `slot` (copied in
      // for this block), or -- with an expert pool -- whichever pool slot holds it
      s_entry[slot] = p.slot_of ? make_entry(kSrcStaged, p.slot_of[e])
                                : p.li == 0 ? make_entry(kSrcRouted, e) : make_entry(kSrcStaged, slot);
      bars->expert[slot] = e;
    }
  } else if (p.li == 0 && !pre && threadIdx.x - kMaxExperts < p.n_shared) {
    const int i = threadIdx.x - kMaxExperts;
    s_entry[n_routed + i] = make_entry(kSrcShared, i);
    bars->expert[n_routed + i] = -1;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const Segment* seg = bars->plan.seg;
  const uint32_t tmem_base = bars->tmem_base;
  if (threadIdx.x == 0) ACM_STAMP(0);
  // Does segment si exist?  With a pre-segment the plan behind segment 0 arrives later (the helper warp opens
  // plan_ready); n_seg is read from shared memory every time.
  const int n_seg_fixed = bars->plan.n_seg;
  auto have_seg = [&](int si, bool wait_for_plan) -> bool {
    if (pre) {
      if (si == 1 && wait_for_plan && !mbar_wait(smem_u32(&bars->plan_ready), 0u, quit, kSitePlanReady)) return false;
      return si < bars->plan.n_seg;
    } else {
      return si < n_seg_fixed;
    }
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ weight producer
    // Streams every weight tile of this CTA (and the x chunk of gate/up stages).  It arms each
    // stage's barrier with the bytes of both operands; the activation chunk of a down stage is
    // added by the helper warp once that expert group is complete, so this stream never stalls on
    // it.  The loop is kept to a few instructions per stage: one thread pays every one of them.
    if (lane == 0) {
      const uint64_t pol_w = policy_evict_first(), pol_x = policy_evict_last();
      uint32_t s = 0, par = 0, n_armed = 0;
      bool ok = true;
      for (int si = 0; ok && have_seg(si, true); ++si) {
        const Segment sg = seg[si];
        if (sg.phase == 1) {
          Sched sc(bars->plan.range[si]);
          int tile, k0, k1;
          while (ok && sc.next(tile, k0, k1)) {
            const int a_of = static_cast<int>(fdiv(static_cast<unsigned>(sg.t0 + tile), p.d_tpe));
            const int32_t ent = s_entry[a_of];
            const int r0 = (sg.t0 + tile - a_of * tpe) * 64, eidx = entry_idx(ent);
            const CUtensorMap* gu = pick_map(entry_src(ent), &maps.gate_up, &maps.shared_gate_up, &maps.staged_gate_up);
            for (int kc = k0; kc < k1; ++kc) {
              if (!(ok = mbar_wait(smem_u32(&bars->empty[s]), par ^ 1u, quit, kSiteStageEmpty))) break;
              const uint32_t full = smem_u32(&bars->full[s]);
              const uint32_t sa = smem_u32(stage_base) + s * kStageBytes;
#if ACM_FFN_MX
              mbar_expect_tx(full, b_bytes);
              {
                const uint32_t rawb = smem_u32(&bars->raw[s]);
                mbar_expect_tx(rawb, kMxStageBytes);
                bulk_load_hint(sa, p.mx_gate_up + (static_cast<size_t>(eidx * tpe + (r0 >> 6)) * kc1 + kc) * kMxStageBytes,
                               kMxStageBytes, rawb, pol_w);
              }
#else
              mbar_expect_tx(full, kABytes + b_bytes);
              tma_load_5d(sa, gu, full, 0, r0, 0, kc * kAtoms, eidx, pol_w);   // 64 gate + 64 up rows, 2 atoms
#endif
              tma_load_3d(sa + kABytes, &x_map, full, 0, 0, kc * kAtoms, pol_x);
              ++n_armed;
              if (++s == kStages) { s = 0; par ^= 1u; }
            }
          }
        } else {
          Sched sc(bars->plan.range[si]);
          int ht, k0, k1;
          while (ok && sc.next(ht, k0, k1)) {
            const int q0 = static_cast<int>(fdiv(static_cast<unsigned>(k0), p.d_kpe));
            int a = sg.a0 + q0, ic = k0 - q0 * kpe;
            int32_t ent = s_entry[a];
            const CUtensorMap* dn = pick_map(entry_src(ent), &maps.down, &maps.shared_down, &maps.staged_down);
            int eidx = entry_idx(ent);
            for (int kc = k0; kc < k1; ++kc) {
              if (!(ok = mbar_wait(smem_u32(&bars->empty[s]), par ^ 1u, quit, kSiteStageEmpty))) break;
              const uint32_t full = smem_u32(&bars->full[s]);
              const uint32_t sa = smem_u32(stage_base) + s * kStageBytes;
#if ACM_FFN_MX
              mbar_expect_tx(full, b_bytes);
              {
                const uint32_t rawb = smem_u32(&bars->raw[s]);
                mbar_expect_tx(rawb, kMxStageBytes);
                bulk_load_hint(sa, p.mx_down + (static_cast<size_t>(eidx * h_tiles + ht) * kpe + ic) * kMxStageBytes,
                               kMxStageBytes, rawb, pol_w);
              }
#else
              mbar_expect_tx(full, kABytes + b_bytes);
              tma_load_4d(sa, dn, full, 0, ht * kTileM, ic * kAtoms, eidx, pol_w);
#endif
              bars->armed = ++n_armed;      // the helper warp may now add this stage's activation chunk
              if (++s == kStages) { s = 0; par ^= 1u; }
              if (++ic == kpe && kc + 1 < k1) {
                ic = 0;
                ent = s_entry[++a];
                dn = pick_map(entry_src(ent), &maps.down, &maps.shared_down, &maps.staged_down);
                eidx = entry_idx(ent);
              }
            }
          }
        }
      }
      // The block's activated-expert counts, by the thread that is done first (its copies are all issued
      // microseconds before the last epilogue): off the kernel's tail.
      if (p.stats && p.li == 0 && blockIdx.x == 0) {
        griddep_wait();                       // early start: the routing kernel is long complete
        int n_all = 0, n_stg = 0;
#pragma unroll
        for (int wd = 0; wd < kMaskWords; ++wd) {
          const uint32_t act = __ldcg(p.act_mask + wd);
          n_all += __popc(act);
          n_stg += p.resident ? __popc(act & ~p.resident[wd]) : 0;
        }
        p.stats->n_activated = n_all;
        p.stats->n_staged = n_stg;
        p.stats->n_streamed = bars->n_routed_slots;
      }
      if (!ok) {
        // giving up: let copies already in flight land before the CTA exits
        const unsigned long long t0 = global_timer();
        while (global_timer() - t0 < 200000ull) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = umma_idesc(p.n_pad);
      const uint64_t desc_hi = umma_smem_desc(0);
      uint32_t it = 0, f = 0;
      bool ok = true;
      for (int si = 0; ok && have_seg(si, true); ++si) {
        Sched sc(bars->plan.range[si]);
        int tile, k0, k1;
        while (ok && sc.next(tile, k0, k1)) {
          const uint32_t b = f % kAcc;
          if (!(ok = mbar_wait(smem_u32(&bars->tempty[b]), ((f / kAcc) & 1u) ^ 1u, quit, kSiteAccEmpty))) break;
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + b * kAccCols;
          for (int kc = k0; kc < k1; ++kc, ++it) {
            const uint32_t s = it % kStages, par = (it / kStages) & 1u;
            if (!(ok = mbar_wait(smem_u32(&bars->full[s]), par, quit, kSiteStageFull))) break;
            tc_fence_after();
            // descriptors: only the address field changes from stage to stage and atom to atom
            const uint32_t sa = smem_u32(stage_base) + s * kStageBytes;
#if !ACM_FFN_MX
            const uint64_t da0 = desc_hi | ((sa & 0x3ffffu) >> 4);
#endif
            const uint64_t db0 = desc_hi | (((sa + kABytes) & 0x3ffffu) >> 4);
#pragma unroll
            for (int at = 0; at < kAtoms; ++at) {
#pragma unroll
              for (int kk = 0; kk < kBK / 16; ++kk) {
#if ACM_FFN_MX
                // the expanded weights are in tensor memory: stage s, 8 columns per 16 K
                umma_bf16_ts(d_tmem, tmem_base + kAcc * kAccCols + s * kMxACols + (at * (kBK / 16) + kk) * 8,
                             db0 + (at * (b_atom_bytes >> 4) + 2 * kk), idesc, (kc > k0 || at > 0 || kk > 0) ? 1u : 0u);
#else
                umma_bf16(d_tmem, da0 + (at * (kAtomABytes >> 4) + 2 * kk), db0 + (at * (b_atom_bytes >> 4) + 2 * kk), idesc,
                          (kc > k0 || at > 0 || kk > 0) ? 1u : 0u);
#endif
              }
            }
            umma_commit(smem_u32(&bars->empty[s]));
          }
          if (!ok) break;
          umma_commit(smem_u32(&bars->tfull[b]));
          ++f;
        }
      }
      if (!ok) {
        // giving up: wait (bounded) for the MMAs already issued before TMEM is released
        umma_commit(smem_u32(&bars->drained));
        const unsigned long long t0 = global_timer();
        while (!mbar_try_wait(smem_u32(&bars->drained), 0) && global_timer() - t0 < 1000000ull) {}
      }
    }
  } else if (warp == 6) {
    // ------------------------------------------------------------------ helper warp
    // Keeps slow global round trips off the other roles' paths: (a) for each gate/up segment whose
    // last fragment is the head of a tile shared with later CTAs, waits for their fragments and sums
    // them into shared memory; (b) for each down segment, waits until every activation tile of its
    // expert group has been stored, then tells the producer.
    bool ok = true;
    int frag_uses = 0;
    uint32_t hs = 0, hidx = 0;   // ring slot and running index of the next stage, tracked through the gate/up stages too
    if (pre) {
      // While the others run the anchors' pre-segment: wait for the eligible set, give the other experts the
      // slots behind the pre-streamed ones (ascending id), append the shared experts, work out the rest of the
      // plan, and let everyone on.
      // eight words per block; lane l takes words l and l + 32 (blocks 0-3 and 4-7), the union goes to lanes 0..7
      bool seen = true;
      uint32_t half = 0u;
      {
        const uint32_t tag = static_cast<uint32_t>(p.sel_epoch) & 0xffffu;
        const int n_words = 2 * kMaskWords * p.sel_blocks;
#pragma unroll
        for (int part = 0; part < 2; ++part) {
          const int j = lane + 32 * part;
          if (j < n_words) {
            bool got = true;
            half |= poll_tagged_word(p.sel_flag + j, tag, p.wait_limit_ns, got);
            seen = seen && got;
          }
        }
        half |= __shfl_xor_sync(0xffffffffu, half, 8);
        half |= __shfl_xor_sync(0xffffffffu, half, 16);
      }
      const bool good = __all_sync(0xffffffffu, seen);
      uint32_t rest[kMaskWords];
      int n_rest = 0;
#pragma unroll
      for (int wd = 0; wd < kMaskWords; ++wd) {
        const uint32_t lo = __shfl_sync(0xffffffffu, half, 2 * wd), hi = __shfl_sync(0xffffffffu, half, 2 * wd + 1);
        rest[wd] = ((lo | (hi << 16)) & p.only[wd]) & ~am[wd];
        n_rest += __popc(rest[wd]);
      }
      if (good) {
        for (int e = lane; e < kMaxExperts; e += 32) {
          const int wd = e >> 5;
          const uint32_t mine = wd == 0 ? rest[0] : wd == 1 ? rest[1] : wd == 2 ? rest[2] : rest[3];
          if ((mine >> (e & 31)) & 1u) {
            int slot = n_pre + __popc(mine & ((1u << (e & 31)) - 1u));
#pragma unroll
            for (int w2 = 0; w2 < kMaskWords; ++w2) slot += w2 < wd ? __popc(rest[w2]) : 0;
            s_entry[slot] = make_entry(kSrcRouted, e);
            bars->expert[slot] = e;
          }
        }
        if (lane < p.n_shared) {
          s_entry[n_pre + n_rest + lane] = make_entry(kSrcShared, lane);
          bars->expert[n_pre + n_rest + lane] = -1;
        }
        if (lane == 0) bars->n_routed_slots = n_pre + n_rest;
        if (lane < 4)
          plan_lane(bars->plan, lane, cta, n_pre + n_rest + p.n_shared, tpe, G, p.d_kc1, kpe, p.d_grid, p.d_tpe, h_tiles,
                    n_pre, 1);
      } else if (lane == 0) {
        give_up(quit, kSiteEligibleWords);
      }
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(smem_u32(&bars->plan_ready));
      }
      ok = good;
    }
    for (int si = 0; ok && have_seg(si, false); ++si) {
      const Segment sg = seg[si];
      const int n_exp = sg.a1 - sg.a0;
      if (sg.phase == 1) {
        hidx += bars->plan.range[si].n_stages;
        hs = hidx % kStages;
        if (sg.whole) continue;          // whole tiles: nothing to exchange
        const unsigned ub = cut_begin(sg, cta, p.d_grid), ue = cut_begin(sg, cta + 1, p.d_grid);
        if (ue <= ub) continue;
        const unsigned last_tile = fdiv(ue - 1, p.d_kc1);
        const unsigned tile_end = (last_tile + 1) * kc1;
        const bool head = (last_tile * kc1 >= ub) && (ue < tile_end);   // starts at chunk 0, ends before the tile does
        if (!head) continue;
        int n_contrib = 0;
        for (int c2 = cta + 1; c2 < G; ++c2) {
          const unsigned b2 = cut_begin(sg, c2, p.d_grid), e2 = cut_begin(sg, c2 + 1, p.d_grid);
          if (b2 >= tile_end) break;
          if (e2 > b2) ++n_contrib;
        }
        // one fragment buffer and one arrival counter per column half of the tile (a wide tile has two)
        for (int h = 0; h < n_halves && ok; ++h) {
          if (frag_uses > 0) {   // the buffer in shared memory still holds the previous sum until the epilogue has read it
            ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->frag_free), (frag_uses - 1) & 1u, quit, kSiteFragFree));
            if (!ok) break;
          }
          float* frag = p.frag + ((static_cast<size_t>(sg.p1_index) * G + cta) * 2 + h) * kFragFloats;   // this CTA's buffer
          int32_t* arrived = p.frag_flag + (sg.p1_index * G + cta) * 2 + h;
          const int n_el = min(p.n_pad - h * kMaxNodes, kMaxNodes) * kTileM;
          // every CTA holding a later part of the tile has reduce-added its fragment: one bulk copy
          bool got = true;
          if (lane == 0) got = flag_wait_ge(arrived, n_contrib, quit, kSiteFragArrivals);
          ok = __all_sync(0xffffffffu, got);
          if (!ok) break;
          if (lane == 0) {
            fence_proxy_async();
            const uint32_t hb = smem_u32(&bars->helper);
            mbar_expect_tx(hb, static_cast<uint32_t>(n_el) * 4u);
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_u32(sfrag)), "l"(frag), "r"(static_cast<uint32_t>(n_el) * 4u), "r"(hb) : "memory");
          }
          ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->helper), frag_uses & 1u, quit, kSiteFragCopy));
          if (!ok) break;
          if (lane == 0) mbar_arrive(smem_u32(&bars->frag_full));
          // leave the buffer and its counter zero for the next launch
          float4* z4 = reinterpret_cast<float4*>(frag);
          for (int i = lane; i < n_el / 4; i += 32) z4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (lane == 0) *arrived = 0;
          ++frag_uses;
        }
        if (!ok) break;
      } else {
        // activation producer: once every activation tile of this expert group is stored, add the
        // activation chunk of each down stage to the barrier the weight producer has armed (or will arm)
        bool good = true;
        {
          // The experts whose activation tiles this CTA's share of the segment reads (one finished-tile counter
          // per expert), polled side by side, one lane each: from the first to the last K-chunk of the share, or
          // the whole group if the share runs on into the next output tile.
          const SegRange& rg = bars->plan.range[si];
          const unsigned n_units = rg.u_end - rg.u;
          if (n_units > 0) {
            int q_lo = 0, q_hi = n_exp - 1;
            if (static_cast<unsigned>(rg.k00) + n_units <= static_cast<unsigned>(rg.kc)) {
              q_lo = static_cast<int>(fdiv(static_cast<unsigned>(rg.k00), p.d_kpe));
              q_hi = static_cast<int>(fdiv(static_cast<unsigned>(rg.k00) + n_units - 1u, p.d_kpe));
            }
            for (int q = q_lo + lane; q <= q_hi && good; q += 32)
              good = flag_wait_ge(&p.ready[sg.a0 + q], tpe * n_halves, quit, kSiteExpertReady);
          }
          good = __all_sync(0xffffffffu, good);
        }
        if (good && lane == 0) {
          const uint64_t pol_x = policy_evict_last();
          Sched sc(bars->plan.range[si]);
          int ht, k0, k1;
          fence_proxy_async();
          while (good && sc.next(ht, k0, k1)) {
            const int q0 = static_cast<int>(fdiv(static_cast<unsigned>(k0), p.d_kpe));
            int a = sg.a0 + q0, ic = k0 - q0 * kpe;
            for (int kc = k0; kc < k1; ++kc) {
              // never ahead of the weight producer: it has found the slot free and armed the barrier
              if (bars->armed <= hidx) {
                const unsigned long long t0 = global_timer();
                while (bars->armed <= hidx) {
                  if (quit->flag) { good = false; break; }
                  if (limit_passed(t0, p.wait_limit_ns)) {
                    give_up(quit, kSiteStageArmed);
                    good = false;
                    break;
                  }
                }
                if (!good) break;
              }
              tma_load_4d(smem_u32(stage_base) + hs * kStageBytes + kABytes, &h_map, smem_u32(&bars->full[hs]),
                          0, 0, ic * kAtoms, a, pol_x);
              ++hidx;
              if (++hs == kStages) hs = 0;
              if (++ic == kpe) { ic = 0; ++a; }
            }
          }
        }
        ok = __all_sync(0xffffffffu, good);
      }
    }
  } else if (warp == 7) {
    // ------------------------------------------------------------------ publisher
    // Moves what the epilogue staged in shared memory to global memory with bulk copies, waits for
    // them to complete and only then announces them (fragment flag / finished-tile counter).
    if (lane == 0) {
      uint32_t ost_n = 0, fin_n = 0;
      bool ok = true;
      for (int si = 0; ok && have_seg(si, true); ++si) {
        const Segment sg = seg[si];
        if (sg.phase != 1) continue;
        float* frag = p.frag + static_cast<size_t>(sg.p1_index) * G * 2 * kFragFloats;
        int32_t* frag_flag = p.frag_flag + sg.p1_index * G * 2;
        Sched sc(bars->plan.range[si]);
        int tile, k0, k1;
        while (ok && sc.next(tile, k0, k1)) {
         for (int h = 0; h < n_halves && ok; ++h) {          // a wide tile comes in two column halves
          if (k0 > 0) {
            if (!(ok = mbar_wait(smem_u32(&bars->ost_full), ost_n & 1u, quit, kSiteOutStaged))) break;
            const uint32_t bytes = static_cast<uint32_t>(min(p.n_pad - h * kMaxNodes, kMaxNodes)) * kTileM * 4u;
            // All CTAs that hold a tail part of this tile add into ONE global buffer, that of the CTA
            // which owns the tile's first chunks and will finish it.  The buffers are zero between
            // launches (the finishing CTA clears its own after reading), so nobody waits for anybody.
            const unsigned tile_begin = static_cast<unsigned>(tile) * kc1;
            int c_head = cta - 1;
            while (c_head > 0 && cut_begin(sg, c_head, p.d_grid) > tile_begin) --c_head;   // owner of the tile's first chunk
            asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.f32 [%0], [%1], %2;"
                         ::"l"(frag + static_cast<size_t>(c_head * 2 + h) * kFragFloats), "r"(smem_u32(ostage)), "r"(bytes) : "memory");
            bulk_commit();
            bulk_wait_all();
            red_release_add(&frag_flag[c_head * 2 + h], 1);
            mbar_arrive(smem_u32(&bars->ost_free));
            ++ost_n;
          } else {
            const uint32_t hb = fin_n & 1u;
            if (!(ok = mbar_wait(smem_u32(&bars->hst_full[hb]), (fin_n >> 1) & 1u, quit, kSiteActStaged))) break;
            const int a = static_cast<int>(fdiv(static_cast<unsigned>(sg.t0 + tile), p.d_tpe)), ti = sg.t0 + tile - a * tpe;
            asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%1, %2, %3, %4}], [%5];"
                         ::"l"(&hs_map), "r"(0), "r"(h * kMaxNodes), "r"(ti), "r"(a), "r"(smem_u32(hstage + hb * kHStageBytes)) : "memory");
            bulk_commit();
            bulk_wait_all();
            red_release_add(&p.ready[a], 1);
            mbar_arrive(smem_u32(&bars->hst_free[hb]));
            ++fin_n;
          }
         }
        }
      }
    }
#if ACM_FFN_MX
  } else if (warp >= 8) {
    // ------------------------------------------------------------------ expanding warps (MXFP4 -> bf16)
    // Thread r owns weight-tile row r = lane r of tensor memory.  Per stage: wait for the packed copy, take
    // the row's 64 code bytes and 4 scale bytes from shared memory, expand them to 128 bf16 in registers and
    // store those into the stage's 64 columns of tensor memory, from where the MMAs take their A operand --
    // the expanded tile never passes through shared memory.
    // A code is sign | 2 exponent bits | 1 mantissa bit with subnormals: put at bits 15 | 8:7 | 6 of a bf16 it
    // is the value times 2^-126 exactly, so one bf16 multiply by 2^(scale byte - 1) finishes the job.
    const int r = threadIdx.x - 256;
    const uint32_t my_lane = static_cast<uint32_t>(r & ~31) << 16;          // this warp's quarter of the lanes
    bool ok = true;
    // the row's packed data of the stage at hand
    uint4 q[4];
    uint32_t sc = 0;
    auto fetch = [&](unsigned it) -> bool {
      const uint32_t s = it % kStages, par = (it / kStages) & 1u;
      if (!mbar_wait(smem_u32(&bars->raw[s]), par, quit, kSitePackedStage)) return false;
      const unsigned char* A = stage_base + static_cast<size_t>(s) * kStageBytes;
      // (the record keeps the row's four 16-byte pieces rotated by the row number, so that a warp's loads
      // spread over all banks)
#pragma unroll
      for (int b = 0; b < 4; ++b) q[b] = *reinterpret_cast<const uint4*>(A + r * 64 + 16 * (b ^ ((r >> 1) & 3)));
      sc = *reinterpret_cast<const uint32_t*>(A + kMxCodeBytes + r * 4);
      return true;
    };
    // stage by stage through the segments (with the anchors' pre-segment the later ones arrive behind plan_ready)
    unsigned it = 0, total = 0;
    bool fetched = false;
    for (int si = 0; ok && have_seg(si, true); ++si) {
     total += bars->plan.range[si].n_stages;
     if (!fetched && it < total) { ok = fetch(it); fetched = true; }
     for (; it < total && ok; ++it) {
      const uint32_t s = it % kStages;
      const uint32_t a_tmem = tmem_base + my_lane + kAcc * kAccCols + s * kMxACols;
      tc_fence_after();
#pragma unroll
      for (int b = 0; b < 4; ++b) {                     // 32 K = one scale = 16 columns
        const uint32_t field = min(((sc >> (8 * b)) & 0xffu) + 126u, 254u) << 7;
        const uint32_t c2 = field | (field << 16);
        const uint32_t words[4] = {q[b].x, q[b].y, q[b].z, q[b].w};
        uint32_t o[16];
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          // a word holds elements 2j (nibble j) and 2j+1 (nibble 4+j): pairs 0 and 1 are masked out where they
          // sit -- the multiplier that moves magnitude and sign into place differs -- pairs 2 and 3 after one shift
          const uint32_t w2 = words[w] >> 8;
          const uint32_t e0 = ((words[w] & 0x000f000fu) * 0x1040u) & 0x81c081c0u;
          const uint32_t e1 = ((words[w] & 0x00f000f0u) * 0x0104u) & 0x81c081c0u;
          const uint32_t e2 = ((w2 & 0x000f000fu) * 0x1040u) & 0x81c081c0u;
          const uint32_t e3 = ((w2 & 0x00f000f0u) * 0x0104u) & 0x81c081c0u;
          asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(o[4 * w + 0]) : "r"(e0), "r"(c2));
          asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(o[4 * w + 1]) : "r"(e1), "r"(c2));
          asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(o[4 * w + 2]) : "r"(e2), "r"(c2));
          asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(o[4 * w + 3]) : "r"(e3), "r"(c2));
        }
        tmem_st16(a_tmem + 16 * b, o);
      }
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->full[s]));
      if (it + 1 < total) ok = fetch(it + 1); else fetched = false;
     }
    }
#endif
  } else {
    // ------------------------------------------------------------------ epilogue (128 threads)
    // On-chip work only: accumulators -> registers -> shared memory.  Everything that has to reach
    // global memory and be announced to other CTAs (fragments, activation tiles) is staged in shared
    // memory and handed to the publisher warp, so these warps never sit in a memory fence.
    const int quarter = warp & 3;               // TMEM lanes this warp may read
    const int row = quarter * 32 + lane;        // accumulator row = weight-tile row
    const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
    uint32_t f = 0, ost_uses = 0, fin_count = 0, frag_reads = 0;
    bool ok = true, waited = !early;
    float v[kMaxNodes];
    // one half (up to 64 columns from column `cb` on) of accumulator b; the accumulator is released with its last half
    auto load_half = [&](uint32_t b, int cb, int np, bool release) {
#pragma unroll
      for (int c = 0; c < kMaxNodes; c += 16)
        if (c < np) tmem_ld16(tmem_base + lane_addr + b * kAccCols + cb + c, v + c);
      tmem_ld_wait();
      if (release) {
        tc_fence_before();
        mbar_arrive(smem_u32(&bars->tempty[b]));
      }
    };
    // the outgoing-fragment buffer (and the exchange buffer aliasing it) is free once the publisher
    // has copied the previous fragment out
    auto wait_ostage = [&]() -> bool {
      if (ost_uses == 0) return true;
      return epi_vote_all(mbar_wait(smem_u32(&bars->ost_free), (ost_uses - 1) & 1u, quit, kSiteOutFree));
    };
    for (int si = 0; ok && have_seg(si, true); ++si) {
      const Segment sg = seg[si];
      if (sg.phase == 1) {
        Sched sc(bars->plan.range[si]);
        int tile, k0, k1;
        while (ok && sc.next(tile, k0, k1)) {
          const uint32_t b = f % kAcc;
          // A tile this CTA will finish needs its expert's combine weights: fetch them (one L2 round
          // trip) while the tile's MMAs run, not after them.  They are the routing kernel's last output.
          float wd_mine = 0.0f;
          const int a = static_cast<int>(fdiv(static_cast<unsigned>(sg.t0 + tile), p.d_tpe));
          if (k0 == 0) {
            if (!waited) {
              griddep_wait();
              waited = true;
            }
            if (row < p.n_pad) {
              const int ex_id = bars->expert[a];      // the table row of a routed expert, 1 for a shared one
              wd_mine = ex_id >= 0 ? __ldcg(p.wtab + static_cast<size_t>(ex_id) * kWtabStride + row) : (row < p.T ? 1.0f : 0.0f);
            }
          }
          ok = epi_vote_all(mbar_wait(smem_u32(&bars->tfull[b]), (f / kAcc) & 1u, quit, kSiteAccFull));
          if (!ok) break;
          tc_fence_after();
          ++f;
          if (k0 == 0 && row < p.n_pad) bars->wd[row] = wd_mine;
          for (int h = 0; h < n_halves && ok; ++h) {
            const int cb = h * kMaxNodes;                              // first node column of this half
            const int np = min(p.n_pad - cb, kMaxNodes);               // its columns (a multiple of 16)
            load_half(b, cb, np, h == n_halves - 1);
            if (k0 > 0) {
              // tail part of a tile whose first chunks belong to an earlier CTA: stage the fragment
              if (!(ok = wait_ostage())) break;
#pragma unroll
              for (int c = 0; c < kMaxNodes; ++c)
                if (c < np) ostage[c * kTileM + row] = v[c];
              fence_proxy_async_smem();
              mbar_arrive(smem_u32(&bars->ost_full));
              ++ost_uses;
              continue;
            }
            if (k1 < kc1) {
              // head part: the helper warp has summed the other CTAs' fragments of this tile (half) into smem
              ok = epi_vote_all(mbar_wait(smem_u32(&bars->frag_full), frag_reads & 1u, quit, kSiteFragFull));
              if (!ok) break;
#pragma unroll
              for (int c = 0; c < kMaxNodes; ++c)
                if (c < np) v[c] += sfrag[c * kTileM + row];
              mbar_arrive(smem_u32(&bars->frag_free));
              ++frag_reads;
            }
            // rows 0..63 hold gate, rows 64..127 the matching up projections.  Each pair of threads
            // (i, i+64) splits the node columns: the gate thread finishes columns [0, 32), the up
            // thread columns [32, 64); they swap the halves they do not finish through smem.
            constexpr int kHalf = kMaxNodes / 2;
            const int feat = row & 63;
            if (!(ok = wait_ostage())) break;
            if (quarter >= 2) {
#pragma unroll
              for (int c = 0; c < kHalf; ++c)
                if (c < np) ex[c * 64 + feat] = v[c];
            } else {
#pragma unroll
              for (int c = kHalf; c < kMaxNodes; ++c)
                if (c < np) ex[c * 64 + feat] = v[c];
            }
            const uint32_t hb = fin_count & 1u;
            bool hst_ok = true;
            if (fin_count >= 2) hst_ok = mbar_wait(smem_u32(&bars->hst_free[hb]), ((fin_count >> 1) - 1) & 1u, quit, kSiteActFree);
            ok = epi_vote_all(hst_ok);      // also orders the exchange writes above before the reads below
            if (!ok) break;
            {
              unsigned char* hs = hstage + hb * kHStageBytes;
              const int c0 = quarter < 2 ? 0 : kHalf;
#pragma unroll
              for (int j0 = 0; j0 < kHalf; j0 += 8) {
                if (c0 + j0 < np) {           // np is a multiple of 16: a block of 8 columns is all in or all out
                  float other[8], wgt[8], hval[8];
#pragma unroll
                  for (int j = 0; j < 8; ++j) {
                    other[j] = ex[(c0 + j0 + j) * 64 + feat];
                    wgt[j] = bars->wd[cb + c0 + j0 + j];
                  }
#pragma unroll
                  for (int j = 0; j < 8; ++j) {
                    const float mine = quarter < 2 ? v[j0 + j] : v[kHalf + j0 + j];
                    const float g = quarter < 2 ? mine : other[j];
                    const float u = quarter < 2 ? other[j] : mine;
                    // w * u * silu(g), silu(g) = g/2 * (1 + tanh(g/2))
                    const float hg = 0.5f * g;
                    float th;
                    asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(hg));
                    const float q = wgt[j] * u * hg;
                    hval[j] = fmaf(q, th, q);
                  }
                  // activation tile [node][64 features] bf16 in the 128-byte-swizzled layout of its TMA store
#pragma unroll
                  for (int j = 0; j < 8; ++j) {
                    const int t = c0 + j0 + j;
                    const int off = t * 128 + ((((feat >> 3) ^ (t & 7))) << 4) + ((feat & 7) << 1);
                    *reinterpret_cast<__nv_bfloat16*>(hs + off) = __float2bfloat16_rn(hval[j]);
                  }
                }
              }
              fence_proxy_async_smem();
              mbar_arrive(smem_u32(&bars->hst_full[hb]));
              ++fin_count;
            }
          }
        }
        if (row == 0) ACM_STAMP(10);
      } else {
        Sched sc(bars->plan.range[si]);
        int ht, k0, k1;
        while (ok && sc.next(ht, k0, k1)) {
          const uint32_t b = f % kAcc;
          ok = epi_vote_all(mbar_wait(smem_u32(&bars->tfull[b]), (f / kAcc) & 1u, quit, kSiteAccFull));
          if (!ok) break;
          tc_fence_after();
          ++f;
          for (int h = 0; h < n_halves; ++h) {
            const int cb = h * kMaxNodes;
            load_half(b, cb, min(p.n_pad - cb, kMaxNodes), h == n_halves - 1);
            float* dst = p.out + static_cast<size_t>(cb) * p.H + static_cast<size_t>(ht) * kTileM + row;
#pragma unroll
            for (int c = 0; c < kMaxNodes; ++c)
              if (cb + c < p.T) atomicAdd(dst + static_cast<size_t>(c) * p.H, v[c]);
          }
        }
        if (row == 0) ACM_STAMP(11);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

#if !ACM_FFN_MX
// ---------------------------------------------------------------------------------- f32 path
// h[t][j][i] = silu(g) * u for routed slot j < k (expert idx[t][j]) and shared slot j >= k.
__global__ void k_ffn_f32_gate_up(const float* __restrict__ x, const float* __restrict__ gate_up,
                                  const float* __restrict__ shared_gate_up, const int32_t* __restrict__ idx,
                                  float* __restrict__ hbuf, int T, int H, int I, int E, int k, int n_shared) {
  const int slots = k + n_shared;
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= T * slots * I) return;
  const int i = warp % I, j = (warp / I) % slots, t = warp / (I * slots);
  int e = j < k ? idx[t * k + j] : j - k;
  if (j < k && e >= E) e = -1;                 // an id outside the layer is an empty slot, like -1
  const float* base = j < k ? gate_up : shared_gate_up;
  float h = 0.0f;
  if (e >= 0) {
    const float* g_row = base + (static_cast<size_t>(e) * 2 * I + i) * H;
    const float* u_row = g_row + static_cast<size_t>(I) * H;
    const float* xr = x + static_cast<size_t>(t) * H;
    float g = 0.f, u = 0.f;
    for (int hh = lane; hh < H; hh += 32) {
      g = fmaf(g_row[hh], xr[hh], g);
      u = fmaf(u_row[hh], xr[hh], u);
    }
    for (int s = 16; s >= 1; s >>= 1) {
      g += __shfl_xor_sync(0xffffffffu, g, s);
      u += __shfl_xor_sync(0xffffffffu, u, s);
    }
    h = (g / (1.0f + expf(-g))) * u;
  }
  if (lane == 0) hbuf[(static_cast<size_t>(t) * slots + j) * I + i] = h;
}

__global__ void k_ffn_f32_down(const float* __restrict__ down, const float* __restrict__ shared_down,
                               const int32_t* __restrict__ idx, const float* __restrict__ w,
                               const float* __restrict__ hbuf, float* __restrict__ out, int T, int H, int I,
                               int E, int k, int n_shared) {
  const int slots = k + n_shared;
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= T * H) return;
  const int hh = warp % H, t = warp / H;
  float y = 0.f;
  for (int j = 0; j < slots; ++j) {
    const int e = j < k ? idx[t * k + j] : j - k;
    if (e < 0 || (j < k && e >= E)) continue;
    const float* d_row = (j < k ? down : shared_down) + (static_cast<size_t>(e) * H + hh) * I;
    const float* hr = hbuf + (static_cast<size_t>(t) * slots + j) * I;
    float acc = 0.f;
    for (int i = lane; i < I; i += 32) acc = fmaf(d_row[i], hr[i], acc);
    for (int s = 16; s >= 1; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
    y += (j < k ? w[t * k + j] : 1.0f) * acc;
  }
  if (lane == 0) out[static_cast<size_t>(t) * H + hh] = y;
}

#endif   // !ACM_FFN_MX

}  // namespace

#if ACM_FFN_MX
cudaError_t ffn_mx_configure() {
  return cudaFuncSetAttribute(ACM_FFN_KERNEL<kMaxNodes>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              static_cast<int>(Geo<kMaxNodes>::kSmemBytes));
}
cudaError_t launch_ffn_mxfp4(const FfnLaunch& L, const FfnMaps& maps, const CUtensorMap& x_map,
                             const CUtensorMap& h_map, const CUtensorMap& hs_map, cudaStream_t s) {
#else

cudaError_t ffn_configure() {
  cudaError_t err = cudaFuncSetAttribute(ACM_FFN_KERNEL<kMaxNodes>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(Geo<kMaxNodes>::kSmemBytes));
  if (err != cudaSuccess) return err;
  return cudaFuncSetAttribute(ACM_FFN_KERNEL<kWideNodes>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              static_cast<int>(Geo<kWideNodes>::kSmemBytes));
}

cudaError_t launch_ffn_bf16(const FfnLaunch& L, const FfnMaps& maps, const CUtensorMap& x_map,
                            const CUtensorMap& h_map, const CUtensorMap& hs_map, cudaStream_t s) {
#endif
  {
    // the schedules count (tile, K-chunk) units times the grid in 32 bits
    const unsigned long long u1 = static_cast<unsigned long long>(kMaxSlots) * (L.I / 64) * (L.H / (kBK * kAtoms));
    const unsigned long long u2 = static_cast<unsigned long long>(L.H / kTileM) * kMaxSlots * ((L.I / 64 + kAtoms - 1) / kAtoms);
    if ((u1 > u2 ? u1 : u2) * (static_cast<unsigned long long>(L.grid) + 1) >= (1ull << 32)) return cudaErrorInvalidValue;
  }
  FfnArgs a;
  {
    const int tpe = L.I / 64;
    a.d_grid = make_fastdiv(static_cast<unsigned>(L.grid));
    a.d_kc1 = make_fastdiv(static_cast<unsigned>(L.H / (kBK * kAtoms)));
    a.d_tpe = make_fastdiv(static_cast<unsigned>(tpe));
    a.d_kpe = make_fastdiv(static_cast<unsigned>((tpe + kAtoms - 1) / kAtoms));
  }
  a.T = L.T; a.H = L.H; a.I = L.I; a.n_pad = L.n_pad;
  a.act_mask = L.act_mask; a.resident = L.resident; a.li = L.li; a.n_shared = L.n_shared; a.slot_of = L.slot_of; a.wtab = L.wtab;
  for (int w = 0; w < 4; ++w) a.only[w] = L.only[w];
  a.stats = L.stats; a.hbuf = static_cast<__nv_bfloat16*>(L.hbuf);
  a.ready = L.ready; a.frag = L.frag; a.frag_flag = L.frag_flag;
  a.sel_flag = L.sel_flag; a.sel_epoch = L.sel_epoch; a.sel_blocks = L.sel_blocks;
  a.anc_flag = (L.sel_blocks < 1 || L.sel_blocks > kMaxEarlyBlocks || L.li != 0 || L.resident || L.slot_of) ? nullptr : L.anc_flag;
  a.out = L.out; a.status = L.status; a.trace = L.trace;
  a.wait_limit_ns = L.wait_limit_ns; a.wait_diag = L.wait_diag; a.launch_tag = L.launch_tag;
#if ACM_FFN_MX
  if (!L.mx_gate_up || !L.mx_down || L.I % 128 != 0 || L.n_shared != 0) return cudaErrorInvalidValue;
  a.mx_gate_up = static_cast<const unsigned char*>(L.mx_gate_up);
  a.mx_down = static_cast<const unsigned char*>(L.mx_down);
#endif
  void* args[] = {const_cast<FfnMaps*>(&maps), const_cast<CUtensorMap*>(&x_map), const_cast<CUtensorMap*>(&h_map),
                  const_cast<CUtensorMap*>(&hs_map), &a};
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(L.grid);
  cfg.blockDim = dim3(kThreads);
#if ACM_FFN_MX
  if (L.n_pad > kMaxNodes) return cudaErrorInvalidValue;
  const bool wide = false;
#else
  const bool wide = L.n_pad > kMaxNodes;       // a batch with more than 64 nodes: 128-column accumulators
  if (L.n_pad > kWideNodes) return cudaErrorInvalidValue;
#endif
  cfg.dynamicSmemBytes = wide ? Geo<kWideNodes>::kSmemBytes : Geo<kMaxNodes>::kSmemBytes;
  cfg.stream = s;
  // The CTAs wait on one another, so all of them must be resident: one CTA per SM on an otherwise
  // idle GPU is, and a cooperative launch makes the driver check it.  A dependent launch cannot be
  // cooperative (its CTAs trickle in behind the previous kernel's); there the waits' limits, which
  // end in an error status instead of a hang, are the guard.
  cudaLaunchAttribute attr[1];
  if (L.pdl) {
    set_pdl_attr(&attr[0]);
  } else {
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
  }
  cfg.attrs = attr;
  cfg.numAttrs = 1;
#if ACM_FFN_MX
  return cudaLaunchKernelExC(&cfg, reinterpret_cast<const void*>(ACM_FFN_KERNEL<kMaxNodes>), args);
#else
  return cudaLaunchKernelExC(&cfg, wide ? reinterpret_cast<const void*>(ACM_FFN_KERNEL<kWideNodes>)
                                        : reinterpret_cast<const void*>(ACM_FFN_KERNEL<kMaxNodes>), args);
#endif
}

#if !ACM_FFN_MX
cudaError_t launch_ffn_f32(const float* x, const float* gate_up, const float* down,
                           const float* shared_gate_up, const float* shared_down, int n_shared,
                           const int32_t* idx, const float* w, float* hbuf, float* out, int T, int H,
                           int I, int E, int k, cudaStream_t s) {
  const int slots = k + n_shared;
  const long long warps1 = static_cast<long long>(T) * slots * I;
  k_ffn_f32_gate_up<<<static_cast<unsigned>((warps1 * 32 + 255) / 256), 256, 0, s>>>(x, gate_up, shared_gate_up, idx, hbuf,
                                                                                   T, H, I, E, k, n_shared);
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  const long long warps2 = static_cast<long long>(T) * H;
  k_ffn_f32_down<<<static_cast<unsigned>((warps2 * 32 + 255) / 256), 256, 0, s>>>(down, shared_down, idx, w, hbuf, out, T,
                                                                                H, I, E, k, n_shared);
  return cudaGetLastError();
}

#endif   // !ACM_FFN_MX

}  // namespace acm

#if !ACM_FFN_MX
// ------------------------------------------------------------------------------------------------
// Allocation-free variant of the f32 expert FFN.  The per-(node, slot) intermediate activations that
// the context-based call keeps in its cudaMalloc'ed workspace live here in a fixed array that is part
// of the library image, so the call never allocates.
// ------------------------------------------------------------------------------------------------
namespace {
constexpr size_t kNoAllocScratchFloats = ACM_NOALLOC_MAX_FLOATS;
static __device__ __align__(256) float g_noalloc_scratch[kNoAllocScratchFloats];

constexpr int kNoAllocMaxDevices = 64;
std::mutex g_noalloc_mutex;
float* g_noalloc_ptr[kNoAllocMaxDevices];   // device address of the array above, per device (0 = not looked up yet)
}  // namespace

extern "C" acm_status acm_expert_ffn_f32_noalloc(const float* x, int T, int hidden, int inter, int n_experts, int top_k,
                                                 const int32_t* idx, const float* w, const float* w_gate_up,
                                                 const float* w_down, float* out, acm_stream stream) {
  if (!x || !idx || !w || !w_gate_up || !w_down || !out) return ACM_ERR_INVALID;
  if (T < 1 || hidden < 1 || inter < 1 || n_experts < 1 || top_k < 1 || top_k > n_experts) return ACM_ERR_INVALID;
  if (T > acm::kMaxNodes || top_k > acm::kMaxTopK || n_experts > acm::kMaxExperts) return ACM_ERR_UNSUPPORTED;
  // the scratch holds one float per (node, slot, intermediate feature): refuse what does not fit
  if (static_cast<size_t>(T) * top_k * inter > kNoAllocScratchFloats) return ACM_ERR_UNSUPPORTED;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return ACM_ERR_CUDA;
  if (dev < 0 || dev >= kNoAllocMaxDevices) return ACM_ERR_UNSUPPORTED;
  float* scratch = nullptr;
  {
    // First call on this device: ask the runtime where this device's copy of the array lives.  In host
    // code the array's name is only a handle; a kernel must be given the address obtained here.
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return ACM_ERR_CUDA;
      g_noalloc_ptr[dev] = static_cast<float*>(p);
    }
    scratch = g_noalloc_ptr[dev];
  }
  const cudaError_t err = acm::launch_ffn_f32(x, w_gate_up, w_down, nullptr, nullptr, 0, idx, w, scratch, out, T, hidden,
                                              inter, n_experts, top_k, static_cast<cudaStream_t>(stream));
  return err == cudaSuccess ? ACM_OK : ACM_ERR_CUDA;
}
#endif   // !ACM_FFN_MX
