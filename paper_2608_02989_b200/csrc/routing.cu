// Stages 1-3 of the verifier-side MoE layer: router logits (Section 3.1), softmax and natural
// top-k (Eq. 1), commitment-weighted demand (Eq. 4), anchors (Eq. 5), self-sized eligible set
// (Eq. 6), residency-aware pruning (Eq. 7) and restricted top-k routing (Eq. 2), plus the
// routing inputs the FFN kernel consumes (activated-expert mask, combine-weight table).
//
// Everything that decides a set member, a count or an index is binary32 in a fixed order
// (explicit round-to-nearest intrinsics, so the compiler can neither contract nor reorder):
// 32 interleaved partial sums + halving tree for the logit dot product, a 128-slot halving
// tree for sums over the expert axis, fixed polynomial recipes for exp and log.
#include <cooperative_groups.h>
#include <cuda_bf16.h>

#include "acm_internal.h"

namespace acm {
namespace {

__device__ __forceinline__ long long time_ns() {     // one clock for every SM (the stamps of acm_stage_timing)
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return static_cast<long long>(t);
}
__device__ __forceinline__ void raise_status(int32_t* status, int code) {
  if (status) atomicCAS(status, 0, code);
}

// exp(x): x = n ln2 + r (two-term ln2), degree-7 Taylor polynomial, scale through the exponent field.
__device__ __forceinline__ float exp_fixed(float x) {
  x = fminf(fmaxf(x, -87.0f), 88.0f);
  const float n = rintf(__fmul_rn(x, 1.44269502162933349609375f));
  float r = __fmaf_rn(n, -0.693145751953125f, x);
  r = __fmaf_rn(n, -1.428606765330187045037746429443359375e-06f, r);
  float p = 1.98412701138295233249664306640625e-04f;
  p = __fmaf_rn(p, r, 1.388888922519981861114501953125e-03f);
  p = __fmaf_rn(p, r, 8.3333337679505348205566406250e-03f);
  p = __fmaf_rn(p, r, 4.16666679084300994873046875e-02f);
  p = __fmaf_rn(p, r, 0.16666667163372039794921875f);
  p = __fmaf_rn(p, r, 0.5f);
  p = __fmaf_rn(p, r, 1.0f);
  p = __fmaf_rn(p, r, 1.0f);
  const float scale = __int_as_float((static_cast<int>(n) + 127) << 23);
  return __fmul_rn(p, scale);
}

// log(q), q positive and normal: q = m 2^e, m in (sqrt(1/2), sqrt(2)], log m = 2 atanh((m-1)/(m+1)).
__device__ __forceinline__ float log_fixed(float q) {
  const int bits = __float_as_int(q);
  int e = ((bits >> 23) & 0xff) - 127;
  float m = __int_as_float((bits & 0x007fffff) | 0x3f800000);
  if (m > 1.41421353816986083984375f) {
    m = __fmul_rn(m, 0.5f);
    e += 1;
  }
  const float s = __fdiv_rn(__fsub_rn(m, 1.0f), __fadd_rn(m, 1.0f));
  const float s2 = __fmul_rn(s, s);
  float p = 9.0909093618392944335937500e-02f;
  p = __fmaf_rn(p, s2, 0.111111111938953399658203125f);
  p = __fmaf_rn(p, s2, 0.14285714924335479736328125f);
  p = __fmaf_rn(p, s2, 0.20000000298023223876953125f);
  p = __fmaf_rn(p, s2, 0.3333333432674407958984375f);
  p = __fmaf_rn(p, s2, 1.0f);
  const float lm = __fmul_rn(2.0f, __fmul_rn(s, p));
  return __fmaf_rn(static_cast<float>(e), 0.693147182464599609375f, lm);
}

// 32-bit orderable image of a float (larger float -> larger unsigned); 0 is below every real value.
__device__ __forceinline__ unsigned order_key(float z) {
  const unsigned u = __float_as_uint(z);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
// One round of a warp-wide top-k over 128 slots (slot e = lane + 32 c, key[c] == 0: not a candidate):
// returns the slot with the largest key, ties to the lowest slot, or -1 if none is left; the
// owning lane clears that key.  One hardware warp reduction (the maximum) and four independent votes per round: the
// lowest slot that holds the maximum is in the lowest c that has it anywhere, at the lowest such lane.
__device__ __forceinline__ int warp_take_best(unsigned (&key)[4], int lane) {
  const unsigned m01 = max(key[0], key[1]), m23 = max(key[2], key[3]);
  const unsigned best = __reduce_max_sync(0xffffffffu, max(m01, m23));
  if (best == 0u) return -1;
  const unsigned h0 = __ballot_sync(0xffffffffu, key[0] == best), h1 = __ballot_sync(0xffffffffu, key[1] == best);
  const unsigned h2 = __ballot_sync(0xffffffffu, key[2] == best), h3 = __ballot_sync(0xffffffffu, key[3] == best);
  const int c = h0 ? 0 : h1 ? 1 : h2 ? 2 : 3;
  const unsigned h = h0 ? h0 : h1 ? h1 : h2 ? h2 : h3;
  const int l = __ffs(h) - 1;
  if (l == lane) {
    key[0] = c == 0 ? 0u : key[0]; key[1] = c == 1 ? 0u : key[1];
    key[2] = c == 2 ? 0u : key[2]; key[3] = c == 3 ? 0u : key[3];
  }
  return 32 * c + l;
}

// Sum of a 128-slot array held as 4 values per lane (slot = lane + 32 c): the halving tree
// a[i] += a[i+s], s = 64, 32, 16, ..., 1.  Result broadcast to the whole warp.
__device__ __forceinline__ float warp_tree_sum_128(float a0, float a1, float a2, float a3) {
  float v = __fadd_rn(__fadd_rn(a0, a2), __fadd_rn(a1, a3));
#pragma unroll
  for (int s = 16; s >= 1; s >>= 1) v = __fadd_rn(v, __shfl_down_sync(0xffffffffu, v, s));
  return __shfl_sync(0xffffffffu, v, 0);
}

// Natural top-k of one logit row held in registers (lane l holds experts l, l + 32, l + 64, l + 96), ranked on the
// logits, ties to the lower index: the set as a bit mask (warp-uniform); the ranked ids go to `nat_row` if given.
__device__ __forceinline__ void topk_bits(const float (&z)[4], int E, int k, int lane, uint32_t (&bits)[kMaskWords],
                                          int32_t* nat_row) {
  unsigned key[4];
#pragma unroll
  for (int c = 0; c < 4; ++c) key[c] = (lane + 32 * c < E) ? order_key(z[c]) : 0u;
  uint32_t b0 = 0u, b1 = 0u, b2 = 0u, b3 = 0u;
  for (int j = 0; j < k; ++j) {
    const int e = warp_take_best(key, lane);
    if (nat_row && lane == 0) nat_row[j] = e;
    if (e >= 0) {
      const uint32_t bit = 1u << (e & 31);
      const int wd = e >> 5;
      b0 |= wd == 0 ? bit : 0u; b1 |= wd == 1 ? bit : 0u; b2 |= wd == 2 ? bit : 0u; b3 |= wd == 3 ? bit : 0u;
    }
  }
  bits[0] = b0; bits[1] = b1; bits[2] = b2; bits[3] = b3;
}

// Stage 1b for ONE node, by one warp, on a logit row held in registers (lane l holds experts l, l + 32, l + 64,
// l + 96; -inf beyond E): softmax over the expert axis (fixed recipe) and natural top-k ranked on the logits.
// Returns the probabilities in the same layout and the top-k set as a bit mask (warp-uniform); the ranked ids
// go to `nat_row` if given.
__device__ __forceinline__ void softmax_topk_regs(const float (&z)[4], int E, int k, int lane, float (&prob)[4],
                                                  uint32_t (&bits)[kMaskWords], int32_t* nat_row, bool want_topk) {
  float y[4];
  float zmax = fmaxf(fmaxf(z[0], z[1]), fmaxf(z[2], z[3]));
#pragma unroll
  for (int s = 16; s >= 1; s >>= 1) zmax = fmaxf(zmax, __shfl_xor_sync(0xffffffffu, zmax, s));
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const float ex = exp_fixed(__fsub_rn(z[c], zmax));
    y[c] = (lane + 32 * c < E) ? ex : 0.0f;
  }
  const float denom = warp_tree_sum_128(y[0], y[1], y[2], y[3]);
#pragma unroll
  for (int c = 0; c < 4; ++c) prob[c] = __fdiv_rn(y[c], denom);
  if (want_topk) {
    topk_bits(z, E, k, lane, bits, nat_row);
  } else {
    bits[0] = bits[1] = bits[2] = bits[3] = 0u;
  }
}

// The same for a row in global memory (`z_row` may have been written by other CTAs: read through L2).
__device__ void softmax_topk_row(const float* z_row, float* probs_row, int32_t* nat_row, uint32_t* natmask_row,
                                 int E, int k, int lane) {
  float z[4], prob[4];
  uint32_t bits[kMaskWords];
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const int e = lane + 32 * c;
    const float v = __ldcg(z_row + min(e, E - 1));
    z[c] = e < E ? v : -INFINITY;
  }
  softmax_topk_regs(z, E, k, lane, prob, bits, nat_row, nat_row != nullptr);
  if (probs_row) {
#pragma unroll
    for (int c = 0; c < 4; ++c)
      if (lane + 32 * c < E) probs_row[lane + 32 * c] = prob[c];
  }
  if (nat_row && natmask_row && lane < kMaskWords)
    natmask_row[lane] = lane == 0 ? bits[0] : lane == 1 ? bits[1] : lane == 2 ? bits[2] : bits[3];
}

// ------------------------------------------------------------------------------------------
// Stage 1a: router logits.  CTA tile = 4 nodes x 8 experts (many small CTAs: the whole GPU works on
// a 64 x 128 x 2048 product), rows staged in shared memory with 16-byte async copies in 4 K-chunks.
// One vector load covers EPT consecutive h, i.e. EPT of the 32 interleaved partial sums; Q = 32/EPT
// threads share one output.
// ------------------------------------------------------------------------------------------
constexpr int kRT = 4, kRE = 8;

template <typename Elem>
struct ElemTraits;
template <>
struct ElemTraits<float> {
  static constexpr int EPT = 4;
  using Vec = uint4;
  __device__ static void unpack(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
};
template <>
struct ElemTraits<__nv_bfloat16> {
  static constexpr int EPT = 4;
  using Vec = uint2;        // 8-byte loads, 8 threads per output: twice the warps to hide latency with
  __device__ static void unpack(const uint2& v, float* f) {
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
  }
};

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __uint_as_float(static_cast<unsigned>(__bfloat16_as_ushort(v)) << 16); }

// ---- bulk asynchronous copies (global -> shared) completing on an mbarrier ----
__device__ __forceinline__ unsigned smem_addr(const void* p) { return static_cast<unsigned>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(unsigned long long* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, unsigned bytes, unsigned long long* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_addr(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}
// Waits for phase `parity` of the barrier; gives up after a bounded number of polls (false).
__device__ __forceinline__ bool mbar_wait_bounded(unsigned long long* bar, unsigned parity) {
  const unsigned a = smem_addr(bar);
  for (int it = 0; it < (1 << 22); ++it) {
    unsigned done;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
        : "=r"(done) : "r"(a), "r"(parity) : "memory");
    if (done) return true;
  }
  return false;
}

template <typename Elem>
__global__ void __launch_bounds__(kRT * kRE * (32 / ElemTraits<Elem>::EPT))
k_router_logits(const Elem* __restrict__ x, const Elem* __restrict__ wr, const float* __restrict__ bias,
                float* logits, int T, int H, int E, int n_chunks, float* zero_buf,
                size_t zero_floats, float* zero_buf2, size_t zero_floats2, int32_t* status, float* probs, int32_t* nat_idx, uint32_t* nat_mask, int k,
                int32_t* tile_done, long long* dbg, RootArgs ro) {
  constexpr int EPT = ElemTraits<Elem>::EPT;
  constexpr int Q = 32 / EPT;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int row_bytes = H * static_cast<int>(sizeof(Elem)) + 64;   // +64 B staggers rows over the banks
  unsigned char* xs = smem_raw;
  unsigned char* ws = smem_raw + static_cast<size_t>(kRT) * row_bytes;

  const int tid = threadIdx.x;
  // The first ro.rows rows of CTAs in the grid work on one block's root each (see below); the node tiles follow.
  const bool for_root = static_cast<int>(blockIdx.y) < ro.rows;
  int root_row = 0;
#pragma unroll
  for (int b = 0; b < kMaxEarlyBlocks; ++b) root_row = static_cast<int>(blockIdx.y) == b ? ro.row[b] : root_row;
  const int e0 = blockIdx.x * kRE, t0 = for_root ? root_row : (static_cast<int>(blockIdx.y) - ro.rows) * kRT;
  griddep_launch_dependents();

  // Staging: the 4 x-rows and 8 router rows of this tile, in n_chunks pieces along h.  One thread
  // per row issues its pieces as bulk copies; piece c of all rows completes on barrier c.  The
  // router rows are requested BEFORE the dependency wait: the weights are constants of the layer
  // (nothing enqueued after they were registered may write them), so a CTA that is resident while the
  // kernel before it drains already has them on the way.  The x rows follow the wait.
  __shared__ __align__(8) unsigned long long chunk_bar[4];
  const unsigned chunk_bytes = static_cast<unsigned>(H * sizeof(Elem)) / n_chunks;
  if (tid == 0) {
    for (int c = 0; c < n_chunks; ++c) mbar_init(&chunk_bar[c], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (tid == 0)
    for (int c = 0; c < n_chunks; ++c) mbar_arrive_expect_tx(&chunk_bar[c], (kRT + kRE) * chunk_bytes);
  if (tid >= kRT && tid < kRT + kRE) {
    const int row = tid - kRT;
    const unsigned char* src = reinterpret_cast<const unsigned char*>(wr + static_cast<size_t>(min(e0 + row, E - 1)) * H);
    unsigned char* dst = ws + static_cast<size_t>(row) * row_bytes;
    for (int c = 0; c < n_chunks; ++c)
      bulk_load(dst + static_cast<size_t>(c) * chunk_bytes, src + static_cast<size_t>(c) * chunk_bytes, chunk_bytes,
                &chunk_bar[c]);
  }
  griddep_wait();
  if (dbg && tid == 0 && blockIdx.x == 0 && blockIdx.y == 0) dbg[13] = time_ns();
  if (tid < kRT) {
    const int row = tid;
    const unsigned char* src = reinterpret_cast<const unsigned char*>(x + static_cast<size_t>(min(t0 + row, T - 1)) * H);
    unsigned char* dst = xs + static_cast<size_t>(row) * row_bytes;
    for (int c = 0; c < n_chunks; ++c)
      bulk_load(dst + static_cast<size_t>(c) * chunk_bytes, src + static_cast<size_t>(c) * chunk_bytes, chunk_bytes,
                &chunk_bar[c]);
  }

  // zero the FFN output buffer (accumulated into by the FFN kernel) and the FFN kernel's routing
  // inputs (activated mask, weight table, finished-tile counters), spread over the grid
  {
    const size_t nb = static_cast<size_t>(gridDim.x) * gridDim.y;
    const size_t b = static_cast<size_t>(blockIdx.y) * gridDim.x + blockIdx.x;
    if (zero_buf) {
      float4* z4 = reinterpret_cast<float4*>(zero_buf);
      for (size_t i = b * blockDim.x + tid; i < zero_floats / 4; i += nb * blockDim.x) z4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (zero_buf2) {
      float4* z4 = reinterpret_cast<float4*>(zero_buf2);
      for (size_t i = b * blockDim.x + tid; i < zero_floats2 / 4; i += nb * blockDim.x) z4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }

  if (for_root) {
    // A root's natural top-k are anchors (Eq. 5): eligible whatever the selection decides, and what the FFN kernel
    // starts streaming on.  These CTAs come first in the grid, so they are resident (router rows on the way) before
    // everyone else, and they give the root's eight logits of their tile a whole warp each -- one lane per partial
    // sum, the same sums in the same order as below -- instead of eight threads: the root's logits are out a
    // microsecond or two before the tile's.  They go out as 64-bit words, the value under the call's 32-bit tag;
    // the first of these CTAs collects all E of them, ranks them by counting (rank = logits that are larger, or
    // equal with a lower index: the order the top-k rounds take them in) and publishes the top-k as the eight
    // tagged anchor words the FFN kernel polls.
    for (int c = 0; c < n_chunks; ++c)
      if (!mbar_wait_bounded(&chunk_bar[c], 0u)) raise_status(status, ACM_ERR_TIMEOUT);
    const int w = tid >> 5, l = tid & 31;
    const Elem* xr = reinterpret_cast<const Elem*>(xs);
    const Elem* wrow = reinterpret_cast<const Elem*>(ws + static_cast<size_t>(w) * row_bytes);
    float acc = 0.0f;
#pragma unroll 8
    for (int j = 0; j < H / 32; ++j) acc = __fmaf_rn(to_f32(xr[32 * j + l]), to_f32(wrow[32 * j + l]), acc);
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) acc = __fadd_rn(acc, __shfl_xor_sync(0xffffffffu, acc, s));
    const int e = e0 + w;
    if (l == 0 && e < E) {
      float z = acc;
      if (bias) z = __fadd_rn(z, bias[e]);
      const unsigned long long word = (static_cast<unsigned long long>(ro.tag) << 32) | __float_as_uint(z);
      asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(ro.words + static_cast<size_t>(blockIdx.y) * kMaxExperts + e), "l"(word) : "memory");
    }
    if (blockIdx.x != 0) return;
    __shared__ unsigned s_key[kMaxExperts];
    __shared__ int s_rank[kMaxExperts];
    if (tid < kMaxExperts) {
      unsigned key = 0u;
      if (tid < E) {
        unsigned long long v = 0ull;
        const long long t_start = time_ns();
        bool seen = false;
        do {
          asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(ro.words + static_cast<size_t>(blockIdx.y) * kMaxExperts + tid) : "memory");
          seen = static_cast<uint32_t>(v >> 32) == ro.tag;
        } while (!seen && time_ns() - t_start < static_cast<long long>(ro.wait_limit_ns));
        if (!seen) raise_status(status, ACM_ERR_TIMEOUT);
        key = seen ? order_key(__uint_as_float(static_cast<uint32_t>(v))) : 0u;
      }
      s_key[tid] = key;
      s_rank[tid] = 0;
    }
    __syncthreads();
    {
      const int mine_e = tid & (kMaxExperts - 1), half = tid >> 7;      // two threads per logit, 64 comparisons each
      const unsigned mine = s_key[mine_e];
      int cnt = 0;
      const uint4* keys4 = reinterpret_cast<const uint4*>(s_key + 64 * half);
#pragma unroll 4
      for (int j = 0; j < 16; ++j) {
        const uint4 kk = keys4[j];
        const int b = 64 * half + 4 * j;
        cnt += (kk.x > mine || (kk.x == mine && b + 0 < mine_e)) ? 1 : 0;
        cnt += (kk.y > mine || (kk.y == mine && b + 1 < mine_e)) ? 1 : 0;
        cnt += (kk.z > mine || (kk.z == mine && b + 2 < mine_e)) ? 1 : 0;
        cnt += (kk.w > mine || (kk.w == mine && b + 3 < mine_e)) ? 1 : 0;
      }
      if (cnt) atomicAdd(&s_rank[mine_e], cnt);
    }
    __syncthreads();
    if (tid < 32) {
      uint32_t bits[kMaskWords];
#pragma unroll
      for (int c = 0; c < kMaskWords; ++c)
        bits[c] = __ballot_sync(0xffffffffu, s_key[tid + 32 * c] != 0u && s_rank[tid + 32 * c] < k);
      if (tid < 2 * kMaskWords) {
        const uint32_t wd = (tid >> 1) == 0 ? bits[0] : (tid >> 1) == 1 ? bits[1] : (tid >> 1) == 2 ? bits[2] : bits[3];
        asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(ro.anc_words + 2 * kMaskWords * blockIdx.y + tid),
                     "r"(((wd >> (16 * (tid & 1))) & 0xffffu) | (ro.anc_tag << 16)) : "memory");
      }
    }
    return;
  }

  const int q = tid % Q;            // which EPT-wide group of the 32 partial sums
  const int mt = tid / Q;           // output of this thread group: one node x one expert
  const int el = mt % kRE, tl = mt / kRE;
  float acc[EPT];
#pragma unroll
  for (int p = 0; p < EPT; ++p) acc[p] = 0.0f;

  using Vec = typename ElemTraits<Elem>::Vec;
  const unsigned char* xr0 = xs + static_cast<size_t>(tl) * row_bytes + q * sizeof(Vec);
  const unsigned char* wrow = ws + static_cast<size_t>(el) * row_bytes + q * sizeof(Vec);
  const int steps_per_chunk = H / 32 / n_chunks;
  const int step_bytes = 32 * static_cast<int>(sizeof(Elem));
  for (int c = 0; c < n_chunks; ++c) {
    if (!mbar_wait_bounded(&chunk_bar[c], 0u)) raise_status(status, ACM_ERR_TIMEOUT);
    const int j0 = c * steps_per_chunk;
#pragma unroll 4
    for (int j = j0; j < j0 + steps_per_chunk; ++j) {
      float xa[EPT], wv[EPT];
      ElemTraits<Elem>::unpack(*reinterpret_cast<const Vec*>(xr0 + static_cast<size_t>(j) * step_bytes), xa);
      ElemTraits<Elem>::unpack(*reinterpret_cast<const Vec*>(wrow + static_cast<size_t>(j) * step_bytes), wv);
#pragma unroll
      for (int p = 0; p < EPT; ++p) acc[p] = __fmaf_rn(xa[p], wv[p], acc[p]);
    }
  }
  // halving tree over the 32 partial sums: partial l = q*EPT + p
#pragma unroll
  for (int s = 16; s >= EPT; s >>= 1) {
#pragma unroll
    for (int p = 0; p < EPT; ++p) acc[p] = __fadd_rn(acc[p], __shfl_xor_sync(0xffffffffu, acc[p], s / EPT));
  }
#pragma unroll
  for (int s = EPT / 2; s >= 1; s >>= 1) {
#pragma unroll
    for (int p = 0; p < s; ++p) acc[p] = __fadd_rn(acc[p], acc[p + s]);
  }
  if (q == 0 && e0 + el < E && t0 + tl < T) {
    const int e = e0 + el, t = t0 + tl;
    float z = acc[0];
    if (bias) z = __fadd_rn(z, bias[e]);
    logits[static_cast<size_t>(t) * E + e] = z;
    if (!isfinite(z)) raise_status(status, ACM_ERR_NONFINITE);
  }
  // The CTA that completes a tile of nodes last (all expert tiles written) finishes those nodes:
  // softmax and natural top-k, one warp per node -- spread over as many SMs as there are node tiles.
  if (tile_done) {
    __shared__ int s_last;
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      const int prev = atomicAdd(&tile_done[blockIdx.y], 1);
      s_last = prev == static_cast<int>(gridDim.x) - 1;
      if (s_last) tile_done[blockIdx.y] = 0;          // re-armed for the next call
    }
    __syncthreads();
    if (s_last) {
      __threadfence();
      const int warp = tid >> 5, lane = tid & 31, nwarps = blockDim.x >> 5;
      for (int r = warp; r < kRT; r += nwarps) {
        const int t = t0 + r;
        if (t < T)
          softmax_topk_row(logits + static_cast<size_t>(t) * E, probs ? probs + static_cast<size_t>(t) * E : nullptr,
                           nat_idx ? nat_idx + static_cast<size_t>(t) * k : nullptr,
                           nat_mask ? nat_mask + static_cast<size_t>(t) * kMaskWords : nullptr, E, k, lane);
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// Stages 2 and 3.  The selection is a decision over the whole block (the demand sums over every
// node) taken by 128 threads, one per expert slot; the routing is per node, one warp each.  The stand-alone
// entry points run them as kernels of their own; the fused calls run both behind the softmax in one CTA per
// block (k_softmax_select_route).
// ------------------------------------------------------------------------------------------
constexpr int kNodesPerCta = 4;
constexpr int kSelThreads = 128;

struct StageSmem {
  float alpha[kMaxNodes];
  uint32_t natmask[kMaxNodes][kMaskWords];
  int32_t votes[kMaxExperts];
  float u[kMaxExperts];
  float tree[2][kMaxExperts];      // two sums over the expert axis in a row use one buffer each
  int32_t rank[kMaxExperts];       // fused kernel: the experts' ranks, counted by four helper warps
  alignas(16) unsigned long long rkey[kMaxExperts];   // ranking keys of the experts (0 = not ranked)
  uint32_t A[kMaskWords], S[kMaskWords], Sp[kMaskWords], Hres[kMaskWords];
  int32_t scal[8];
};

// The selection stage runs on threads 0..127 only (one per expert slot) and synchronises them
// with a named barrier, so further warps of a larger CTA would not take part in its barriers.
__device__ __forceinline__ void sel_sync() { asm volatile("bar.sync 2, 128;" ::: "memory"); }
__device__ __forceinline__ int sel_count(bool pred) {
  int n;
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %1, 0;\n\tbar.red.popc.u32 %0, 2, 128, p;\n\t}\n"
      : "=r"(n) : "r"(static_cast<unsigned>(pred)) : "memory");
  return n;
}
// 128-slot halving tree (threads 0..127 hold one slot each): every warp forms levels 64 and 32 from shared
// memory and the remaining levels with shuffles -- the same additions in the same order as a[i] += a[i+s],
// s = 64, 32, ..., 1, so all four warps hold the same sum and nothing has to be passed back.  (`tree` must not be
// the buffer of the sum before: a slower warp may still be reading that.)
__device__ float sel_tree_sum_128(float* tree, float mine) {
  const int tid = threadIdx.x, lane = tid & 31;
  tree[tid] = mine;
  sel_sync();
  return warp_tree_sum_128(tree[lane], tree[lane + 32], tree[lane + 64], tree[lane + 96]);
}
// Barriers between the four selection warps and the four helper warps of the fused kernel (256 threads): the side that
// has produced something arrives, the side that needs it waits.
__device__ __forceinline__ void pair_arrive(int id) { asm volatile("bar.arrive %0, 256;" ::"r"(id) : "memory"); }
__device__ __forceinline__ void pair_wait(int id) { asm volatile("bar.sync %0, 256;" ::"r"(id) : "memory"); }
constexpr int kBarKeys = 3, kBarRanks = 4;
// Rank of an expert inside R by (u descending, index ascending) = the number of larger 64-bit keys.
__device__ __forceinline__ int rank_of(const unsigned long long* rkey, unsigned long long mykey) {
  int rank = 0;
  const ulonglong2* keys2 = reinterpret_cast<const ulonglong2*>(rkey);
#pragma unroll 8
  for (int j = 0; j < kMaxExperts / 2; ++j) {
    const ulonglong2 kk = keys2[j];
    rank += (kk.x > mykey ? 1 : 0) + (kk.y > mykey ? 1 : 0);
  }
  return rank;
}
// The helper warps' part (threads 128..255 of the fused kernel): the ranks, while the selection warps work out how
// many experts to keep.
__device__ void stage_select_helper(StageSmem& sm) {
  const int h = threadIdx.x - kSelThreads;
  pair_wait(kBarKeys);
  sm.rank[h] = rank_of(sm.rkey, sm.rkey[h]);
  __threadfence_block();
  pair_arrive(kBarRanks);
}

// Stage 2: demand, anchors, self-sizing, pruning.  Called by threads 0..127; thread e owns expert e.
// kStaged = false: r comes straight from global memory (every load is issued before the first wait); the natural
// top-k sets come as bit masks from `natmask_g` ([T][4], written by the router kernel) or, if that
// is null, are built here from a.nat_idx.  kStaged = true: the caller has put the probabilities in shared memory
// (`s_probs`, [T][E]) and filled sm.alpha and sm.natmask (rows >= T zero) before a CTA-wide barrier.
// Global results are written only if `write_out`.
template <bool kStaged>
__device__ void stage_select(const SelectArgs& a, StageSmem& sm, int T, int E, int k, const uint32_t* natmask_g,
                             bool write_out, uint32_t* publish_words = nullptr, uint32_t publish_tag = 0,
                             const float* s_probs = nullptr) {
  const int tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  const bool live = tid < E;
  float pr[kStaged ? 1 : kMaxNodes];
  if constexpr (!kStaged) {
    // small loads first (they gate the first barrier), then the 64 probabilities of this expert's column
    const float my_alpha = tid < kMaxNodes ? a.alpha[min(tid, T - 1)] : 0.0f;
    uint32_t my_nm[2] = {0u, 0u};
    if (natmask_g) {
#pragma unroll
      for (int i = 0; i < 2; ++i) my_nm[i] = __ldcg(natmask_g + min(tid + i * kSelThreads, T * kMaskWords - 1));
    }
    {
      const float* col = a.probs + min(tid, E - 1);
#pragma unroll
      for (int t = 0; t < kMaxNodes; ++t) pr[t] = __ldcg(col + static_cast<size_t>(min(t, T - 1)) * E);
    }
    if (tid < kMaxNodes) sm.alpha[tid] = my_alpha;
    if (natmask_g) {
#pragma unroll
      for (int i = 0; i < 2; ++i) (&sm.natmask[0][0])[tid + i * kSelThreads] = my_nm[i];
    } else {
      for (int i = tid; i < kMaxNodes * kMaskWords; i += kSelThreads) (&sm.natmask[0][0])[i] = 0u;
      sel_sync();
      for (int i = tid; i < T * k; i += kSelThreads) {
        const int e = a.nat_idx[i];
        if (e >= 0 && e < E) atomicOr(&sm.natmask[i / k][e >> 5], 1u << (e & 31));
      }
    }
  }
  if constexpr (!kStaged) {         // (the fused kernel has done this before its barrier)
    if (tid < kMaskWords) sm.Hres[tid] = (tid < (E + 31) / 32) ? (a.resident ? a.resident[tid] : 0xffffffffu) : 0u;
    if (tid < 8) sm.scal[tid] = 0;
    sel_sync();
  }
  if (tid < kMaskWords) {           // anchors (Eq. 5): union of the anchor nodes' natural sets
    uint32_t A = 0u;
    if (a.prm.use_anchors) {
      const int n_nodes = a.anchor_nodes ? a.n_anchor_nodes : 1;
      for (int i = 0; i < n_nodes; ++i) {
        const int t = a.anchor_nodes ? a.anchor_nodes[i] : 0;
        if (t >= 0 && t < T) A |= sm.natmask[t][tid];
      }
    }
    sm.A[tid] = A;
  }

  // votes v_e and demand u_e (nodes ascending, fused multiply-add)
  int votes = 0;
  float u = 0.0f;
  const int demand_mode = a.prm.demand;
  if constexpr (kStaged) {
    // (a rolled loop of sixteen nodes a turn: in the fused kernel the code is fetched while the FFN kernel streams
    // weights, and every further line of straight-line code is one more slow instruction fetch)
    const float* pcol = s_probs + min(tid, E - 1);
#pragma unroll 1
    for (int t0 = 0; t0 < T; t0 += 16) {
      float al[16], pj[16];
      unsigned in_mask = 0;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const int t = min(t0 + j, T - 1);
        al[j] = sm.alpha[t];
        pj[j] = pcol[t * E];
        in_mask |= ((sm.natmask[t][warp] >> lane) & 1u) << j;
      }
      const unsigned valid = t0 + 16 > T ? (1u << (T - t0)) - 1u : 0xffffu;
      in_mask &= valid;
      votes += __popc(in_mask);
      const unsigned take = demand_mode == ACM_DEMAND_FULL_MASS ? valid
                          : demand_mode == ACM_DEMAND_TOPK_MASS ? in_mask : 0u;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const float nu = __fmaf_rn(al[j], pj[j], u);
        u = ((take >> j) & 1u) ? nu : u;
      }
    }
  } else {
#pragma unroll
  for (int t0 = 0; t0 < kMaxNodes; t0 += 16) {
    if (t0 < T) {
      float al[16];
      unsigned in_mask = 0;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const int t = min(t0 + j, T - 1);
        al[j] = sm.alpha[t];
        in_mask |= ((sm.natmask[t][warp] >> lane) & 1u) << j;
      }
      const unsigned valid = t0 + 16 > T ? (1u << (T - t0)) - 1u : 0xffffu;
      in_mask &= valid;
      votes += __popc(in_mask);
      // which nodes enter the chain; the chain itself is branch-free (multiply-add, then select)
      const unsigned take = demand_mode == ACM_DEMAND_FULL_MASS ? valid
                          : demand_mode == ACM_DEMAND_TOPK_MASS ? in_mask : 0u;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const float nu = __fmaf_rn(al[j], pr[t0 + j], u);
        u = ((take >> j) & 1u) ? nu : u;
      }
    }
  }
  }
  if (!live) { votes = 0; u = 0.0f; }
  if (a.prm.demand == ACM_DEMAND_VOTES) u = static_cast<float>(votes);
  sm.votes[tid] = votes;
  sm.u[tid] = u;
  sel_sync();                       // sm.A
  const bool in_A = live && ((sm.A[warp] >> lane) & 1u);
  const bool in_R = live && !in_A;
  const int nA = sel_count(in_A);
  const int nR = E - nA;
  const int n_positive = sel_count(in_R && u > 0.0f);
  const float upos = in_R ? fmaxf(u, 0.0f) : 0.0f;
  // rank inside R by (u descending, index ascending): one 64-bit key per expert
  const unsigned long long mykey =
      in_R ? ((static_cast<unsigned long long>(order_key(u)) << 32) | (0xffffffffu - tid)) : 0ull;
  sm.rkey[tid] = mykey;
  if constexpr (kStaged) {
    __threadfence_block();
    pair_arrive(kBarKeys);          // the helper warps count the ranks meanwhile
  }
  const float Z = sel_tree_sum_128(sm.tree[0], upos);

  const int floor_keep = max(0, k - nA);
  int n_er = 0, n_keep;
  if (a.prm.fixed_budget > 0) {
    n_keep = max(max(0, a.prm.fixed_budget - nA), floor_keep);
  } else if (Z > 0.0f) {
    const float qv = __fdiv_rn(upos, Z);
    const float h = (qv >= 1.17549435e-38f) ? __fmul_rn(qv, log_fixed(qv)) : 0.0f;
    const float entropy = -sel_tree_sum_128(sm.tree[1], h);
    const float perp = exp_fixed(entropy);
    n_er = static_cast<int>(ceilf(__fsub_rn(perp, a.prm.ceil_guard)));
    n_er = min(max(n_er, 1), n_positive);
    n_keep = max(n_er, floor_keep);
  } else {
    n_keep = floor_keep;
  }
  n_keep = min(n_keep, nR);

  bool in_S = in_A;
  if constexpr (kStaged) {
    pair_wait(kBarRanks);
    if (in_R) in_S = sm.rank[tid] < n_keep;
  } else {
    sel_sync();
    if (in_R) in_S = rank_of(sm.rkey, mykey) < n_keep;
  }
  const unsigned s_word = __ballot_sync(0xffffffffu, in_S);
  if (lane == 0) sm.S[warp] = s_word;
  const int nS = sel_count(in_S);
  const int n_union = sel_count(live && votes > 0);
  if (live && votes > 0 && !in_S) atomicAdd(&sm.scal[0], votes);   // a(S)
  sel_sync();
  const int aS = sm.scal[0];

  bool in_Sp = in_S;
  int m_star = 0;
  const bool resident = live && ((sm.Hres[warp] >> lane) & 1u);
  if (a.prm.residency == 1 && a.resident) {
    const bool in_C = in_S && !resident;
    bool removed = false;
    if (in_C) {
      int pos = 1, cum = votes;     // position in pi (1-based) and votes of the prefix ending here
      for (int j = 0; j < E; ++j) {
        if (j == tid) continue;
        const bool j_in_C = ((sm.S[j >> 5] >> (j & 31)) & 1u) && !((sm.Hres[j >> 5] >> (j & 31)) & 1u);
        const float uj = sm.u[j];
        if (j_in_C && (uj < u || (uj == u && j < tid))) {
          pos += 1;
          cum += sm.votes[j];
        }
      }
      removed = cum <= aS && nS - pos >= k && pos <= a.prm.max_remove;
    }
    in_Sp = in_S && !removed;
    m_star = sel_count(removed);
  } else if (a.prm.residency == 2 && a.resident) {
    in_Sp = (in_S && resident) || in_A;
  }
  const unsigned sp_word = __ballot_sync(0xffffffffu, in_Sp);
  if (lane == 0) sm.Sp[warp] = sp_word;
  const int nSp = sel_count(in_Sp);          // (a barrier: sm.Sp is complete)
  if (publish_words && tid < 2 * kMaskWords) {
    // The FFN kernel may start on the eligible set now, before the outputs below are written and while the
    // routes are made: eight self-validating words, 16 mask bits under a 16-bit tag of this call each.
    const uint32_t bits = (sm.Sp[tid >> 1] >> (16 * (tid & 1))) & 0xffffu;
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(publish_words + tid), "r"(bits | (publish_tag << 16)) : "memory");
  }
  if (a.prm.residency == 2 && a.resident) m_star = nS - nSp;

  if (write_out) {
    const int words = (E + 31) / 32;
    if (tid < words) {
      a.mask_out[tid] = sm.Sp[tid];
      if (a.unpruned_out) a.unpruned_out[tid] = sm.S[tid];
    }
    if (live && a.demand_out) a.demand_out[tid] = u;
    if (tid == 0) {
      *a.count_out = nSp;
      if (a.stats_out) {
        acm_block_stats st;
        st.n_anchor = nA; st.n_er = n_er; st.n_eligible = nS; st.n_eligible_pruned = nSp;
        st.n_activated = 0; st.n_natural_union = n_union; st.displaced_aS = aS; st.pruned_m = m_star;
        st.n_staged = 0; st.n_streamed = 0; st.reserved[0] = st.reserved[1] = 0;
        *a.stats_out = st;
      }
    }
  }
  sel_sync();
}

// Stage 3 for ONE node, by one warp: restricted top-k (Eq. 2) ranked on the logits, and the
// combine weights.  Lane j < k returns the j-th choice (expert id or -1) and its weight.
__device__ __forceinline__ void route_node(const float (&z)[4], const uint32_t (&mask_w)[4], int E, int k, int lane,
                                           int weighting, float routed_scale, int& e_out, float& w_out) {
  float y[4];
  unsigned key[4];
  float zmax = fmaxf(fmaxf(z[0], z[1]), fmaxf(z[2], z[3]));
#pragma unroll
  for (int s = 16; s >= 1; s >>= 1) zmax = fmaxf(zmax, __shfl_xor_sync(0xffffffffu, zmax, s));
  float s_all = 0.f, s_elig = 0.f, s_sel = 0.f, my_y = 0.f;
  int my_e = -1;
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const bool in_e = lane + 32 * c < E;
    const bool elig = in_e && ((mask_w[c] >> lane) & 1u);
    y[c] = in_e ? __expf(z[c] - zmax) : 0.0f;
    s_all += y[c];
    s_elig += elig ? y[c] : 0.0f;
    key[c] = elig ? order_key(z[c]) : 0u;
  }
  if (weighting != ACM_W_RENORM_TOPK) {      // warp-uniform: only the denominator that is used
    float other = weighting == ACM_W_SOFTMAX_RAW ? s_all : s_elig;
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) other += __shfl_xor_sync(0xffffffffu, other, s);
    s_all = s_elig = other;
  }
  for (int j = 0; j < k; ++j) {
    const int e = warp_take_best(key, lane);
    const int c = (e >= 0 ? e : 0) >> 5;
    const float cand = c == 0 ? y[0] : c == 1 ? y[1] : c == 2 ? y[2] : y[3];
    const float got = __shfl_sync(0xffffffffu, cand, (e >= 0 ? e : 0) & 31);
    const float ye = e >= 0 ? got : 0.f;
    s_sel += ye;
    if (lane == j) { my_e = e; my_y = ye; }
  }
  const float den = weighting == ACM_W_RENORM_TOPK ? s_sel : weighting == ACM_W_SOFTMAX_RAW ? s_all : s_elig;
  e_out = my_e;
  w_out = my_e >= 0 ? routed_scale * my_y / den : 0.0f;
}

__device__ __forceinline__ void load_logit_row(const float* logits, int t, int E, int lane, float (&z)[4]) {
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const int e = lane + 32 * c;
    const float v = __ldcg(logits + static_cast<size_t>(t) * E + min(e, E - 1));
    z[c] = e < E ? v : -INFINITY;
  }
}

// One node's routes (lane j < k holds choice j) OR-ed into a mask in shared memory (what one block activates)
__device__ __forceinline__ void publish_routes_local(uint32_t* s_act, int k, int lane, int e) {
  const bool has = lane < k && e >= 0;
#pragma unroll
  for (int wd = 0; wd < kMaskWords; ++wd) {
    const unsigned bits = __reduce_or_sync(0xffffffffu, (has && (e >> 5) == wd) ? 1u << (e & 31) : 0u);
    if (lane == wd && bits) atomicOr(s_act + wd, bits);
  }
}

__global__ void __launch_bounds__(kSelThreads) k_select(SelectArgs a, int T, int E, int k) {
  __shared__ StageSmem sm;
  stage_select<false>(a, sm, T, E, k, nullptr, true);
}

// grid = ceil(T / 4) CTAs of four warps, one node per warp
__global__ void __launch_bounds__(kSelThreads) k_route(RouteArgs a, int T, int E, int k) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int t = blockIdx.x * kNodesPerCta + warp;
  if (t >= T) return;
  float z[4];
  uint32_t mask_w[4];
  load_logit_row(a.logits, t, E, lane, z);
#pragma unroll
  for (int c = 0; c < 4; ++c) mask_w[c] = a.mask[min(c, (E + 31) / 32 - 1)];
  int e;
  float w;
  route_node(z, mask_w, E, k, lane, a.weighting, a.routed_scale, e, w);
  if (lane < k) {
    a.idx_out[static_cast<size_t>(t) * k + lane] = e;
    a.w_out[static_cast<size_t>(t) * k + lane] = w;
  }
}

// The FFN kernel may start on the eligible set while the routes are made.  The set is published as
// eight self-validating words, 16 mask bits under a 16-bit tag of this call each: a reader needs no
// second load to know that what it read is current.  (Relaxed stores: everything else the reader
// depends on was complete before this kernel passed its dependency wait.)
__device__ __forceinline__ void publish_eligible(const RouteArgs& ra, const StageSmem& sm, int i) {
  const uint32_t bits = (sm.Sp[i >> 1] >> (16 * (i & 1))) & 0xffffu;
  const uint32_t word = bits | (static_cast<uint32_t>(ra.sel_epoch) << 16);
  asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(ra.sel_flag + i), "r"(word) : "memory");
}

#define ACM_RT(slot) do { if (ra.dbg && blockIdx.x == 0 && threadIdx.x == 0) ra.dbg[slot] = time_ns(); } while (0)
// Stages 1b-3 of the fused calls and the FFN kernel's routing inputs in ONE launch: a cluster of up to four CTAs
// per verification block (block b = the rows bd.off[b] .. bd.off[b+1]-1 of every per-node array; a single block is a
// batch of one), sixteen warps each, ONE ROW PER WARP -- softmax + top-k of a row is a chain of a few hundred
// dependent instructions, so the rows are spread over as many warps and SMs as it takes to give each its own.  The
// router kernel before it has written the logits only.  Every warp loads its row (the one trip through L2 of the
// whole chain: with the FFN kernel already streaming weights, each further one would cost well over a microsecond),
// then
//   1b  softmax and natural top-k of the row (Eq. 1); the probabilities and the top-k mask go into the shared memory
//       of EVERY CTA of the cluster (distributed shared memory), the logits stay in registers;
//   --  cluster barrier: every CTA now holds the whole block's probabilities and natural sets
//   2   the selection (Eq. 3-7; it sees nothing of the other blocks), repeated by warps 0-3 of every CTA -- it is
//       deterministic, so all hold the same S' and no second exchange is needed; the cluster's first CTA writes the
//       outputs and publishes the eligible set as eight tagged words, ra.sel_flag + 8 b;
//   3   the row's routes inside that set (Eq. 2).
// The FFN kernel's inputs are shared by all blocks: the activated mask is OR-ed into by every CTA, the weight table
// is indexed by the row in the stacked batch.  The CTAs ask for more shared memory than they use so that no CTA of
// the FFN kernel (launched as a dependent while this one runs) fits beside them: its polling and streaming would
// slow the selection by half.
namespace cg = cooperative_groups;
constexpr int kFusedWarps = 16;
constexpr int kFusedMaxCtas = 4;
constexpr size_t kFusedSmemRequest = 100u << 10;
struct FusedSmem {
  StageSmem st;
  alignas(16) float probs[kMaxNodes * kMaxExperts];   // [T][E], every row written by the warp (of some CTA) that owns it
  uint32_t act[kMaskWords];                             // experts this CTA's rows activate (first CTA: the block's)
};
static_assert(sizeof(FusedSmem) <= kFusedSmemRequest, "shared memory of the selection kernel");
__global__ void __launch_bounds__(32 * kFusedWarps)
k_softmax_select_route(SelectArgs sa, RouteArgs ra, BatchDesc bd, const uint32_t* mask_override, int E, int k) {
  extern __shared__ __align__(16) unsigned char fused_raw[];
  FusedSmem& fs = *reinterpret_cast<FusedSmem*>(fused_raw);
  StageSmem& sm = fs.st;
  cg::cluster_group cluster = cg::this_cluster();
  const int C = static_cast<int>(cluster.num_blocks()), q = static_cast<int>(cluster.block_rank());
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.x / C, t_lo = bd.off[b], T = bd.off[b + 1] - t_lo;
  const int r = q * kFusedWarps + warp;                 // this warp's row of the block
  const bool first = q == 0;
  const bool report = sa.stats_out != nullptr || ra.host_stage_list != nullptr;
  const uint32_t tag = static_cast<uint32_t>(ra.sel_epoch) & 0xffffu;
  griddep_launch_dependents();
  if (tid < kMaskWords) fs.act[tid] = 0u;
  for (int i = tid; i < kMaxNodes * kMaskWords; i += blockDim.x) (&sm.natmask[0][0])[i] = 0u;
  cluster.sync();                 // every CTA of the cluster is running and has cleared what the others write into
  griddep_wait();
  ACM_RT(0);
  float z[4];
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const int e = lane + 32 * c;
    const float v = __ldcg(ra.logits + static_cast<size_t>(t_lo + min(r, T - 1)) * E + min(e, E - 1));
    z[c] = (r < T && e < E) ? v : -INFINITY;
  }
  if (!mask_override && tid < kMaxNodes) sm.alpha[tid] = sa.alpha[t_lo + min(tid, T - 1)];
  if (tid < kMaskWords) sm.Hres[tid] = (tid < (E + 31) / 32) ? (sa.resident ? sa.resident[tid] : 0xffffffffu) : 0u;
  if (tid < 8) sm.scal[tid] = 0;
  if (r < T && !mask_override) {
    float prob[4];
    uint32_t bits[kMaskWords];
    softmax_topk_regs(z, E, k, lane, prob, bits, nullptr, true);
    const uint32_t my_bits = lane == 0 ? bits[0] : lane == 1 ? bits[1] : lane == 2 ? bits[2] : bits[3];
    for (int p = 0; p < C; ++p) {
      float* probs_p = cluster.map_shared_rank(fs.probs, p);
      uint32_t* nat_p = cluster.map_shared_rank(&sm.natmask[0][0], p);
#pragma unroll
      for (int c = 0; c < 4; ++c)
        if (lane + 32 * c < E) probs_p[r * E + lane + 32 * c] = prob[c];
      if (lane < kMaskWords) nat_p[r * kMaskWords + lane] = my_bits;
    }
  }
  cluster.sync();                 // the whole block's probabilities and natural sets are in every CTA

  // 2
  SelectArgs mine = sa;
  mine.anchor_nodes = nullptr;
  mine.n_anchor_nodes = 0;
  mine.mask_out += b * kMaskWords;
  if (mine.unpruned_out) mine.unpruned_out += b * kMaskWords;
  mine.count_out += b;
  if (mine.demand_out) mine.demand_out += static_cast<size_t>(b) * kMaxExperts;
  if (mine.stats_out) mine.stats_out += b;
  if (mask_override) {            // (single block) the caller's set instead of a selection
    if (tid < kMaskWords) {
      const uint32_t m = tid < (E + 31) / 32 ? mask_override[tid] : 0u;
      sm.Sp[tid] = m;
      if (first && tid < (E + 31) / 32) mine.mask_out[tid] = m;
    }
    if (first && tid == 0 && mine.stats_out) {
      acm_block_stats st = {};
      *mine.stats_out = st;
    }
    __syncthreads();
    if (first && ra.sel_flag && tid < 2 * kMaskWords) publish_eligible(ra, sm, tid);
  } else {
    if (tid < kSelThreads)
      stage_select<true>(mine, sm, T, E, k, nullptr, first,
                         (first && ra.sel_flag) ? ra.sel_flag + 2 * kMaskWords * b : nullptr, tag, fs.probs);
    else if (tid < 2 * kSelThreads)
      stage_select_helper(sm);
    __syncthreads();
  }
  ACM_RT(2);

  // 3
  if (r < T) {
    uint32_t mask_w[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) mask_w[c] = sm.Sp[c];
    const int t = t_lo + r;
    int e;
    float w;
    route_node(z, mask_w, E, k, lane, ra.weighting, ra.routed_scale, e, w);
    if (lane < k) {
      ra.idx_out[static_cast<size_t>(t) * k + lane] = e;
      ra.w_out[static_cast<size_t>(t) * k + lane] = w;
      if (e >= 0 && ra.wtab) ra.wtab[static_cast<size_t>(e) * kWtabStride + t] = w;
    }
    publish_routes_local(fs.act, k, lane, e);
  }
  ACM_RT(3);
  __syncthreads();
  if (tid < kMaskWords && fs.act[tid]) {
    if (ra.act_mask) atomicOr(ra.act_mask + tid, fs.act[tid]);
    if (report && !first) atomicOr(cluster.map_shared_rank(fs.act, 0) + tid, fs.act[tid]);
  }
  if (!report) return;
  // the block's own report, by the cluster's first CTA: its activated experts and (single block, offloaded layer)
  // which of them have to be copied in, in ascending id order = their staging slots
  cluster.sync();
  if (first && warp == 0) {
    const int words = (E + 31) / 32;
    const uint32_t act = lane < words ? fs.act[lane] : 0u;
    const uint32_t res = lane < words ? (ra.resident ? ra.resident[lane] : 0xffffffffu) : 0u;
    const uint32_t stg = act & ~res;
    int n_act = __popc(act), n_stg = __popc(stg), before = 0;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
      const int up = __shfl_up_sync(0xffffffffu, n_stg, s);      // inclusive scan of the staged counts
      n_stg += lane >= s ? up : 0;
    }
    before = n_stg - __popc(stg);
    const int tot_stg = __shfl_sync(0xffffffffu, n_stg, 31);
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) n_act += __shfl_xor_sync(0xffffffffu, n_act, s);
    if (ra.host_stage_list) {
      uint32_t m = stg;
      int pos = before;
      while (m) {
        const int bit = __ffs(m) - 1;
        m &= m - 1;
        ra.host_stage_list[1 + pos++] = lane * 32 + bit;
      }
      if (lane == 0) ra.host_stage_list[0] = tot_stg;
      if (lane < kMaskWords) ra.host_stage_list[1 + kMaxExperts + lane] = static_cast<int32_t>(act);   // the activated set
    }
    if (lane == 0 && mine.stats_out) {
      mine.stats_out->n_activated = n_act;
      mine.stats_out->n_staged = tot_stg;
    }
  }
}

// Routes given by the caller (acm_expert_ffn) -> the FFN kernel's inputs.  One CTA.
__global__ void __launch_bounds__(512) k_routes_to_table(const int32_t* idx, const float* w, uint32_t* act_mask,
                                                         float* wtab, int32_t* ready, int T, int E, int k) {
  for (int i = threadIdx.x; i < kMaxExperts * kWtabStride; i += blockDim.x) wtab[i] = 0.0f;
  for (int i = threadIdx.x; i < 2 * kMaxSlots; i += blockDim.x) ready[i] = 0;
  if (threadIdx.x < kMaskWords) act_mask[threadIdx.x] = 0u;
  __syncthreads();
  for (int i = threadIdx.x; i < T * k; i += blockDim.x) {
    const int e = idx[i];
    if (e >= 0 && e < E) {
      atomicOr(act_mask + (e >> 5), 1u << (e & 31));
      wtab[static_cast<size_t>(e) * kWtabStride + i / k] = w[i];
    }
  }
}

}  // namespace

cudaError_t launch_router_logits(int dtype, const void* x, const void* w_router, const float* bias,
                                 float* logits, int T, int H, int E, float* zero_buf,
                                 size_t zero_floats, float* zero_buf2, size_t zero_floats2, int32_t* status,
                                 float* probs, int32_t* nat_idx, uint32_t* nat_mask, int k, int32_t* tile_done,
                                 bool pdl, cudaStream_t s, long long* dbg, const RootArgs* root) {
  if (!probs && !nat_idx) tile_done = nullptr;
  RootArgs ro = {};
  if (root) ro = *root;
  if (ro.rows != 0 && (!ro.words || !ro.anc_words || ro.rows < 0 || ro.rows > kMaxEarlyBlocks)) return cudaErrorInvalidValue;
  cudaLaunchAttribute attr[1];
  set_pdl_attr(attr);
  cudaLaunchConfig_t cfg = {};
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  const dim3 grid((E + kRE - 1) / kRE, (T + kRT - 1) / kRT + ro.rows);
  const int elt = dtype == ACM_F32 ? 4 : 2;
  size_t smem = static_cast<size_t>(kRT + kRE) * (static_cast<size_t>(H) * elt + 64);
  // At most two CTAs per SM (by asking for more shared memory than the tile needs): the grid then
  // spreads over the whole GPU instead of piling four deep onto the SMs that happen to be free first.
  if (smem < (104u << 10)) smem = 104u << 10;
  // pieces of at least 4 KB per row: every bulk copy has a fixed cost, and few large ones land sooner
  const size_t row = static_cast<size_t>(H) * elt;
  const int n_chunks = (row >= 16384 && H % 128 == 0) ? 4 : (row >= 8192 && H % 64 == 0) ? 2 : 1;
  if ((static_cast<size_t>(H) * elt) % 16 != 0) return cudaErrorInvalidValue;   // rows are copied in 16-byte units
  if (dtype == ACM_F32) {
    auto kern = k_router_logits<float>;
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (err != cudaSuccess) return err;
    cfg.gridDim = grid; cfg.blockDim = dim3(kRT * kRE * 8); cfg.dynamicSmemBytes = smem;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<const float*>(x), static_cast<const float*>(w_router), bias,
                              logits, T, H, E, n_chunks, zero_buf, zero_floats, zero_buf2, zero_floats2, status, probs, nat_idx, nat_mask, k,
                              tile_done, dbg, ro);
  } else {
    auto kern = k_router_logits<__nv_bfloat16>;
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (err != cudaSuccess) return err;
    cfg.gridDim = grid; cfg.blockDim = dim3(kRT * kRE * (32 / ElemTraits<__nv_bfloat16>::EPT)); cfg.dynamicSmemBytes = smem;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<const __nv_bfloat16*>(x),
                              static_cast<const __nv_bfloat16*>(w_router), bias, logits, T, H, E, n_chunks, zero_buf,
                              zero_floats, zero_buf2, zero_floats2, status, probs, nat_idx, nat_mask, k, tile_done, dbg, ro);
  }
}

cudaError_t launch_select(const SelectArgs& a, int T, int E, int k, cudaStream_t s) {
  k_select<<<1, kSelThreads, 0, s>>>(a, T, E, k);
  return cudaGetLastError();
}

cudaError_t launch_route(const RouteArgs& a, int T, int E, int k, cudaStream_t s) {
  k_route<<<(T + kNodesPerCta - 1) / kNodesPerCta, kSelThreads, 0, s>>>(a, T, E, k);
  return cudaGetLastError();
}

cudaError_t select_configure() {
  return cudaFuncSetAttribute(k_softmax_select_route, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              static_cast<int>(kFusedSmemRequest));
}

int select_ctas_per_block(int widest) {
  const int c = (widest + kFusedWarps - 1) / kFusedWarps;
  return c <= 1 ? 1 : c == 2 ? 2 : kFusedMaxCtas;
}

cudaError_t launch_softmax_select_route(const SelectArgs& sa, const RouteArgs& ra, const BatchDesc& bd,
                                        const uint32_t* mask_override, int E, int k, bool pdl, cudaStream_t s) {
  int widest = 1;
  for (int b = 0; b < bd.n_blocks; ++b) widest = bd.off[b + 1] - bd.off[b] > widest ? bd.off[b + 1] - bd.off[b] : widest;
  if (widest > kFusedMaxCtas * kFusedWarps) return cudaErrorInvalidValue;      // a warp per row
  const int C = select_ctas_per_block(widest);
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  set_pdl_attr(attr + 1);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(bd.n_blocks * C);
  cfg.blockDim = dim3(32 * kFusedWarps);
  cfg.dynamicSmemBytes = kFusedSmemRequest;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, k_softmax_select_route, sa, ra, bd, mask_override, E, k);
}

cudaError_t launch_routes_to_table(const int32_t* idx, const float* w, uint32_t* act_mask, float* wtab,
                                   int32_t* ready, int T, int E, int k, cudaStream_t s) {
  k_routes_to_table<<<1, 512, 0, s>>>(idx, w, act_mask, wtab, ready, T, E, k);
  return cudaGetLastError();
}

}  // namespace acm
