// Internal declarations shared by the translation units of libacm (not part of the C ABI).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/acm.h"

namespace acm {

constexpr int kMaxExperts = 128;   // E limit; also the padded length of expert-axis tree sums
constexpr int kMaxTopK = 8;
constexpr int kMaxNodes = 64;      // T limit of one verification block; the FFN kernel handles node columns 64 at a time
constexpr int kWideNodes = 128;    // T limit of a batch of blocks = node columns of one wide FFN accumulator tile
constexpr int kWtabStride = kWideNodes;   // row length of the combine-weight table [expert][node]
constexpr int kMaxShared = 4;
constexpr int kMaxSlots = kMaxExperts + kMaxShared;   // activated-expert slots of one work list
constexpr int kMaskWords = 4;

// Work-list entry: which weight tensor an activated expert streams from, and its index there.
constexpr int kSrcRouted = 0;   // the layer's device tensors, index = expert id
constexpr int kSrcShared = 1;   // the layer's shared-expert tensors, index = shared id
constexpr int kSrcStaged = 2;   // the context's staging slots (experts copied from the host)
__host__ __device__ inline int32_t make_entry(int src, int idx) { return (src << 28) | idx; }
__host__ __device__ inline int entry_src(int32_t e) { return (e >> 28) & 3; }
__host__ __device__ inline int entry_idx(int32_t e) { return e & 0x0fffffff; }

// The FFN kernel takes its activated experts from a bit mask over the routed experts (slot a = the
// a-th set bit, i.e. ascending expert id; shared experts are appended) and the combine weights from a
// dense table indexed [expert][node] (0 where the node is not routed there).  Both are filled
// straight by the routing warps, so nothing has to gather the routes into lists first.
// Device workspace of one context (one allocation, carved on the host).
struct Workspace {
  float* logits;        // [T,E]
  int32_t* idx;         // [T,k]
  float* w;             // [T,k]
  // per block of a batch (a single block uses entry 0)
  uint32_t* mask;       // [64][4] eligible set S'
  uint32_t* unpruned;   // [64][4] S
  int32_t* count;       // [64]
  float* demand;        // [64][kMaxExperts]
  acm_block_stats* stats;   // [64]
  uint32_t* act_mask;   // [4] activated routed experts of the current block
  float* wtab;          // [kMaxExperts][kWtabStride] combine weight of (expert, node)
  void* hbuf;           // [2][kMaxSlots][kWideNodes][I] bf16 (f32 path: [T][k+ns][I] float)
  float* frag;          // [2][grid][2 column halves][128*64] split-K partial sums, accumulated into the finishing CTA's buffer; zero between launches
  int32_t* frag_flag;   // [2][grid][2] how many CTAs have added to that buffer; zero between launches
  int32_t* ready;       // [2][kMaxSlots] finished gate/up tiles per activated slot
  int32_t* status;      // [1] sticky device-side status
  int32_t* tile_done;   // [64] router kernel: expert tiles finished per node tile (self-resetting)
  int32_t* ticket;      // [4] spare words (the MXFP4 scale check keeps its maximum in one)
  uint32_t* sel_words;  // [kMaxEarlyBlocks][8] the eligible masks as tagged 16-bit pieces (early start of the FFN kernel)
  unsigned long long* root_words;   // [kMaxEarlyBlocks][kMaxExperts] the roots' logits under the call's 32-bit tag (router kernel, see RootArgs)
  uint32_t* anc_words;  // [kMaxEarlyBlocks][8] the anchor experts (each root's natural top-k) as tagged 16-bit pieces, published by the router kernel's root CTAs
};

struct SelectArgs {
  const float* probs;
  const int32_t* nat_idx;
  const float* alpha;
  const int32_t* anchor_nodes;
  int n_anchor_nodes;
  const uint32_t* resident;      // may be null
  acm_select_params prm;
  uint32_t* mask_out;
  uint32_t* unpruned_out;        // may be null
  int32_t* count_out;
  float* demand_out;             // may be null
  acm_block_stats* stats_out;    // may be null
};

// A batch of verification blocks stacked along the node axis: block b owns rows off[b] .. off[b+1]-1.
struct BatchDesc {
  int n_blocks;
  int off[kMaxNodes + 1];    // (at most 64 blocks, at most kWideNodes rows in all, at most kMaxNodes rows a block)
};
constexpr int kMaxEarlyBlocks = 8;   // blocks whose eligible sets the FFN kernel can poll for (8 tagged words each)

// Fused calls with an early start of the FFN kernel: the router kernel puts `rows` rows of CTAs (one per block, at most
// kMaxEarlyBlocks) in front of its grid; row b works out the logits of block b's root, the node row[b], ahead of
// everyone (published as 64-bit words, the value under `tag`, in words[b][kMaxExperts]) and from them the block's
// anchors (Eq. 5), published as the eight tagged words anc_words[b][8].
struct RootArgs {
  int rows;
  int row[kMaxEarlyBlocks];
  unsigned long long* words;
  uint32_t tag;
  uint32_t* anc_words;
  uint32_t anc_tag;
  unsigned long long wait_limit_ns;
};

struct RouteArgs {
  const float* logits;
  const uint32_t* mask;
  int32_t* idx_out;
  float* w_out;
  int weighting;
  float routed_scale;
  // inputs of the FFN kernel (all null when only the routes are wanted); zero on entry
  uint32_t* act_mask;            // [4] activated experts, OR-ed into
  float* wtab;                   // [kMaxExperts][kWtabStride] combine weights by (expert, node)
  // the block's own report (single block):
  const uint32_t* resident;      // non-null: activated experts outside it are "staged"
  int32_t* host_stage_list;      // mapped pinned memory (may be null): [0] = n_stage, [1..] = staged expert ids,
                                 // [1 + kMaxExperts ..] = the activated mask (4 words)
  uint32_t* sel_flag;            // non-null: [8] words, the eligible mask in 16-bit pieces tagged with sel_epoch
  int32_t sel_epoch;
  long long* dbg;                // optional time stamps in ns (acm_stage_timing): [0] start, [2] selection done, [3] routes done
};

// Programmatic dependent launch: a kernel launched with `pdl` may start while the kernel before it
// in the stream is still running; it runs its set-up, then waits (griddepcontrol.wait) for that
// kernel to complete before it touches global memory.  Every kernel of the hot path signals its
// dependents at once and waits before its first global access, so completion stays transitive.
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
inline void set_pdl_attr(cudaLaunchAttribute* attr) {
  attr->id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr->val.programmaticStreamSerializationAllowed = 1;
}

// ---- launchers (routing.cu) -------------------------------------------------------------
cudaError_t launch_router_logits(int dtype, const void* x, const void* w_router, const float* bias,
                                 float* logits, int T, int H, int E, float* zero_buf,
                                 size_t zero_floats, float* zero_buf2, size_t zero_floats2, int32_t* status,
                                 float* probs, int32_t* nat_idx, uint32_t* nat_mask, int k, int32_t* tile_done,
                                 bool pdl, cudaStream_t s, long long* dbg = nullptr, const RootArgs* root = nullptr);
cudaError_t launch_select(const SelectArgs& a, int T, int E, int k, cudaStream_t s);
cudaError_t launch_route(const RouteArgs& a, int T, int E, int k, cudaStream_t s);
// The fused calls' stages 1b-3 in ONE launch, a cluster of select_ctas_per_block(widest block) CTAs per block of `bd`
// (a single block: n_blocks = 1, off = {0, T}): softmax and natural top-k of the logits in ra.logits, selection
// (unless mask_override, single block only), routes, the FFN kernel's routing inputs.  The per-block outputs of `sa`
// (mask, unpruned, count, demand [kMaxExperts each], stats) are arrays over the blocks; ra.sel_flag (may be
// null) holds 8 tagged words per block for the eligible set.
int select_ctas_per_block(int widest);
cudaError_t select_configure();   // the kernel's function attributes, once per device (when a context is created)
cudaError_t launch_softmax_select_route(const SelectArgs& sa, const RouteArgs& ra, const BatchDesc& bd,
                                        const uint32_t* mask_override, int E, int k, bool pdl, cudaStream_t s);
// routes given by the caller -> activated mask, weight table (both cleared first) and cleared `ready`
cudaError_t launch_routes_to_table(const int32_t* idx, const float* w, uint32_t* act_mask, float* wtab,
                                   int32_t* ready, int T, int E, int k, cudaStream_t s);

// ---- launchers (ffn.cu) -----------------------------------------------------------------
struct FfnMaps {               // TMA descriptors of one layer (bf16 path)
  CUtensorMap gate_up, down;               // routed experts  [E,2I,H] / [E,H,I]
  CUtensorMap shared_gate_up, shared_down; // shared experts (copies of the above if none)
  CUtensorMap staged_gate_up, staged_down; // staging slots   (copies of the above if none)
};
struct FfnLaunch {
  int T, H, I, n_pad;
  const uint32_t* act_mask;  // [4] activated routed experts
  const uint32_t* resident;  // [4] or null (all resident)
  int li;                    // 0: resident activated experts + shared experts; 1: the staged (non-resident) ones
  uint32_t only[4];          // further restriction of this launch's experts (all ones: none); one wave of list 1
  int n_shared;
  const int32_t* slot_of;    // non-null: expert id -> slot of the layer's expert pool (the `staged` tensor maps)
  const float* wtab;         // [kMaxExperts][kWtabStride] combine weights by (expert, node)
  acm_block_stats* stats;    // list 0 fills n_activated / n_staged (may be null)
  void* hbuf;                // [kMaxSlots][kWideNodes][I] bf16 of this list
  int32_t* ready;            // [kMaxSlots] of this list (zero on entry)
  float* frag;
  int32_t* frag_flag;
  // Early start: if sel_flag is given the kernel does not wait for the routing kernel to complete.  It
  // polls the eight tagged words at sel_flag (16 bits of the ELIGIBLE mask under the low 16 bits of
  // sel_epoch each) and takes the eligible set as its work list -- an eligible expert no node chose
  // has zero combine weights and contributes nothing.  The combine weights are read only when the
  // first tile is finalised, after a full dependency wait.
  const uint32_t* sel_flag;
  int32_t sel_epoch;
  int sel_blocks;            // blocks of a batch (1..kMaxEarlyBlocks): eight words each, the work list is their union
  const uint32_t* anc_flag = nullptr;   // with sel_flag: eight words tagged alike holding the anchor experts (published by the
                             // router kernel, earlier): their gate/up tiles are streamed while the selection still runs
  float* out;                // [T,H], accumulated into (zeroed by the caller)
  int32_t* status;
  int grid;
  bool pdl;                  // launch with programmatic stream serialization
  unsigned long long wait_limit_ns = 1000000000ull;   // the longest any single device-side wait may last
  int32_t* wait_diag = nullptr;   // [grid] per-CTA words: (launch number << 8) | the wait that gave up first (0: none)
  int32_t launch_tag = 0;         // launch number << 8
  const void* mx_gate_up = nullptr;   // MXFP4 layers (launch_ffn_mxfp4): the tiled code + scale tensors
  const void* mx_down = nullptr;
  unsigned long long* trace; // optional [grid][32] device time stamps (acm_stage_timing) or null
};
cudaError_t ffn_configure();   // one-time function attributes
cudaError_t launch_ffn_bf16(const FfnLaunch& p, const FfnMaps& maps, const CUtensorMap& x_map,
                            const CUtensorMap& h_map, const CUtensorMap& h_store_map, cudaStream_t s);
cudaError_t ffn_mx_configure();
cudaError_t launch_ffn_mxfp4(const FfnLaunch& p, const FfnMaps& maps, const CUtensorMap& x_map,
                             const CUtensorMap& h_map, const CUtensorMap& h_store_map, cudaStream_t s);
cudaError_t launch_ffn_f32(const float* x, const float* gate_up, const float* down,
                           const float* shared_gate_up, const float* shared_down, int n_shared,
                           const int32_t* idx, const float* w, float* hbuf, float* out, int T, int H,
                           int I, int E, int k, cudaStream_t s);

}  // namespace acm
