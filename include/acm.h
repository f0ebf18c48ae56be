/*
 * acm.h -- C ABI of the B200 (sm_100a) AcceptMoE verifier-side MoE layer.
 *
 * One call processes ONE speculative-decoding verification block (T <= 64 draft-tree
 * nodes, node 0 = root) through ONE MoE layer of the target model:
 *
 *   stage 1  router logits z_t = W_r x_t (+ bias), r_t = softmax(z_t), natural top-k K_t
 *            (Section 3.1, Eq. 1)
 *   stage 2  commitment-weighted demand u_e (Eq. 3, Eq. 4), root anchor A (Eq. 5),
 *            self-sized eligible set S = A u Top_{n_er}(U_R) (Eq. 6), and under
 *            offloading the residency-aware pruning S -> S' (Eq. 7)
 *   stage 3  top-k routing restricted to S' (Eq. 2) with the target's own weighting
 *   stage 4  grouped SwiGLU expert FFN over the activated experts + weighted combine
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer on the context's device unless marked "host".
 *   - Matrices are row-major and dense.  dtype ACM_BF16: 2-byte bfloat16; ACM_F32: float.
 *   - Expert e (0-based) is bit e%32 of word e/32 in every bitmask (uint32 words).
 *   - All calls are asynchronous on `stream` and return after enqueueing; argument errors
 *     are found on the host before anything is enqueued and leave outputs untouched.
 *     Failures seen by device code (a bounded wait that ran out, a non-finite logit) are
 *     sticky in a status word read by acm_device_status().  Nothing traps, aborts or prints.
 *   - A context serves one stream at a time (its workspace is shared by its calls), and its calls
 *     must not be captured into a CUDA graph: every fused call carries a host-side sequence number
 *     that tags what its kernels hand to one another, so a replay would meet the tags of the run
 *     before it.
 *   - The caller owns every buffer it passes.  The context borrows weight pointers until
 *     acm_destroy() or the next acm_set_layer_weights() for that layer, and owns its
 *     workspace (allocated in acm_create with cudaMalloc on the current device).
 *   - One context serves one stream at a time: calls on the same context that overlap on
 *     the GPU race on its workspace.
 *   - The fused calls expect the GPU to themselves (see acm_set_overlap): by default the expert-FFN kernel is
 *     started ahead of stream order, one CTA per SM, and its CTAs wait on one another.  If other work of
 *     the process (another stream, another context) can hold SMs while a fused call runs, select
 *     ACM_OVERLAP_NONE; otherwise a CTA that finds no SM makes the others wait until their limit runs out
 *     (ACM_ERR_TIMEOUT from acm_device_status, output of that call invalid, context still usable).
 *   - Limits (else ACM_ERR_UNSUPPORTED): n_experts <= 128, top_k <= 8, T <= 64;
 *     bf16: hidden % 128 == 0, inter % 64 == 0; f32: hidden % 32 == 0.
 *
 * Numerical contract of stages 1-3.  Everything that decides a set member, a count or an
 * index is IEEE binary32 in a fixed order: the logit dot product keeps 32 interleaved
 * partial sums (partial l takes h = l, l+32, ... ascending, fused multiply-add) folded by a
 * halving tree; sums over the expert axis use a 128-slot halving tree; exp/log are fixed
 * polynomial recipes; demand accumulates with fused multiply-add over nodes in ascending
 * order; every ranking is total, ties to the lower expert index.  Routing weights and FFN
 * outputs carry no such contract (tensor-core accumulation order is unspecified).
 */
#ifndef ACM_H_
#define ACM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct acm_ctx acm_ctx;          /* opaque */
typedef void* acm_stream;                /* a cudaStream_t (NULL = default stream) */

typedef enum {
  ACM_OK = 0,
  ACM_ERR_INVALID = 1,      /* bad argument */
  ACM_ERR_UNSUPPORTED = 2,  /* outside the limits above */
  ACM_ERR_CUDA = 3,         /* a CUDA runtime/driver call failed */
  ACM_ERR_TIMEOUT = 4,      /* a bounded device-side wait ran out */
  ACM_ERR_NOMEM = 5,
  ACM_ERR_NONFINITE = 6     /* a router logit was NaN or infinite */
} acm_status;

typedef enum { ACM_F32 = 0, ACM_BF16 = 1 } acm_dtype;

/* How the k selected experts' outputs are weighted: restricted routing keeps whatever rule the target model
 * applies after its own top-k (Section 3.1, below Eq. 2), so the rule is a property of the model. */
typedef enum {
  ACM_W_RENORM_TOPK = 0,     /* w = r_e / sum of r over the k selected experts          */
  ACM_W_SOFTMAX_RAW = 1,     /* w = r_e of the unmasked softmax (zero-probability mask) */
  ACM_W_SOFTMAX_MASKED = 2   /* w = softmax over the eligible experts only (logit mask) */
} acm_weighting;

typedef enum {
  ACM_DEMAND_TOPK_MASS = 0,  /* Eq. 4: router mass inside each node's natural top-k */
  ACM_DEMAND_FULL_MASS = 1,  /* sum_t alpha_t r_{t,e} without the indicator (MoE-Spec aggregation) */
  ACM_DEMAND_VOTES = 2       /* natural top-k vote counts */
} acm_demand_mode;

typedef struct {
  int32_t hidden;        /* H */
  int32_t n_experts;     /* E, routed experts */
  int32_t top_k;         /* k */
  int32_t inter;         /* I, per-expert SwiGLU intermediate size */
  int32_t n_shared;      /* always-on shared experts (weight 1, outside selection), 0..4 */
  int32_t max_nodes;     /* largest T that will be passed (<= 64) */
  int32_t n_layers;      /* number of layer slots */
  int32_t dtype;         /* acm_dtype of hidden states and all weights */
  int32_t weighting;     /* acm_weighting */
  float routed_scale;    /* multiplies every routed combine weight (1 = none) */
} acm_model_desc;

typedef struct {
  int32_t demand;        /* acm_demand_mode; 0 = the paper's Eq. 4 */
  int32_t use_anchors;   /* 1 = keep the anchor nodes' natural top-k (Eq. 5) */
  int32_t fixed_budget;  /* 0 = self-sized (Eq. 6); B > 0 = hold the total set size at B */
  float ceil_guard;      /* tau in n_er = ceil(exp(H) - tau); 2^-10 by default, 0 = literal */
  int32_t residency;     /* 0 off; 1 = Eq. 7 pruning; 2 = (S intersect resident) union anchors */
  int32_t max_remove;    /* optional cap on Eq. 7 removals; >= n_experts = nonbinding */
} acm_select_params;

/* Written by device code (all int32 so that it can live in device or pinned memory). */
typedef struct {
  int32_t n_anchor;           /* |A| */
  int32_t n_er;               /* effective-rank cardinality of Eq. 6 (0 if unused) */
  int32_t n_eligible;         /* |S| before pruning */
  int32_t n_eligible_pruned;  /* |S'| */
  int32_t n_activated;        /* eligible experts that received at least one node */
  int32_t n_natural_union;    /* |U_nat| of Eq. 1 */
  int32_t displaced_aS;       /* a(S): natural assignments displaced by restricting to S */
  int32_t pruned_m;           /* m* of Eq. 7 */
  int32_t n_staged;           /* activated experts that were not GPU-resident */
  int32_t n_streamed;         /* routed experts whose weights the block's first FFN launch streamed: the activated ones,
                                 or -- when it starts before the routes exist -- the eligible ones (anchors included) */
  int32_t reserved[2];
} acm_block_stats;

/* Fills the paper's defaults: Eq. 4 demand, anchors on, self-sized, tau = 2^-10, no residency. */
void acm_default_select_params(acm_select_params* p);

/* Creates a context on the current CUDA device and allocates its workspace.  host pointers. */
acm_status acm_create(const acm_model_desc* desc, acm_ctx** out);
acm_status acm_destroy(acm_ctx* ctx);

/* Registers (borrows) the device weights of one layer:
 *   w_router [E,H]; router_bias [E] float or NULL; w_gate_up [E,2I,H] (rows 0..I-1 gate,
 *   I..2I-1 up); w_down [E,H,I]; shared_gate_up [n_shared,2I,H] and shared_down
 *   [n_shared,H,I] (NULL when n_shared == 0).  bf16 expert tensors must be 16-byte aligned.
 *   The weights are constants to the library: their contents must be complete on the device
 *   when this call is made and must not be written while a call that uses the layer is enqueued or
 *   running (the router rows are fetched ahead of stream order, while the kernel before is still
 *   draining).  To change them, synchronise the stream, write, and register them again. */
acm_status acm_set_layer_weights(acm_ctx* ctx, int layer, const void* w_router,
                                 const float* router_bias, const void* w_gate_up,
                                 const void* w_down, const void* shared_gate_up,
                                 const void* shared_down);

/* The same for a layer whose routed experts are stored in MXFP4 (microscaling FP4 -- the storage the
 * paper's offload measurements name for GPT-OSS, Section 4.4): 4-bit E2M1 codes, one E8M0 scale byte
 * (2^(s-127)) per 32 consecutive K elements.  The FFN kernel expands the codes to bf16 on the way to the
 * tensor cores -- every MXFP4 value is a bf16, so the layer computes exactly what a bf16 layer with the
 * dequantised weights computes -- and streams a quarter of the bytes.  The tensors are in the library's
 * tiled layout (one contiguous 8704-byte record per weight tile and pipeline stage):
 *   gate_up_tiles [E][I/64][H/128][8704]: tile t = gate rows 64t..64t+63 then up rows I+64t..I+64t+63,
 *   down_tiles    [E][H/128][I/128][8704]: tile t = rows 128t..128t+127,
 *   record = 128 rows x 64 code bytes, then 128 rows x 4 scale bytes, for 128 consecutive K; each
 *   32-bit word of code bytes holds 8 consecutive K elements, the even ones in the nibbles of its low
 *   half, the odd ones in the nibbles of its high half (element 2j = nibble j, 2j+1 = nibble 4+j).
 *   The four 16-byte pieces of a row's code bytes (32 K each) are stored rotated by the row number:
 *   piece p of row r (0..127 inside the record) at position p ^ ((r >> 1) & 3).
 * Scale bytes above 128 (block scales above 2) are not supported: the tensors are scanned when they are registered
 * (here, and the host tensors in acm_set_slot_pool) and ACM_ERR_UNSUPPORTED is returned.  bf16 contexts with n_shared == 0,
 * hidden % 128 == 0 and inter % 128 == 0 only.  Both tile tensors may be NULL when the layer's experts
 * live in a pool (acm_set_slot_pool, called next): its pool and host tensors are then in this tiled
 * layout too ([n_slots][...] and [E][...]), and a loaded expert costs a quarter of the bf16 bytes.
 * acm_set_resident (the static residency with staging slots) is not available on such a layer. */
acm_status acm_set_layer_weights_mxfp4(acm_ctx* ctx, int layer, const void* w_router,
                                       const float* router_bias, const void* gate_up_tiles,
                                       const void* down_tiles);

/* Eq. 3 on the host: alpha_t = p_table[depth_t]^beta * N_{depth_t}^{-1/2} (width factor
 * optional), evaluated in double and rounded once.  All pointers are HOST pointers.
 * ACM_ERR_INVALID if a depth lies outside the table. */
acm_status acm_node_weights(const int32_t* depth, int T, const float* p_table, int n_depths,
                            float beta, int width_norm, float* alpha_out);

/* Stage 1 (Section 3.1): x [T,H] -> logits [T,E], probs [T,E] (float), nat_idx [T,k]
 * (int32, best first; ties to the lower index).  probs / nat_idx may be NULL. */
acm_status acm_router(acm_ctx* ctx, int layer, const void* x, int T, float* logits,
                      float* probs, int32_t* nat_idx, acm_stream stream);

/* Stage 2 (Sections 3.2-3.4): probs [T,E], nat_idx [T,k], alpha [T] ->
 * eligible_mask [ceil(E/32)] (= S', the set routing is restricted to), eligible_count [1].
 * anchor_nodes: int32 node ids or NULL for {0}.  resident_mask: [ceil(E/32)] words, needed
 * when params->residency != 0.  Optional outputs (may be NULL): demand [E] float,
 * unpruned_mask [ceil(E/32)] (= S), stats [1]. */
acm_status acm_select_eligible(acm_ctx* ctx, const float* probs, const int32_t* nat_idx, int T,
                               const float* alpha, const int32_t* anchor_nodes,
                               int n_anchor_nodes, const acm_select_params* params /*host*/,
                               const uint32_t* resident_mask, uint32_t* eligible_mask,
                               int32_t* eligible_count, float* demand, uint32_t* unpruned_mask,
                               acm_block_stats* stats, acm_stream stream);

/* Stage 3 (Eq. 2): logits [T,E], eligible_mask -> idx [T,k] (int32, best first, -1 where
 * fewer than k experts are eligible), w [T,k] (float combine weights, 0 for empty slots). */
acm_status acm_route_restricted(acm_ctx* ctx, const float* logits, const uint32_t* eligible_mask,
                                int T, int32_t* idx, float* w, acm_stream stream);

/* Stage 4 alone: y_t = sum_j w[t,j] * down_e( silu(gate_e x_t) * up_e x_t ), e = idx[t,j]
 * (+ shared experts with weight 1).  x [T,H], idx/w [T,k] -> out [T,H] float (overwritten). */
acm_status acm_expert_ffn(acm_ctx* ctx, int layer, const void* x, int T, const int32_t* idx,
                          const float* w, float* out, acm_stream stream);

/* Stages 1-4 for one block and layer.  alpha [T] device.  eligible_mask_override != NULL
 * skips stage 2 and routes inside the given set (all ones = the natural-routing union path).
 * Optional outputs (NULL to skip): idx_out [T,k], w_out [T,k], mask_out [ceil(E/32)],
 * stats [1].  out [T,H] float is overwritten.  stats in memory of the context's device is written
 * by the kernels themselves; anywhere else (pinned host memory) it is copied at the end of the
 * call, and so are idx_out, w_out and mask_out -- a copy between this call's last kernel and the
 * next call's first ends the overlap of the two, so ask only for what is needed in a tight loop.
 * With a residency registered for the layer (acm_set_resident) and params->residency != 0,
 * activated experts that are not GPU-resident are copied from the registered pinned host
 * tensors into the context's staging slots before their FFN runs; this needs one host
 * synchronisation on `stream` inside the call. */
acm_status acm_moe_verify(acm_ctx* ctx, int layer, const void* x, int T, const float* alpha,
                          const acm_select_params* params /*host*/,
                          const uint32_t* eligible_mask_override, float* out, int32_t* idx_out,
                          float* w_out, uint32_t* mask_out, acm_block_stats* stats,
                          acm_stream stream);

/* Multi-block batch (the paper verifies one block at a time, Section 4.1 "batch size one"; this is the
 * same layer step for several verification blocks that share one pass over the expert weights).  The
 * blocks' nodes are stacked along the node axis: block b owns rows block_offsets[b] ..
 * block_offsets[b+1]-1 of x [T,hidden], alpha [T], out, idx_out, w_out (T = block_offsets[n_blocks] <=
 * 128, every block at most max_nodes <= 64 rows -- two full blocks fit; block_offsets is a HOST array of
 * n_blocks+1 ascending entries starting at 0; every block has at least one node and its first row is its
 * root; MXFP4 layers: T <= 64).  Stages 1-3 run per block exactly as in
 * acm_moe_verify: block b's eligible set comes from its own nodes (Eq. 3-7) and its nodes are routed
 * inside it (Eq. 2), so every per-block result equals that of a single-block call on the block's rows.
 * Stage 4 runs once over all rows: an expert activated by several blocks is streamed from HBM once.
 * mask_out [n_blocks][ceil(E/32)] = the blocks' eligible sets; activated_out [ceil(E/32)] = the union of
 * activated experts (what was streamed); stats [n_blocks] (n_activated = experts activated by that
 * block's own nodes).  All optional, device (stats: device or pinned).  bf16 layers without a
 * residency only (ACM_ERR_UNSUPPORTED otherwise). */
acm_status acm_moe_verify_batch(acm_ctx* ctx, int layer, const void* x, int n_blocks,
                                const int32_t* block_offsets /*host*/, const float* alpha,
                                const acm_select_params* params /*host*/, float* out, int32_t* idx_out,
                                float* w_out, uint32_t* mask_out, uint32_t* activated_out,
                                acm_block_stats* stats, acm_stream stream);

/* The same call for HOST buffers (Section 3.1's per-layer step as a serving loop sees it): x_host
 * [T,H] and alpha_host [T] are read from, and out_host [T,H] float is written to, PINNED host
 * memory.  The copies run on the context's own copy streams through two alternating sets of device
 * buffers, so the upload of the next block and the download of the previous one overlap this block's
 * kernels; the kernels run on `stream`.  The call returns once everything is enqueued.  out_host and
 * stats_host (optional, host) are valid after acm_host_synchronize(); x_host and alpha_host must stay
 * unchanged until then (or until two later calls of this function have returned and `stream` has
 * passed them).  Not available with a residency registered for the layer. */
acm_status acm_moe_verify_host(acm_ctx* ctx, int layer, const void* x_host, int T,
                               const float* alpha_host, const acm_select_params* params /*host*/,
                               float* out_host, acm_block_stats* stats_host, acm_stream stream);

/* Waits until every copy enqueued by acm_moe_verify_host has completed. */
acm_status acm_host_synchronize(acm_ctx* ctx);

/* Offload variant (Section 3.4): marks which experts of `layer` are GPU-resident
 * (resident_mask: HOST words) and registers pinned HOST copies of the full expert tensors
 * used to load non-resident experts on demand.  The device tensors registered with
 * acm_set_layer_weights are then read only at resident experts.  NULL mask clears it. */
acm_status acm_set_resident(acm_ctx* ctx, int layer, const uint32_t* resident_mask,
                            const void* host_gate_up, const void* host_down);

/* Offload variant with the per-layer expert pool of Section 3.4 (a fixed number of expert slots in GPU memory,
 * replaced least-recently-used first): the layer's routed experts live in `n_slots` slots of the caller's device tensors
 * pool_gate_up [n_slots,2I,H] / pool_down [n_slots,H,I] (128-byte aligned; the tensors given to
 * acm_set_layer_weights may then be NULL), the full weights in PINNED host tensors [E,...].  The first
 * n_initial slots are filled with initial_experts (host ids; copied synchronously).  From then on, with
 * params->residency != 0, acm_moe_verify takes the pool's current contents as the resident set H of
 * Eq. 7; an activated expert that is not in the pool is copied into the least recently used slot this
 * block does not use before its FFN runs, and stays for later blocks.  When the activated experts
 * outnumber the free slots the loads go in waves (each wave: copies, then one FFN launch over the experts
 * just loaded; a later wave waits for the launch before it and may replace any slot).  One host
 * synchronisation on `stream` per call, as with acm_set_resident.  acm_set_resident(layer, NULL, ...)
 * removes the pool. */
acm_status acm_set_slot_pool(acm_ctx* ctx, int layer, int n_slots, void* pool_gate_up, void* pool_down,
                             const void* host_gate_up, const void* host_down,
                             const int32_t* initial_experts /*host*/, int n_initial);

/* Pool counters since the last reset (host pointers, any may be NULL): activated experts found in the
 * pool, activated experts loaded, bytes loaded; slot_expert [n_slots] = expert id in each slot or -1. */
acm_status acm_pool_stats(acm_ctx* ctx, int layer, uint64_t* hits, uint64_t* misses, uint64_t* h2d_bytes,
                          int32_t* slot_expert, int reset);

/* The pool's replacement policy by itself (pure host code, no GPU; what acm_moe_verify runs for a layer with
 * a pool).  One block: the activated experts (mask words, host) found in the pool are hits and count as used
 * now; the others are loaded in ascending id, wave by wave.  Wave 0 runs beside the FFN over the hits and may
 * only take slots this block does not use; every later wave may replace any slot not loaded in the same wave.
 * Inside a wave the victim is the least recently used slot it may take (empty slots first, ties to the lower
 * slot).  In-out (host): slot_expert [n_slots] (expert id or -1), last_use [n_slots], *tick (advanced by one).
 * Out (host, room for n_experts entries each): load i puts load_expert[i] into load_slot[i] in wave
 * load_wave[i]; *n_loads, *n_hits. */
acm_status acm_pool_plan(int n_experts, int n_slots, int32_t* slot_expert, uint64_t* last_use, uint64_t* tick,
                         const uint32_t* activated_mask, int32_t* load_expert, int32_t* load_slot,
                         int32_t* load_wave, int32_t* n_loads, int32_t* n_hits);

/* Host->device bytes copied for non-resident experts since the last call with reset != 0. */
acm_status acm_h2d_bytes(acm_ctx* ctx, uint64_t* bytes_out /*host*/, int reset);

/* Per-launch timing of the expert-FFN kernel with CUDA events on the launching stream.
 * enable = n > 0 starts recording every n-th launch of that kernel, counted from this call (n = 1:
 * every launch; at most `capacity` launches are kept); enable = 0 stops.  A bracketed launch is
 * ordered strictly after the kernel before it (no dependent-launch overlap), so its duration is the
 * kernel's own.  acm_ffn_time_ms synchronises the events and returns their summed duration and
 * count (host pointers). */
acm_status acm_ffn_timing(acm_ctx* ctx, int enable, int capacity);
acm_status acm_ffn_time_ms(acm_ctx* ctx, float* total_ms, int32_t* launches);

/* Offload variant (Section 3.4): where a call's time goes on a layer with a static residency (acm_set_resident).
 * acm_offload_timing(enable, capacity) starts (enable != 0) or stops recording CUDA events in up to `capacity`
 * such calls; acm_offload_times synchronises them and returns sums over the recorded calls, ms_out [4] (host,
 * milliseconds): [0] whole call on the device, from before its first kernel to after its last; [1] from there to
 * the end of the FFN over the experts that were resident; [2] the host-to-device copies of the loaded experts
 * (on the copy stream); [3] the stall: how long the copies went on after the resident part was done, i.e. the
 * time the stream spent waiting for them -- [0] minus [3] is the call without its host-to-device wait. */
acm_status acm_offload_timing(acm_ctx* ctx, int enable, int capacity);
acm_status acm_offload_times(acm_ctx* ctx, double* ms_out /*host [4]*/, int32_t* calls /*host*/);

/* Per-stage device times of the fused call, from time stamps the kernels themselves take (one global
 * nanosecond clock) -- the launch sequence, its overlaps included, stays as it is.  acm_stage_timing
 * switches the stamps on or off (it synchronises the device; on costs a few stores per CTA).
 * acm_stage_times synchronises and reports, for the LAST acm_moe_verify call on a bf16 layer without a
 * residency, us_out [5] (host, microseconds):
 *   [0] stage 1: from the router kernel passing its dependency wait (everything before it in the
 *       stream is complete) to the selection kernel passing its own -- the logits;
 *   [1] stage 2: softmax and natural top-k (Eq. 1) and the selection (Eq. 4-7), until the eligible set
 *       is published;
 *   [2] stage 3: the routes (Eq. 2) and the FFN kernel's routing inputs;
 *   [3] stage 4: the FFN kernel from its first CTA's roles starting to its last tile finished -- it
 *       starts on the anchor experts while stages 1 and 2 still run, so [0..3] overlap and do not add up to
 *   [4] the whole: from the start of [0] to the end of [3].
 * ACM_ERR_INVALID when the stamps are off or no such call has run. */
acm_status acm_stage_timing(acm_ctx* ctx, int enable);
acm_status acm_stage_times(acm_ctx* ctx, double* us_out /*host [5]*/);

/* Number of kernel launches this context has enqueued since creation (host counter). */
acm_status acm_launch_count(acm_ctx* ctx, uint64_t* launches_out /*host*/);

/* Allocation-free expert FFN for fp32 layers (the paper has no counterpart: this exists for
 * callers that must not allocate device memory when they call -- code running inside a memory
 * pool it does not own, under an allocator that is frozen, or where cudaMalloc's implicit
 * device synchronisation is not acceptable).  Same computation as acm_expert_ffn on an ACM_F32
 * layer without shared experts: y_t = sum_j w[t,j] * down_e( silu(gate_e x_t) * up_e x_t ),
 * e = idx[t,j] (-1 = empty slot).  All pointers are device pointers: x [T,hidden], idx/w
 * [T,top_k], w_gate_up [n_experts,2*inter,hidden], w_down [n_experts,hidden,inter], out
 * [T,hidden] (overwritten).  It needs no context and calls no allocator: the intermediate
 * activations go to a fixed 4 MiB array inside the library image, which every GPU that loads
 * the library holds until the process exits.
 *   - Limit: T * top_k * inter <= ACM_NOALLOC_MAX_FLOATS (2^20), T <= 64, top_k <= 8,
 *     n_experts <= 128; anything larger returns ACM_ERR_UNSUPPORTED and launches nothing.
 *   - The first call on each device looks up that device's address of the array (one
 *     cudaGetSymbolAddress, with that device current); make that first call before starting
 *     any stream capture.
 *   - Every call uses the same array and leaves its contents behind.  Nothing in it has to be
 *     zero on entry (each element is written before it is read), but two calls that overlap on
 *     the GPU -- different streams, or different threads -- race on it: serialise them. */
#define ACM_NOALLOC_MAX_FLOATS (1u << 20)
acm_status acm_expert_ffn_f32_noalloc(const float* x, int T, int hidden, int inter, int n_experts,
                                      int top_k, const int32_t* idx, const float* w,
                                      const float* w_gate_up, const float* w_down, float* out,
                                      acm_stream stream);

/* The expert-FFN kernel's work plan, listed on the host (no GPU is touched): how one launch that streams
 * n_experts_streamed experts of a bf16 layer (hidden, inter) on `grid` CTAs deals its weight tiles, for inspection
 * and for tests of the plan's coverage.  n_anchor_first > 0 lists the plan of a launch that starts on that many
 * anchor experts (Eq. 5) before the rest of the set is known (their tiles, one per CTA, are segment 0).
 * pieces [capacity][8] (host) receives, in each
 * CTA's execution order: CTA, segment, phase (1 = gate/up: 64 gate + 64 up rows x hidden; 2 = down: 128 output
 * rows), for gate/up whether the tile is given whole (1) or cut along K (0) (down: 0), the tile (gate/up: slot *
 * inter/64 + sub-tile; down: output tile), the piece's
 * first and one-past-last K-chunk of 128 K (down: counted through the segment's expert group), and the cut
 * segment's exchange buffer (gate/up) or the group's first expert slot (down).  ACM_ERR_NOMEM if capacity is too
 * small (*n_pieces then tells how many there are). */
acm_status acm_ffn_plan(int n_experts_streamed, int n_anchor_first, int hidden, int inter, int grid,
                        int32_t* pieces /*host*/, int capacity, int32_t* n_pieces /*host*/, int32_t* n_segments /*host*/);

/* How far the kernels of a fused call (acm_moe_verify, acm_moe_verify_batch, acm_moe_verify_host) overlap.
 * The stages of Section 3.1-3.4 form a chain, and the expert FFN needs only part of its result to start:
 *   ACM_OVERLAP_NONE       plain stream order.  The FFN kernel is a cooperative launch, so the driver itself
 *                          checks that all its CTAs can be resident together.  The mode to use when anything
 *                          else may run on the GPU at the same time.
 *   ACM_OVERLAP_DEPENDENT  each kernel is launched as a programmatic dependent of the one before: it is
 *                          resident and set up while its predecessor drains, then waits for it.
 *   ACM_OVERLAP_ELIGIBLE   ... and the FFN kernel starts streaming as soon as the eligible set S' (Eq. 6, 7)
 *                          is published, before the routes (Eq. 2) are written.
 *   ACM_OVERLAP_ANCHORS    ... and before that on the anchor experts (Eq. 5), which are in every eligible
 *                          set, while the selection still runs.  The default.
 * From ACM_OVERLAP_DEPENDENT on, the FFN kernel's CTAs (one per SM, they exchange partial sums) are not
 * checked for co-residency by the driver: the GPU must be otherwise idle while a fused call runs.
 * Takes effect from the next call; results do not depend on the level. */
typedef enum {
  ACM_OVERLAP_NONE = 0,
  ACM_OVERLAP_DEPENDENT = 1,
  ACM_OVERLAP_ELIGIBLE = 2,
  ACM_OVERLAP_ANCHORS = 3
} acm_overlap;
acm_status acm_set_overlap(acm_ctx* ctx, int level);

/* Every device-side wait (on a barrier, a counter another CTA raises, a word an earlier kernel publishes) is
 * bounded: after `nanoseconds` without progress the waiting CTA raises ACM_ERR_TIMEOUT in the status word,
 * lets its copies in flight land, frees its tensor memory and returns; the launch's output is then invalid
 * and acm_device_status re-arms the workspace.  Default 1 s; 1 us .. 60 s (else ACM_ERR_INVALID).  Healthy
 * waits last microseconds, so a few milliseconds are safe on an idle GPU. */
acm_status acm_set_wait_limit(acm_ctx* ctx, uint64_t nanoseconds);

/* After ACM_ERR_TIMEOUT: which wait of the LAST expert-FFN launch gave up first in each of its CTAs.
 * Synchronises the device.  site_out [capacity] (host): 0 = that CTA saw no wait run out, -1 = that CTA never
 * started (it found no SM), else a wait-site number (1, 2: words published by the router / selection kernel;
 * 3-5: the CTA's own pipeline; 6-10: data from other CTAs; 11-16: hand-overs inside the CTA; 17: the rest of
 * the plan; 18: a packed MXFP4 stage).  *n_ctas = CTAs of that launch.  Call it before acm_device_status
 * clears the state, or after: the words are kept until the next launch. */
acm_status acm_wait_report(acm_ctx* ctx, int32_t* site_out /*host*/, int capacity, int32_t* n_ctas /*host*/);

/* Failure injection for tests of the error path above (made on the host; nothing faults): launches the
 * expert-FFN kernel of a bf16 layer in its early-start form, waiting for an eligible set (Eq. 6) under a
 * sequence tag that no selection kernel is ever given.  Every CTA's first wait therefore runs out after the
 * wait limit: the kernel returns, acm_device_status reports ACM_ERR_TIMEOUT and re-arms the workspace, and
 * the next call on the context must be correct again.  out [T,hidden] is zeroed.  Set a short limit first
 * (acm_set_wait_limit): the call keeps the GPU busy for that long. */
acm_status acm_inject_unpublished_wait(acm_ctx* ctx, int layer, const void* x, int T, float* out,
                                       acm_stream stream);

/* Synchronises `stream` and returns the sticky device-side status (ACM_OK if none), then clears it. */
acm_status acm_device_status(acm_ctx* ctx, acm_stream stream);

const char* acm_status_string(acm_status s);

#ifdef __cplusplus
}
#endif
#endif  /* ACM_H_ */
