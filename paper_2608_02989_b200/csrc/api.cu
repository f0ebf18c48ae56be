// Host side of the C ABI declared in include/acm.h: context and workspace, argument checks,
// TMA descriptors, launch sequencing, on-demand host->device staging of non-resident experts.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "acm_internal.h"
#include "ffn_plan.h"

using namespace acm;

namespace {

struct Layer {
  const void* w_router = nullptr;
  const float* bias = nullptr;
  const void* gate_up = nullptr;
  const void* down = nullptr;
  const void* shared_gate_up = nullptr;
  const void* shared_down = nullptr;
  FfnMaps maps;
  bool set = false;
  bool mx = false;                      // MXFP4 layer (acm_set_layer_weights_mxfp4): expert tensors are tiled codes + scales
  const void* mx_gate_up = nullptr;     // [E][I/64][H/128][8704] (null when the experts only live in a pool)
  const void* mx_down = nullptr;
  bool has_resident = false;
  const void* host_gate_up = nullptr;   // pinned host copies for on-demand loads
  const void* host_down = nullptr;
  // LRU expert pool (acm_set_slot_pool): the layer's experts live in n_slots device slots
  bool has_pool = false;
  int n_slots = 0;
  void* pool_gate_up = nullptr;         // device [n_slots, 2I, H]
  void* pool_down = nullptr;            // device [n_slots, H, I]
  CUtensorMap pool_map_gu, pool_map_dn;
  std::vector<int32_t> slot_expert;     // slot -> expert id or -1
  std::vector<int32_t> expert_slot;     // expert id -> slot or -1
  std::vector<uint64_t> last_use;       // slot -> tick of its last use
  uint64_t tick = 0;
  int32_t* slot_of_dev[2] = {nullptr, nullptr};   // device copies of expert_slot, alternating (see acm_moe_verify)
  int slot_of_cur = 0;
  uint64_t pool_hits = 0, pool_misses = 0, pool_h2d = 0, pool_waves = 0;
};

// The pool's replacement policy for ONE block, pure host logic (no CUDA): given the pool's state and the
// block's activated experts, marks the hits as used now and plans the loads of the misses, in ascending expert
// id, wave by wave.  Wave 0 runs beside the FFN over the hits, so it may only take slots this block does not
// use; every later wave starts after the FFN launched before it and may replace any slot not loaded in the
// same wave.  Within a wave the victim is the least recently used eligible slot (empty slots count as never
// used; ties go to the lower slot).  Returns false on an inconsistent state.
constexpr int kSlotTableRing = 32;
struct PoolLoad {
  int32_t expert, slot, wave;
};
bool plan_pool_block(int E, int n_slots, std::vector<int32_t>& slot_expert, std::vector<int32_t>& expert_slot,
                     std::vector<uint64_t>& last_use, uint64_t& tick, const uint32_t* act, std::vector<PoolLoad>& loads,
                     int& n_hits) {
  loads.clear();
  n_hits = 0;
  tick += 1;
  std::vector<int32_t> misses;
  for (int e = 0; e < E; ++e) {
    if (!((act[e >> 5] >> (e & 31)) & 1u)) continue;
    if (expert_slot[e] >= 0) {
      last_use[expert_slot[e]] = tick;
      n_hits += 1;
    } else {
      misses.push_back(e);
    }
  }
  if (n_hits > n_slots) return false;
  std::vector<int32_t> wave_of(n_slots, -1);
  size_t done = 0;
  int wave = 0;
  while (done < misses.size()) {
    while (done < misses.size()) {
      int victim = -1;
      for (int sl = 0; sl < n_slots; ++sl) {
        if (wave_of[sl] == wave) continue;                  // just loaded for this wave
        if (wave == 0 && last_use[sl] == tick) continue;    // in use by the FFN over the hits
        if (victim < 0 || last_use[sl] < last_use[victim]) victim = sl;
      }
      if (victim < 0) break;                                // this wave is full
      const int e = misses[done];
      if (slot_expert[victim] >= 0) expert_slot[slot_expert[victim]] = -1;
      slot_expert[victim] = e;
      expert_slot[e] = victim;
      last_use[victim] = tick;
      wave_of[victim] = wave;
      loads.push_back(PoolLoad{e, victim, wave});
      ++done;
    }
    ++wave;
    if (wave > static_cast<int>(misses.size()) + 1) return false;   // cannot happen: every wave after the first has room
  }
  return true;
}

// MXFP4 tile records: 128 x 64 code bytes, then 128 x 4 E8M0 scale bytes.  The FFN kernel applies a scale with one
// bf16 multiply, which covers block scales up to 2 (scale byte 128); larger ones are refused at registration.
constexpr size_t kMxRecordBytes = 128 * 64 + 128 * 4;
constexpr int kMxMaxScaleByte = 128;
__global__ void k_mx_max_scale(const unsigned char* tiles, size_t n_records, int* max_out) {
  int m = 0;
  for (size_t r = blockIdx.x; r < n_records; r += gridDim.x) {
    const unsigned char* sc = tiles + r * kMxRecordBytes + 128 * 64;
    for (int i = threadIdx.x; i < 512; i += blockDim.x) m = max(m, static_cast<int>(sc[i]));
  }
  m = __reduce_max_sync(0xffffffffu, m);
  if ((threadIdx.x & 31) == 0 && m > 0) atomicMax(max_out, m);
}
int mx_max_scale_host(const unsigned char* tiles, size_t n_records) {
  int m = 0;
  for (size_t r = 0; r < n_records; ++r) {
    const unsigned char* sc = tiles + r * kMxRecordBytes + 128 * 64;
    for (int i = 0; i < 512; ++i) m = sc[i] > m ? sc[i] : m;
  }
  return m;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

struct acm_ctx {
  acm_model_desc desc;
  int device = 0;
  int sm_count = 0;
  void* ws_base = nullptr;
  Workspace ws;
  uint32_t* resident_dev = nullptr;      // [n_layers][4]
  std::vector<Layer> layers;
  EncodeTiledFn encode = nullptr;
  int32_t epoch = 0;
  size_t frag_bytes = 0, flag_bytes = 0;   // fragment buffers and arrival counters (zero between launches)
  CUtensorMap h_map[2];
  CUtensorMap h_store_map[2];            // same buffers, one 64-feature tile per TMA store
  int h_map_npad = 0;
  // staging of non-resident experts
  void* stage_gate_up = nullptr;
  void* stage_down = nullptr;
  CUtensorMap stage_map_gu, stage_map_dn;
  int32_t* host_stage_list = nullptr;    // pinned + mapped: [0] = count, [1..] = expert ids
  int32_t* host_stage_list_dev = nullptr;
  int32_t* slot_table_pinned = nullptr;        // pinned ring of expert -> slot tables in flight (kSlotTableRing x kMaxExperts)
  uint64_t slot_table_next = 0;
  uint32_t* resident_words_pinned = nullptr;   // pinned ring of resident-mask updates in flight (64 x 4 words)
  unsigned long long resident_words_next = 0;
  bool pool_waves_list1_used = false;   // within one call: the second work list has been used by an earlier wave
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_lists = nullptr, ev_copied = nullptr, ev_stage_free = nullptr;
  bool stage_in_use = false;
  uint64_t h2d_bytes = 0;
  // host-buffer path (acm_moe_verify_host): two alternating sets of device buffers and copy streams
  cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
  void* hx_dev[2] = {nullptr, nullptr};
  float* halpha_dev[2] = {nullptr, nullptr};
  float* hout_dev[2] = {nullptr, nullptr};
  acm_block_stats* hstats_dev[2] = {nullptr, nullptr};
  cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_done[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr};
  unsigned long long host_calls = 0;
  size_t host_h2d = 0, host_d2h = 0;   // bytes copied by that path
  // per-launch FFN timing
  size_t ffn_in_floats = 0;     // length of the block wtab | ready | act_mask, in floats
  bool timing = false;
  int timing_period = 1;        // every n-th FFN launch is bracketed by events
  long long timing_seen = 0;
  // how far the kernels of a fused call overlap (acm_set_overlap)
  int overlap = ACM_OVERLAP_ANCHORS;
  bool pdl = true;              // >= DEPENDENT: programmatic dependent launches between the kernels of the hot path
  bool early_start = true;      // >= ELIGIBLE: the FFN kernel starts on the eligible set, before the routes are final
  bool anchor_start = true;     // ANCHORS: ... and before that on the anchors, while the selection runs
  std::vector<cudaEvent_t> ev_pool;
  size_t ev_used = 0;
  uint64_t launches = 0;
  unsigned long long* trace = nullptr;   // acm_stage_timing: per-CTA time stamps of the last FFN launch + the routing kernels' stamps
  bool mx_configured = false;
  // offload timing (acm_offload_timing): five events per call on a layer with a static residency
  bool off_timing = false;
  std::vector<cudaEvent_t> off_ev;
  std::vector<unsigned char> off_has_copies;   // per recorded call: did it load anything?
  size_t off_calls = 0;
  // bounded device-side waits (acm_set_wait_limit, acm_wait_report)
  unsigned long long wait_limit_ns = 1000000000ull;
  int32_t* wait_diag = nullptr;          // [sm_count] per-CTA words of the FFN kernel
  int32_t ffn_launch_no = 0;             // numbers the FFN launches (24 bits are kept in the words)
  int last_ffn_grid = 0;
};

namespace {

#define ACM_CUDA(expr)                         \
  do {                                         \
    cudaError_t e__ = (expr);                  \
    if (e__ != cudaSuccess) return ACM_ERR_CUDA; \
  } while (0)

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int mask_words(int E) { return (E + 31) / 32; }

acm_status check_desc(const acm_model_desc& d) {
  if (d.hidden <= 0 || d.n_experts <= 0 || d.top_k <= 0 || d.inter <= 0 || d.n_shared < 0 || d.max_nodes <= 0 ||
      d.n_layers <= 0 || d.top_k > d.n_experts)
    return ACM_ERR_INVALID;
  if (d.dtype != ACM_F32 && d.dtype != ACM_BF16) return ACM_ERR_INVALID;
  if (d.weighting < 0 || d.weighting > 2) return ACM_ERR_INVALID;
  if (!std::isfinite(d.routed_scale)) return ACM_ERR_INVALID;
  if (d.n_experts > kMaxExperts || d.top_k > kMaxTopK || d.max_nodes > kMaxNodes || d.n_shared > kMaxShared)
    return ACM_ERR_UNSUPPORTED;
  if (d.dtype == ACM_BF16 && (d.hidden % 128 != 0 || d.inter % 64 != 0)) return ACM_ERR_UNSUPPORTED;
  if (d.dtype == ACM_F32 && d.hidden % 32 != 0) return ACM_ERR_UNSUPPORTED;
  return ACM_OK;
}

acm_status check_params(const acm_select_params* p) {
  if (!p) return ACM_ERR_INVALID;
  if (p->demand < 0 || p->demand > 2 || p->fixed_budget < 0 || p->residency < 0 || p->residency > 2 ||
      p->max_remove < 0 || !(p->ceil_guard >= 0.0f) || !(p->ceil_guard < 1.0f))
    return ACM_ERR_INVALID;
  return ACM_OK;
}

// bf16 tensor view for TMA with 128-byte swizzle.  Dimension 0 is always one 64-element (128-byte)
// swizzle atom along K; the atom index is a dimension of its own, so that one copy can fetch
// several atoms of the same rows and lay them out in shared memory atom after atom.
acm_status encode_view(acm_ctx* c, CUtensorMap* m, const void* base, int rank, const uint64_t* dims,
                       const uint64_t* strides_bytes /* rank-1 entries, for dims 1.. */, const uint32_t* box) {
  if (reinterpret_cast<uintptr_t>(base) % 16 != 0) return ACM_ERR_INVALID;
  cuuint64_t d[5], st[4];
  cuuint32_t bx[5], es[5];
  for (int i = 0; i < rank; ++i) {
    d[i] = dims[i];
    bx[i] = box[i];
    es[i] = 1;
    if (i > 0) st[i - 1] = strides_bytes[i - 1];
  }
  const CUresult r = c->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(base), d, st, bx, es,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? ACM_OK : ACM_ERR_CUDA;
}

// gate_up [n, 2I, H] as {k in atom, row in I, gate|up, atom of H, expert}; one box = 64 gate rows +
// the 64 matching up rows x 2 atoms (32 KB), stored atom-major: [atom][gate rows, up rows][64].
acm_status encode_gate_up(acm_ctx* c, CUtensorMap* m, const void* base, uint64_t n) {
  const uint64_t H = c->desc.hidden, I = c->desc.inter;
  const uint64_t dims[5] = {64, I, 2, H / 64, n};
  const uint64_t strides[4] = {H * 2, I * H * 2, 128, 2 * I * H * 2};
  const uint32_t box[5] = {64, 64, 2, 2, 1};
  return encode_view(c, m, base, 5, dims, strides, box);
}
// down [n, H, I] as {k in atom, row in H, atom of I, expert}; one box = 128 rows x 2 atoms (32 KB).
acm_status encode_down(acm_ctx* c, CUtensorMap* m, const void* base, uint64_t n) {
  const uint64_t H = c->desc.hidden, I = c->desc.inter;
  const uint64_t dims[4] = {64, H, I / 64, n};
  const uint64_t strides[3] = {I * 2, 128, H * I * 2};
  const uint32_t box[4] = {64, 128, 2, 1};
  return encode_view(c, m, base, 4, dims, strides, box);
}
// x [T, H] as {k in atom, node, atom of H}; one box = n_pad nodes x 2 atoms.
acm_status encode_x(acm_ctx* c, CUtensorMap* m, const void* x, int T, int n_pad) {
  const uint64_t H = c->desc.hidden;
  const uint64_t dims[3] = {64, static_cast<uint64_t>(T), H / 64};
  const uint64_t strides[2] = {H * 2, 128};
  const uint32_t box[3] = {64, static_cast<uint32_t>(n_pad), 2};
  return encode_view(c, m, x, 3, dims, strides, box);
}
// activations [slots, 64, I] as {k in atom, node, atom of I, slot}; one box = n_pad nodes x 2 atoms.
acm_status encode_h(acm_ctx* c, CUtensorMap* m, const void* base, int n_pad, int atoms) {
  const uint64_t I = c->desc.inter;
  const uint64_t dims[4] = {64, kWideNodes, I / 64, kMaxSlots};
  const uint64_t strides[3] = {I * 2, 128, kWideNodes * I * 2};
  const uint32_t box[4] = {64, static_cast<uint32_t>(n_pad), static_cast<uint32_t>(atoms), 1};
  return encode_view(c, m, base, 4, dims, strides, box);
}

acm_status ensure_h_maps(acm_ctx* c, int n_pad) {
  if (c->h_map_npad == n_pad) return ACM_OK;
  const size_t list_bytes = static_cast<size_t>(kMaxSlots) * kWideNodes * c->desc.inter * 2;
  for (int l = 0; l < 2; ++l) {
    acm_status st = encode_h(c, &c->h_map[l], static_cast<char*>(c->ws.hbuf) + l * list_bytes, n_pad, 2);
    if (st != ACM_OK) return st;
    // (stored 64 node rows at a time: a wide tile in two halves)
    st = encode_h(c, &c->h_store_map[l], static_cast<char*>(c->ws.hbuf) + l * list_bytes, n_pad < kMaxNodes ? n_pad : kMaxNodes, 1);
    if (st != ACM_OK) return st;
  }
  c->h_map_npad = n_pad;
  return ACM_OK;
}

acm_status check_block_args(const acm_ctx* c, int layer, int T, bool need_weights) {
  if (!c) return ACM_ERR_INVALID;
  if (layer < 0 || layer >= c->desc.n_layers) return ACM_ERR_INVALID;
  if (T < 1 || T > c->desc.max_nodes) return ACM_ERR_INVALID;
  if (need_weights && !c->layers[layer].set) return ACM_ERR_INVALID;
  return ACM_OK;
}

// Where the kernels write a call's statistics: straight into the caller's buffer when that is memory of this
// device (no copy node then sits between this call's last kernel and the next call's first, which would end the
// overlap of the two), else into the workspace, copied out at the end of the call.
acm_block_stats* stats_target(acm_ctx* c, acm_block_stats* user, bool* direct) {
  *direct = false;
  if (!user) return c->ws.stats;
  cudaPointerAttributes attr;
  if (cudaPointerGetAttributes(&attr, user) == cudaSuccess && attr.type == cudaMemoryTypeDevice && attr.device == c->device) {
    *direct = true;
    return user;
  }
  cudaGetLastError();      // (an unregistered host pointer sets an error on some drivers)
  return c->ws.stats;
}

// bytes of one expert's gate/up and down tensors as the layer stores them (bf16, or MXFP4 tile records)
void expert_tensor_bytes(const acm_model_desc& d, bool mx, size_t* gu, size_t* dn) {
  if (mx) {
    const size_t rec = 128 * 64 + 128 * 4;
    *gu = static_cast<size_t>(d.inter / 64) * (d.hidden / 128) * rec;
    *dn = static_cast<size_t>(d.hidden / 128) * (d.inter / 128) * rec;
  } else {
    *gu = static_cast<size_t>(2) * d.inter * d.hidden * 2;
    *dn = static_cast<size_t>(d.hidden) * d.inter * 2;
  }
}

// One FFN launch over work list `li` (0 = resident + shared, 1 = staged).
acm_status run_ffn_list(acm_ctx* c, const Layer& L, const void* x, int T, int li, float* out, cudaStream_t s,
                        const uint32_t* res_dev = nullptr, acm_block_stats* stats_dev = nullptr, bool pdl_ok = false,
                        int32_t early_epoch = 0, const uint32_t* only = nullptr, int n_blocks = 0,
                        bool anchors_first = false, int widest_block = 0) {
  const acm_model_desc& d = c->desc;
  const int n_pad = (T + 15) / 16 * 16;
  acm_status st = ensure_h_maps(c, n_pad);
  if (st != ACM_OK) return st;
  CUtensorMap x_map;
  st = encode_x(c, &x_map, x, T, n_pad);
  if (st != ACM_OK) return st;
  FfnMaps maps = L.maps;
  if (L.has_pool) {
    maps.staged_gate_up = L.pool_map_gu;
    maps.staged_down = L.pool_map_dn;
  } else if (c->stage_gate_up) {
    maps.staged_gate_up = c->stage_map_gu;
    maps.staged_down = c->stage_map_dn;
  }
  FfnLaunch p;
  p.T = T; p.H = d.hidden; p.I = d.inter; p.n_pad = n_pad;
  p.act_mask = c->ws.act_mask;
  p.resident = res_dev;
  p.li = li;
  for (int w = 0; w < 4; ++w) p.only[w] = only ? only[w] : 0xffffffffu;
  p.n_shared = d.n_shared;
  p.slot_of = L.has_pool ? L.slot_of_dev[L.slot_of_cur] : nullptr;
  p.wtab = c->ws.wtab;
  p.stats = stats_dev;
  p.hbuf = static_cast<char*>(c->ws.hbuf) + static_cast<size_t>(li) * kMaxSlots * kWideNodes * d.inter * 2;
  p.ready = c->ws.ready + li * kMaxSlots;
  p.frag = c->ws.frag; p.frag_flag = c->ws.frag_flag;
  p.sel_flag = nullptr; p.sel_epoch = 0; p.sel_blocks = n_blocks > 0 ? n_blocks : 1;
  if (early_epoch != 0) {
    p.sel_flag = c->ws.sel_words;
    p.sel_epoch = early_epoch;
  }
  p.out = out; p.status = c->ws.status;
  p.grid = c->sm_count;
  p.trace = c->trace;
  p.pdl = false;
  p.wait_limit_ns = c->wait_limit_ns;
  p.wait_diag = c->wait_diag;
  c->ffn_launch_no = (c->ffn_launch_no + 1) & 0x7fffff;
  if (c->ffn_launch_no == 0) c->ffn_launch_no = 1;
  p.launch_tag = c->ffn_launch_no << 8;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  if (c->timing && (c->timing_seen++ % c->timing_period) == 0 && c->ev_used + 2 <= c->ev_pool.size()) {
    e0 = c->ev_pool[c->ev_used];
    e1 = c->ev_pool[c->ev_used + 1];
    c->ev_used += 2;
    ACM_CUDA(cudaEventRecord(e0, s));
  }
  // dependent launch only straight after the select/route kernel (no event, memset or copy between)
  p.pdl = pdl_ok && c->pdl && !e0;
  // the anchors' pre-segment pays only when this launch overlaps the selection; a launch ordered after it (one
  // bracketed by events) has the whole set at hand and takes the balanced plan
  if (anchors_first && p.pdl && early_epoch != 0) p.anc_flag = c->ws.anc_words;
  // Straight after the routing kernel: the few SMs it ran on (or still holds, in an early start) take
  // microseconds longer to accept a CTA of this kernel -- an SM changes hands slowly when the shared-memory
  // split changes -- and one late CTA delays every CTA that exchanges fragments with it.  Leave them out.
  const int routing_ctas = (n_blocks > 0 ? n_blocks : 1) * select_ctas_per_block(widest_block > 0 ? widest_block : T);
  if (pdl_ok && c->sm_count > 2 * routing_ctas) p.grid = c->sm_count - routing_ctas;
  c->last_ffn_grid = p.grid;
  if (L.mx) {
    p.mx_gate_up = L.has_pool ? L.pool_gate_up : L.mx_gate_up;      // a pool: slot s of the pool tensors
    p.mx_down = L.has_pool ? L.pool_down : L.mx_down;
    ACM_CUDA(launch_ffn_mxfp4(p, maps, x_map, c->h_map[li], c->h_store_map[li], s));
  } else {
    ACM_CUDA(launch_ffn_bf16(p, maps, x_map, c->h_map[li], c->h_store_map[li], s));
  }
  c->launches += 1;
  if (e1) ACM_CUDA(cudaEventRecord(e1, s));
  return ACM_OK;
}

// The sequence number of a fused call: its low 16 bits tag the words its kernels publish for one another (0 is
// never a valid tag).  The tags come round every 65535 calls, and a word that no call has rewritten since (a
// later block's words after single-block calls) would then look current: when they come round, the words are
// cleared, in stream order, before the call's first kernel.
acm_status next_epoch(acm_ctx* c, cudaStream_t s, int32_t* epoch_out) {
  int32_t e = ++c->epoch;
  if (e <= 0) e = c->epoch = 0x10000;
  if ((e & 0xffff) == 0) {
    ACM_CUDA(cudaMemsetAsync(c->ws.sel_words, 0, 32 * kMaxEarlyBlocks, s));
    ACM_CUDA(cudaMemsetAsync(c->ws.anc_words, 0, 32 * kMaxEarlyBlocks, s));
    e = ++c->epoch;
  }
  *epoch_out = e;
  return ACM_OK;
}

// what both offload variants need: the pinned report buffer, the copy stream and its events
acm_status ensure_offload_common(acm_ctx* c) {
  if (c->host_stage_list) return ACM_OK;
  const size_t n = (kMaxExperts + 1 + kMaskWords) * sizeof(int32_t);
  ACM_CUDA(cudaHostAlloc(reinterpret_cast<void**>(&c->host_stage_list), n, cudaHostAllocMapped));
  std::memset(c->host_stage_list, 0, n);
  ACM_CUDA(cudaHostGetDevicePointer(reinterpret_cast<void**>(&c->host_stage_list_dev), c->host_stage_list, 0));
  ACM_CUDA(cudaHostAlloc(reinterpret_cast<void**>(&c->resident_words_pinned), 64 * kMaskWords * sizeof(uint32_t),
                         cudaHostAllocDefault));
  ACM_CUDA(cudaHostAlloc(reinterpret_cast<void**>(&c->slot_table_pinned),
                         static_cast<size_t>(kSlotTableRing) * kMaxExperts * sizeof(int32_t), cudaHostAllocDefault));
  ACM_CUDA(cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
  ACM_CUDA(cudaEventCreateWithFlags(&c->ev_lists, cudaEventDisableTiming));
  ACM_CUDA(cudaEventCreateWithFlags(&c->ev_copied, cudaEventDisableTiming));
  ACM_CUDA(cudaEventCreateWithFlags(&c->ev_stage_free, cudaEventDisableTiming));
  return ACM_OK;
}

acm_status ensure_staging(acm_ctx* c) {
  if (c->stage_gate_up) return ACM_OK;
  acm_status st0 = ensure_offload_common(c);
  if (st0 != ACM_OK) return st0;
  const acm_model_desc& d = c->desc;
  const size_t gu = static_cast<size_t>(d.n_experts) * 2 * d.inter * d.hidden * 2;
  const size_t dn = static_cast<size_t>(d.n_experts) * d.hidden * d.inter * 2;
  if (cudaMalloc(&c->stage_gate_up, gu) != cudaSuccess) return ACM_ERR_NOMEM;
  if (cudaMalloc(&c->stage_down, dn) != cudaSuccess) return ACM_ERR_NOMEM;
  acm_status st = encode_gate_up(c, &c->stage_map_gu, c->stage_gate_up, d.n_experts);
  if (st != ACM_OK) return st;
  st = encode_down(c, &c->stage_map_dn, c->stage_down, d.n_experts);
  if (st != ACM_OK) return st;
  return ACM_OK;
}

}  // namespace

extern "C" {

void acm_default_select_params(acm_select_params* p) {
  if (!p) return;
  p->demand = ACM_DEMAND_TOPK_MASS;
  p->use_anchors = 1;
  p->fixed_budget = 0;
  p->ceil_guard = 0.0009765625f;
  p->residency = 0;
  p->max_remove = kMaxExperts;
}

const char* acm_status_string(acm_status s) {
  switch (s) {
    case ACM_OK: return "ok";
    case ACM_ERR_INVALID: return "invalid argument";
    case ACM_ERR_UNSUPPORTED: return "outside the supported limits";
    case ACM_ERR_CUDA: return "CUDA call failed";
    case ACM_ERR_TIMEOUT: return "bounded device-side wait ran out";
    case ACM_ERR_NOMEM: return "out of memory";
    case ACM_ERR_NONFINITE: return "non-finite router logit";
  }
  return "unknown status";
}

acm_status acm_create(const acm_model_desc* desc, acm_ctx** out) {
  if (!desc || !out) return ACM_ERR_INVALID;
  *out = nullptr;
  acm_status st = check_desc(*desc);
  if (st != ACM_OK) return st;
  acm_ctx* c = new (std::nothrow) acm_ctx();
  if (!c) return ACM_ERR_NOMEM;
  c->desc = *desc;
  c->layers.resize(desc->n_layers);
  auto fail = [&](acm_status s) {
    acm_destroy(c);
    return s;
  };
  if (cudaGetDevice(&c->device) != cudaSuccess) return fail(ACM_ERR_CUDA);
  if (cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device) != cudaSuccess)
    return fail(ACM_ERR_CUDA);
  if (desc->dtype == ACM_BF16) {
    int major = 0;
    cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, c->device);
    if (major != 10) return fail(ACM_ERR_UNSUPPORTED);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess)
      return fail(ACM_ERR_CUDA);
    c->encode = reinterpret_cast<EncodeTiledFn>(fn);
    if (ffn_configure() != cudaSuccess) return fail(ACM_ERR_CUDA);
  }
  if (select_configure() != cudaSuccess) return fail(ACM_ERR_CUDA);

  const int Tm = kWideNodes, E = desc->n_experts, k = desc->top_k, I = desc->inter;
  size_t off = 0;
  auto carve = [&](size_t bytes) {
    const size_t at = off;
    off = align_up(off + bytes, 1024);
    return at;
  };
  const size_t o_logits = carve(sizeof(float) * Tm * E);
  const size_t o_idx = carve(sizeof(int32_t) * Tm * k);
  const size_t o_w = carve(sizeof(float) * Tm * k), o_mask = carve(16 * Tm), o_unpr = carve(16 * Tm), o_cnt = carve(4 * Tm);
  const size_t o_dem = carve(sizeof(float) * kMaxExperts * Tm), o_stats = carve(sizeof(acm_block_stats) * Tm);
  // the FFN kernel's routing inputs, contiguous so that one pass clears them: weight table, finished-tile
  // counters, activated mask
  const size_t ffn_in_bytes = sizeof(float) * kMaxExperts * kWtabStride + sizeof(int32_t) * 2 * kMaxSlots + 16;
  const size_t o_ffn_in = carve(align_up(ffn_in_bytes, 16));
  const size_t hbuf_bf16 = static_cast<size_t>(2) * kMaxSlots * kWideNodes * I * 2;
  const size_t hbuf_f32 = static_cast<size_t>(Tm) * (k + desc->n_shared) * I * 4;
  const size_t o_h = carve(hbuf_bf16 > hbuf_f32 ? hbuf_bf16 : hbuf_f32);
  const size_t o_frag = carve(sizeof(float) * 2 * 2 * static_cast<size_t>(c->sm_count) * 128 * kMaxNodes);
  const size_t o_flag = carve(sizeof(int32_t) * 2 * 2 * c->sm_count);
  const size_t o_status = carve(16);
  const size_t o_tile = carve(sizeof(int32_t) * kMaxNodes);
  const size_t o_ticket = carve(16);
  const size_t o_selw = carve(32 * kMaxEarlyBlocks);
  const size_t o_ancw = carve(32 * kMaxEarlyBlocks);
  const size_t o_rootw = carve(sizeof(unsigned long long) * kMaxExperts * kMaxEarlyBlocks);
  const size_t o_res = carve(sizeof(uint32_t) * 4 * desc->n_layers);
  const size_t o_diag = carve(sizeof(int32_t) * c->sm_count);
  if (cudaMalloc(&c->ws_base, off) != cudaSuccess) return fail(ACM_ERR_NOMEM);
  if (cudaMemset(c->ws_base, 0, off) != cudaSuccess) return fail(ACM_ERR_CUDA);
  char* b = static_cast<char*>(c->ws_base);
  c->ws.logits = reinterpret_cast<float*>(b + o_logits);
  c->ws.idx = reinterpret_cast<int32_t*>(b + o_idx);
  c->ws.w = reinterpret_cast<float*>(b + o_w);
  c->ws.mask = reinterpret_cast<uint32_t*>(b + o_mask);
  c->ws.unpruned = reinterpret_cast<uint32_t*>(b + o_unpr);
  c->ws.count = reinterpret_cast<int32_t*>(b + o_cnt);
  c->ws.demand = reinterpret_cast<float*>(b + o_dem);
  c->ws.stats = reinterpret_cast<acm_block_stats*>(b + o_stats);
  c->ws.wtab = reinterpret_cast<float*>(b + o_ffn_in);
  c->ws.ready = reinterpret_cast<int32_t*>(b + o_ffn_in + sizeof(float) * kMaxExperts * kWtabStride);
  c->ws.act_mask = reinterpret_cast<uint32_t*>(b + o_ffn_in + sizeof(float) * kMaxExperts * kWtabStride +
                                               sizeof(int32_t) * 2 * kMaxSlots);
  c->ffn_in_floats = align_up(ffn_in_bytes, 16) / sizeof(float);
  c->ws.hbuf = b + o_h;
  c->ws.frag = reinterpret_cast<float*>(b + o_frag);
  c->frag_bytes = sizeof(float) * 2 * 2 * static_cast<size_t>(c->sm_count) * 128 * kMaxNodes;
  c->flag_bytes = sizeof(int32_t) * 2 * 2 * c->sm_count;
  c->ws.frag_flag = reinterpret_cast<int32_t*>(b + o_flag);
  c->ws.status = reinterpret_cast<int32_t*>(b + o_status);
  c->ws.tile_done = reinterpret_cast<int32_t*>(b + o_tile);
  c->ws.ticket = reinterpret_cast<int32_t*>(b + o_ticket);
  c->ws.sel_words = reinterpret_cast<uint32_t*>(b + o_selw);
  c->ws.anc_words = reinterpret_cast<uint32_t*>(b + o_ancw);
  c->ws.root_words = reinterpret_cast<unsigned long long*>(b + o_rootw);
  c->resident_dev = reinterpret_cast<uint32_t*>(b + o_res);
  c->wait_diag = reinterpret_cast<int32_t*>(b + o_diag);
  *out = c;
  return ACM_OK;
}

acm_status acm_destroy(acm_ctx* c) {
  if (!c) return ACM_ERR_INVALID;
  cudaDeviceSynchronize();
  for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
  for (cudaEvent_t e : c->off_ev) cudaEventDestroy(e);
  if (c->ev_lists) cudaEventDestroy(c->ev_lists);
  if (c->ev_copied) cudaEventDestroy(c->ev_copied);
  if (c->ev_stage_free) cudaEventDestroy(c->ev_stage_free);
  if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
  if (c->h2d_stream) cudaStreamDestroy(c->h2d_stream);
  if (c->d2h_stream) cudaStreamDestroy(c->d2h_stream);
  for (int b = 0; b < 2; ++b) {
    if (c->hx_dev[b]) cudaFree(c->hx_dev[b]);
    if (c->halpha_dev[b]) cudaFree(c->halpha_dev[b]);
    if (c->hout_dev[b]) cudaFree(c->hout_dev[b]);
    if (c->hstats_dev[b]) cudaFree(c->hstats_dev[b]);
    if (c->ev_in[b]) cudaEventDestroy(c->ev_in[b]);
    if (c->ev_done[b]) cudaEventDestroy(c->ev_done[b]);
    if (c->ev_out[b]) cudaEventDestroy(c->ev_out[b]);
  }
  if (c->host_stage_list) cudaFreeHost(c->host_stage_list);
  if (c->resident_words_pinned) cudaFreeHost(c->resident_words_pinned);
  if (c->slot_table_pinned) cudaFreeHost(c->slot_table_pinned);
  for (Layer& L : c->layers)
    for (int b = 0; b < 2; ++b)
      if (L.slot_of_dev[b]) cudaFree(L.slot_of_dev[b]);
  if (c->stage_gate_up) cudaFree(c->stage_gate_up);
  if (c->stage_down) cudaFree(c->stage_down);
  if (c->ws_base) cudaFree(c->ws_base);
  if (c->trace) cudaFree(c->trace);
  delete c;
  return ACM_OK;
}

acm_status acm_set_layer_weights(acm_ctx* c, int layer, const void* w_router, const float* router_bias,
                                 const void* w_gate_up, const void* w_down, const void* shared_gate_up,
                                 const void* shared_down) {
  if (!c || layer < 0 || layer >= c->desc.n_layers || !w_router) return ACM_ERR_INVALID;
  const acm_model_desc& d = c->desc;
  if ((w_gate_up == nullptr) != (w_down == nullptr)) return ACM_ERR_INVALID;
  if (d.n_shared > 0 && w_gate_up && (!shared_gate_up || !shared_down)) return ACM_ERR_INVALID;
  if (reinterpret_cast<uintptr_t>(w_router) % 16 != 0) return ACM_ERR_INVALID;
  Layer L;
  L.w_router = w_router; L.bias = router_bias; L.gate_up = w_gate_up; L.down = w_down;
  L.shared_gate_up = d.n_shared ? shared_gate_up : nullptr;
  L.shared_down = d.n_shared ? shared_down : nullptr;
  if (d.dtype == ACM_BF16 && w_gate_up) {
    acm_status st = encode_gate_up(c, &L.maps.gate_up, w_gate_up, d.n_experts);
    if (st != ACM_OK) return st;
    st = encode_down(c, &L.maps.down, w_down, d.n_experts);
    if (st != ACM_OK) return st;
    L.maps.shared_gate_up = L.maps.gate_up;
    L.maps.shared_down = L.maps.down;
    if (d.n_shared) {
      st = encode_gate_up(c, &L.maps.shared_gate_up, shared_gate_up, d.n_shared);
      if (st != ACM_OK) return st;
      st = encode_down(c, &L.maps.shared_down, shared_down, d.n_shared);
      if (st != ACM_OK) return st;
    }
    L.maps.staged_gate_up = L.maps.gate_up;
    L.maps.staged_down = L.maps.down;
  }
  L.set = true;
  c->layers[layer] = L;
  return ACM_OK;
}

acm_status acm_set_layer_weights_mxfp4(acm_ctx* c, int layer, const void* w_router, const float* router_bias,
                                       const void* gate_up_tiles, const void* down_tiles) {
  if (!c || layer < 0 || layer >= c->desc.n_layers || !w_router) return ACM_ERR_INVALID;
  if ((gate_up_tiles == nullptr) != (down_tiles == nullptr)) return ACM_ERR_INVALID;
  const acm_model_desc& d = c->desc;
  if (d.dtype != ACM_BF16 || d.n_shared != 0 || d.inter % 128 != 0 || d.hidden % 128 != 0) return ACM_ERR_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(w_router) % 16 != 0 || reinterpret_cast<uintptr_t>(gate_up_tiles) % 16 != 0 ||
      reinterpret_cast<uintptr_t>(down_tiles) % 16 != 0)
    return ACM_ERR_INVALID;
  if (!c->mx_configured) {
    if (ffn_mx_configure() != cudaSuccess) return ACM_ERR_CUDA;
    c->mx_configured = true;
  }
  if (gate_up_tiles) {
    // every scale byte of both tensors, once, at registration (a small kernel and one synchronous read-back)
    const size_t rec_gu = static_cast<size_t>(d.n_experts) * (d.inter / 64) * (d.hidden / 128);
    const size_t rec_dn = static_cast<size_t>(d.n_experts) * (d.hidden / 128) * (d.inter / 128);
    int* max_dev = reinterpret_cast<int*>(c->ws.ticket) + 2;      // (a spare word of the workspace)
    ACM_CUDA(cudaMemset(max_dev, 0, sizeof(int)));
    k_mx_max_scale<<<256, 256>>>(static_cast<const unsigned char*>(gate_up_tiles), rec_gu, max_dev);
    k_mx_max_scale<<<256, 256>>>(static_cast<const unsigned char*>(down_tiles), rec_dn, max_dev);
    int max_scale = 0;
    ACM_CUDA(cudaMemcpy(&max_scale, max_dev, sizeof(int), cudaMemcpyDeviceToHost));
    ACM_CUDA(cudaMemset(max_dev, 0, sizeof(int)));
    if (max_scale > kMxMaxScaleByte) return ACM_ERR_UNSUPPORTED;
  }
  Layer L;
  L.w_router = w_router; L.bias = router_bias;
  L.mx = true;
  L.mx_gate_up = gate_up_tiles; L.mx_down = down_tiles;
  std::memset(&L.maps, 0, sizeof L.maps);      // the MXFP4 kernel fetches its weights with plain bulk copies
  L.set = true;
  c->layers[layer] = L;
  return ACM_OK;
}

acm_status acm_node_weights(const int32_t* depth, int T, const float* p_table, int n_depths, float beta,
                            int width_norm, float* alpha_out) {
  if (!depth || !p_table || !alpha_out || T < 1 || n_depths < 1) return ACM_ERR_INVALID;
  std::vector<int> width(n_depths, 0);
  for (int t = 0; t < T; ++t) {
    if (depth[t] < 0 || depth[t] >= n_depths) return ACM_ERR_INVALID;
    ++width[depth[t]];
  }
  for (int t = 0; t < T; ++t) {
    double a = std::pow(static_cast<double>(p_table[depth[t]]), static_cast<double>(beta));
    if (width_norm) a /= std::sqrt(static_cast<double>(width[depth[t]]));
    alpha_out[t] = static_cast<float>(a);
  }
  return ACM_OK;
}

acm_status acm_router(acm_ctx* c, int layer, const void* x, int T, float* logits, float* probs,
                      int32_t* nat_idx, acm_stream stream) {
  acm_status st = check_block_args(c, layer, T, true);
  if (st != ACM_OK) return st;
  if (!x || !logits || reinterpret_cast<uintptr_t>(x) % 16 != 0) return ACM_ERR_INVALID;
  const acm_model_desc& d = c->desc;
  const Layer& L = c->layers[layer];
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // softmax and natural top-k are finished inside the same launch (last CTA of each node tile)
  ACM_CUDA(launch_router_logits(d.dtype, x, L.w_router, L.bias, logits, T, d.hidden, d.n_experts, nullptr, 0,
                                nullptr, 0, c->ws.status, probs, nat_idx, nullptr, d.top_k, c->ws.tile_done, false, s,
                                c->trace ? reinterpret_cast<long long*>(c->trace) + 32 * c->sm_count : nullptr));
  c->launches += 1;
  return ACM_OK;
}

acm_status acm_select_eligible(acm_ctx* c, const float* probs, const int32_t* nat_idx, int T, const float* alpha,
                               const int32_t* anchor_nodes, int n_anchor_nodes, const acm_select_params* params,
                               const uint32_t* resident_mask, uint32_t* eligible_mask, int32_t* eligible_count,
                               float* demand, uint32_t* unpruned_mask, acm_block_stats* stats, acm_stream stream) {
  if (!c || T < 1 || T > c->desc.max_nodes) return ACM_ERR_INVALID;
  if (!probs || !nat_idx || !alpha || !eligible_mask || !eligible_count) return ACM_ERR_INVALID;
  acm_status st = check_params(params);
  if (st != ACM_OK) return st;
  if (params->residency != 0 && !resident_mask) return ACM_ERR_INVALID;
  if (anchor_nodes && (n_anchor_nodes < 1 || n_anchor_nodes > kMaxNodes)) return ACM_ERR_INVALID;
  SelectArgs a;
  a.probs = probs; a.nat_idx = nat_idx; a.alpha = alpha; a.anchor_nodes = anchor_nodes;
  a.n_anchor_nodes = n_anchor_nodes; a.resident = params->residency ? resident_mask : nullptr; a.prm = *params;
  a.mask_out = eligible_mask; a.unpruned_out = unpruned_mask; a.count_out = eligible_count;
  a.demand_out = demand; a.stats_out = stats;
  ACM_CUDA(launch_select(a, T, c->desc.n_experts, c->desc.top_k, static_cast<cudaStream_t>(stream)));
  c->launches += 1;
  return ACM_OK;
}

acm_status acm_route_restricted(acm_ctx* c, const float* logits, const uint32_t* eligible_mask, int T,
                                int32_t* idx, float* w, acm_stream stream) {
  if (!c || T < 1 || T > c->desc.max_nodes) return ACM_ERR_INVALID;
  if (!logits || !eligible_mask || !idx || !w) return ACM_ERR_INVALID;
  RouteArgs a = {};
  a.logits = logits; a.mask = eligible_mask; a.idx_out = idx; a.w_out = w;
  a.weighting = c->desc.weighting; a.routed_scale = c->desc.routed_scale;
  ACM_CUDA(launch_route(a, T, c->desc.n_experts, c->desc.top_k, static_cast<cudaStream_t>(stream)));
  c->launches += 1;
  return ACM_OK;
}

acm_status acm_expert_ffn(acm_ctx* c, int layer, const void* x, int T, const int32_t* idx, const float* w,
                          float* out, acm_stream stream) {
  acm_status st = check_block_args(c, layer, T, true);
  if (st != ACM_OK) return st;
  const Layer& L = c->layers[layer];
  if (!x || !idx || !w || !out || (!L.gate_up && !L.mx_gate_up)) return ACM_ERR_INVALID;
  if (reinterpret_cast<uintptr_t>(x) % 16 != 0 || reinterpret_cast<uintptr_t>(out) % 16 != 0) return ACM_ERR_INVALID;
  if (L.has_resident) return ACM_ERR_UNSUPPORTED;   // staging is driven by acm_moe_verify
  const acm_model_desc& d = c->desc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (d.dtype == ACM_F32) {
    ACM_CUDA(launch_ffn_f32(static_cast<const float*>(x), static_cast<const float*>(L.gate_up),
                            static_cast<const float*>(L.down), static_cast<const float*>(L.shared_gate_up),
                            static_cast<const float*>(L.shared_down), d.n_shared, idx, w,
                            static_cast<float*>(c->ws.hbuf), out, T, d.hidden, d.inter, d.n_experts, d.top_k, s));
    c->launches += 2;
    return ACM_OK;
  }
  ACM_CUDA(cudaMemsetAsync(out, 0, sizeof(float) * static_cast<size_t>(T) * d.hidden, s));
  ACM_CUDA(launch_routes_to_table(idx, w, c->ws.act_mask, c->ws.wtab, c->ws.ready, T, d.n_experts, d.top_k, s));
  c->launches += 1;
  return run_ffn_list(c, L, x, T, 0, out, s);
}

acm_status acm_moe_verify(acm_ctx* c, int layer, const void* x, int T, const float* alpha,
                          const acm_select_params* params, const uint32_t* eligible_mask_override, float* out,
                          int32_t* idx_out, float* w_out, uint32_t* mask_out, acm_block_stats* stats,
                          acm_stream stream) {
  acm_status st = check_block_args(c, layer, T, true);
  if (st != ACM_OK) return st;
  const Layer& L = c->layers[layer];
  if (!x || !out || (!L.gate_up && !L.has_pool && !L.mx_gate_up)) return ACM_ERR_INVALID;
  if (reinterpret_cast<uintptr_t>(x) % 16 != 0 || reinterpret_cast<uintptr_t>(out) % 16 != 0) return ACM_ERR_INVALID;
  acm_select_params prm;
  if (eligible_mask_override) {
    acm_default_select_params(&prm);
  } else {
    if (!alpha) return ACM_ERR_INVALID;
    st = check_params(params);
    if (st != ACM_OK) return st;
    prm = *params;
    if (prm.residency != 0 && !L.has_resident) return ACM_ERR_INVALID;
  }
  const acm_model_desc& d = c->desc;
  const int E = d.n_experts, k = d.top_k;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const bool f32 = d.dtype == ACM_F32;
  uint32_t* res_dev = L.has_resident ? c->resident_dev + 4 * layer : nullptr;

  // Early start of the FFN kernel on the eligible set: when a selection runs (the eligible experts are
  // then nearly always all activated; with an override mask they need not be) and every expert is resident.
  const bool early = !f32 && !L.has_resident && !eligible_mask_override && c->early_start;
  int32_t early_epoch = 0;
  if (early) {
    st = next_epoch(c, s, &early_epoch);
    if (st != ACM_OK) return st;
  }
  // ... and earlier still on the anchors (Eq. 5 with the default anchor, the root): the router kernel's first CTAs
  // work out the root's logits ahead of the rest and publish its natural top-k, the FFN kernel streams their gate/up
  // tiles while the softmax and the selection run.  They are in every eligible set the selection can return without a residency.
  const bool anchors_first = early && c->anchor_start && prm.use_anchors != 0;
  // offload timing: events around the resident part, the copies and the loaded part of this call
  cudaEvent_t* oev = nullptr;
  if (c->off_timing && L.has_resident && !L.has_pool && 5 * (c->off_calls + 1) <= c->off_ev.size()) {
    oev = c->off_ev.data() + 5 * c->off_calls;
    ACM_CUDA(cudaEventRecord(oev[0], s));
  }
  // stage 1a: the logits (the kernel also clears the output the FFN accumulates into and the FFN kernel's
  // routing inputs); on an early call its first CTAs also work out the root's logits ahead of the rest and publish
  // the anchors (on every early call, used or not: the words never carry an old tag)
  RootArgs root = {};
  root.rows = 1;
  root.row[0] = 0;
  root.words = c->ws.root_words;
  root.tag = static_cast<uint32_t>(early_epoch);
  root.anc_words = c->ws.anc_words;
  root.anc_tag = static_cast<uint32_t>(early_epoch) & 0xffffu;
  root.wait_limit_ns = c->wait_limit_ns;
  ACM_CUDA(launch_router_logits(d.dtype, x, L.w_router, L.bias, c->ws.logits, T, d.hidden, E, f32 ? nullptr : out,
                                f32 ? 0 : static_cast<size_t>(T) * d.hidden, c->ws.wtab, c->ffn_in_floats,
                                c->ws.status, nullptr, nullptr, nullptr, k, nullptr, c->pdl, s,
                                c->trace ? reinterpret_cast<long long*>(c->trace) + 32 * c->sm_count : nullptr,
                                early ? &root : nullptr));
  // stages 1b-3: one cluster of CTAs, which also fills the FFN kernel's routing inputs
  SelectArgs sa;
  sa.probs = nullptr; sa.nat_idx = nullptr; sa.alpha = alpha; sa.anchor_nodes = nullptr;   // (the fused kernel keeps both on chip)
  sa.n_anchor_nodes = 0; sa.resident = prm.residency ? res_dev : nullptr; sa.prm = prm;
  sa.mask_out = c->ws.mask; sa.unpruned_out = c->ws.unpruned; sa.count_out = c->ws.count;
  bool stats_direct = false;
  acm_block_stats* stats_dev = stats_target(c, stats, &stats_direct);
  sa.demand_out = c->ws.demand; sa.stats_out = stats_dev;
  RouteArgs ra = {};
  ra.logits = c->ws.logits; ra.mask = c->ws.mask; ra.idx_out = c->ws.idx; ra.w_out = c->ws.w;
  ra.weighting = d.weighting; ra.routed_scale = d.routed_scale;
  ra.act_mask = c->ws.act_mask; ra.wtab = c->ws.wtab; ra.resident = res_dev;
  ra.host_stage_list = L.has_resident ? c->host_stage_list_dev : nullptr;
  if (early) {
    ra.sel_flag = c->ws.sel_words;
    ra.sel_epoch = early_epoch;
  }
  ra.dbg = c->trace ? reinterpret_cast<long long*>(c->trace) + 32 * c->sm_count : nullptr;
  BatchDesc one = {};
  one.n_blocks = 1;
  one.off[0] = 0;
  one.off[1] = T;
  ACM_CUDA(launch_softmax_select_route(sa, ra, one, eligible_mask_override, E, k, c->pdl, s));
  c->launches += 2;

  if (f32) {
    ACM_CUDA(launch_ffn_f32(static_cast<const float*>(x), static_cast<const float*>(L.gate_up),
                            static_cast<const float*>(L.down), static_cast<const float*>(L.shared_gate_up),
                            static_cast<const float*>(L.shared_down), d.n_shared, c->ws.idx, c->ws.w,
                            static_cast<float*>(c->ws.hbuf), out, T, d.hidden, d.inter, E, k, s));
    c->launches += 2;
  } else if (!L.has_resident) {
    st = run_ffn_list(c, L, x, T, 0, out, s, nullptr, stats_dev, true, early_epoch, nullptr, 0, anchors_first);
    if (st != ACM_OK) return st;
  } else {
    // resident + shared experts run at once; the others are copied in from pinned host memory first
    ACM_CUDA(cudaEventRecord(c->ev_lists, s));
    st = run_ffn_list(c, L, x, T, 0, out, s, res_dev, stats_dev);
    if (st != ACM_OK) return st;
    if (oev) ACM_CUDA(cudaEventRecord(oev[1], s));
    ACM_CUDA(cudaEventSynchronize(c->ev_lists));
    const int n_stage = c->host_stage_list[0];
    if (n_stage < 0 || n_stage > E) return ACM_ERR_CUDA;
    size_t gu, dn;
    expert_tensor_bytes(d, L.mx, &gu, &dn);
    if (L.has_pool) {
      // LRU expert pool: the experts activated by this block that were resident are touched; the others
      // are loaded, synchronously with respect to their FFN, into the least recently used slots that this
      // block does not use, and stay resident for later blocks.
      Layer& P = c->layers[layer];
      uint32_t act[kMaskWords];
      for (int w = 0; w < kMaskWords; ++w) act[w] = static_cast<uint32_t>(c->host_stage_list[1 + kMaxExperts + w]);
      // The activated experts that are not in the pool are loaded in WAVES (Section 3.4: a routed union
      // larger than the pool is processed in several waves that each fit).  The first wave needs no wait -- it
      // only takes slots this block does not use, while the FFN over the resident experts is running; every
      // later wave first waits for the FFN launched before it.  The expert FFN is a sum over experts, so a
      // wave is a subset of experts over all nodes: each expert is loaded once.
      std::vector<PoolLoad> loads;
      int n_hits = 0;
      if (!plan_pool_block(E, P.n_slots, P.slot_expert, P.expert_slot, P.last_use, P.tick, act, loads, n_hits))
        return ACM_ERR_CUDA;
      if (static_cast<int>(loads.size()) != n_stage) return ACM_ERR_CUDA;     // the kernel's report and the host's view agree
      P.pool_hits += n_hits;
      size_t at = 0;
      for (int wave = 0; at < loads.size(); ++wave) {
        if (wave > 0) {
          ACM_CUDA(cudaEventRecord(c->ev_stage_free, s));
          ACM_CUDA(cudaStreamWaitEvent(c->copy_stream, c->ev_stage_free, 0));
        }
        uint32_t only[kMaskWords] = {0, 0, 0, 0};
        // the expert -> slot table this wave's launch reads: where its own experts are (the planner has already
        // applied later waves too, which may have moved other experts on; after the last wave it is exact)
        std::vector<int32_t> table(P.expert_slot);
        for (; at < loads.size() && loads[at].wave == wave; ++at) {
          const int e = loads[at].expert, sl = loads[at].slot;
          only[e >> 5] |= 1u << (e & 31);
          table[e] = sl;
          ACM_CUDA(cudaMemcpyAsync(static_cast<char*>(P.pool_gate_up) + sl * gu,
                                   static_cast<const char*>(P.host_gate_up) + e * gu, gu, cudaMemcpyHostToDevice,
                                   c->copy_stream));
          ACM_CUDA(cudaMemcpyAsync(static_cast<char*>(P.pool_down) + sl * dn,
                                   static_cast<const char*>(P.host_down) + e * dn, dn, cudaMemcpyHostToDevice,
                                   c->copy_stream));
          P.pool_misses += 1;
          P.pool_h2d += gu + dn;
          c->h2d_bytes += gu + dn;
        }
        // the new expert -> slot table goes into the other device copy (a running kernel may read this one)
        const int nxt = P.slot_of_cur ^ 1;
        if (c->slot_table_next % kSlotTableRing == kSlotTableRing - 1)
          ACM_CUDA(cudaStreamSynchronize(c->copy_stream));       // the ring of pinned tables is about to wrap
        int32_t* staged_table = c->slot_table_pinned + static_cast<size_t>(kMaxExperts) * (c->slot_table_next % kSlotTableRing);
        std::memcpy(staged_table, table.data(), sizeof(int32_t) * E);
        ACM_CUDA(cudaMemcpyAsync(P.slot_of_dev[nxt], staged_table, sizeof(int32_t) * E, cudaMemcpyHostToDevice,
                                 c->copy_stream));
        c->slot_table_next += 1;
        ACM_CUDA(cudaEventRecord(c->ev_copied, c->copy_stream));
        ACM_CUDA(cudaStreamWaitEvent(s, c->ev_copied, 0));
        P.slot_of_cur = nxt;
        if (c->pool_waves_list1_used)      // the second work list's counters are cleared once per block by the router kernel
          ACM_CUDA(cudaMemsetAsync(c->ws.ready + kMaxSlots, 0, sizeof(int32_t) * kMaxSlots, s));
        c->pool_waves_list1_used = true;
        st = run_ffn_list(c, P, x, T, 1, out, s, res_dev, nullptr, false, 0, only);
        if (st != ACM_OK) return st;
        P.pool_waves += 1;
      }
      c->pool_waves_list1_used = false;
      if (n_stage > 0) {
        // the resident set of the next block (this block's kernels still read the old one: stream order)
        uint32_t words[kMaskWords] = {0, 0, 0, 0};
        for (int e = 0; e < E; ++e)
          if (P.expert_slot[e] >= 0) words[e >> 5] |= 1u << (e & 31);
        std::memcpy(c->resident_words_pinned + kMaskWords * (c->resident_words_next % 64), words, sizeof words);
        ACM_CUDA(cudaMemcpyAsync(c->resident_dev + 4 * layer,
                                 c->resident_words_pinned + kMaskWords * (c->resident_words_next % 64), sizeof words,
                                 cudaMemcpyHostToDevice, s));
        c->resident_words_next += 1;
      }
    } else if (n_stage > 0) {
      if (c->stage_in_use) ACM_CUDA(cudaStreamWaitEvent(c->copy_stream, c->ev_stage_free, 0));
      if (oev) ACM_CUDA(cudaEventRecord(oev[2], c->copy_stream));
      for (int i = 0; i < n_stage; ++i) {
        const int e = c->host_stage_list[1 + i];
        if (e < 0 || e >= E) return ACM_ERR_CUDA;
        ACM_CUDA(cudaMemcpyAsync(static_cast<char*>(c->stage_gate_up) + i * gu,
                                 static_cast<const char*>(L.host_gate_up) + e * gu, gu, cudaMemcpyHostToDevice,
                                 c->copy_stream));
        ACM_CUDA(cudaMemcpyAsync(static_cast<char*>(c->stage_down) + i * dn,
                                 static_cast<const char*>(L.host_down) + e * dn, dn, cudaMemcpyHostToDevice,
                                 c->copy_stream));
        c->h2d_bytes += gu + dn;
      }
      if (oev) ACM_CUDA(cudaEventRecord(oev[3], c->copy_stream));
      ACM_CUDA(cudaEventRecord(c->ev_copied, c->copy_stream));
      ACM_CUDA(cudaStreamWaitEvent(s, c->ev_copied, 0));
      st = run_ffn_list(c, L, x, T, 1, out, s, res_dev, nullptr);
      if (st != ACM_OK) return st;
      ACM_CUDA(cudaEventRecord(c->ev_stage_free, s));
      c->stage_in_use = true;
    }
    if (oev) {
      ACM_CUDA(cudaEventRecord(oev[4], s));
      c->off_has_copies[c->off_calls] = (!L.has_pool && n_stage > 0) ? 1 : 0;
      c->off_calls += 1;
    }
  }

  const size_t tk = static_cast<size_t>(T) * k;
  if (idx_out) ACM_CUDA(cudaMemcpyAsync(idx_out, c->ws.idx, sizeof(int32_t) * tk, cudaMemcpyDeviceToDevice, s));
  if (w_out) ACM_CUDA(cudaMemcpyAsync(w_out, c->ws.w, sizeof(float) * tk, cudaMemcpyDeviceToDevice, s));
  if (mask_out)
    ACM_CUDA(cudaMemcpyAsync(mask_out, c->ws.mask, sizeof(uint32_t) * mask_words(E), cudaMemcpyDeviceToDevice, s));
  if (stats && !stats_direct) ACM_CUDA(cudaMemcpyAsync(stats, c->ws.stats, sizeof(acm_block_stats), cudaMemcpyDefault, s));
  return ACM_OK;
}

acm_status acm_moe_verify_batch(acm_ctx* c, int layer, const void* x, int n_blocks, const int32_t* block_offsets,
                                const float* alpha, const acm_select_params* params, float* out, int32_t* idx_out,
                                float* w_out, uint32_t* mask_out, uint32_t* activated_out, acm_block_stats* stats,
                                acm_stream stream) {
  if (!c || !block_offsets || n_blocks < 1 || n_blocks > kMaxNodes) return ACM_ERR_INVALID;
  BatchDesc bd;
  bd.n_blocks = n_blocks;
  if (block_offsets[0] != 0) return ACM_ERR_INVALID;
  for (int b = 0; b <= n_blocks; ++b) {
    if (b > 0 && block_offsets[b] <= block_offsets[b - 1]) return ACM_ERR_INVALID;     // every block has a node
    if (b > 0 && block_offsets[b] - block_offsets[b - 1] > c->desc.max_nodes) return ACM_ERR_INVALID;   // a block's own limit
    if (block_offsets[b] > kWideNodes) return ACM_ERR_INVALID;
    bd.off[b] = block_offsets[b];
  }
  const int T = block_offsets[n_blocks];
  acm_status st = check_block_args(c, layer, 1, true);
  if (st != ACM_OK) return st;
  const Layer& L = c->layers[layer];
  if (T > kMaxNodes && L.mx) return ACM_ERR_UNSUPPORTED;      // (the MXFP4 kernel's tensor memory holds 64-column accumulators only)
  if (!x || !out || !alpha || (!L.gate_up && !L.mx_gate_up)) return ACM_ERR_INVALID;
  if (reinterpret_cast<uintptr_t>(x) % 16 != 0 || reinterpret_cast<uintptr_t>(out) % 16 != 0) return ACM_ERR_INVALID;
  st = check_params(params);
  if (st != ACM_OK) return st;
  const acm_model_desc& d = c->desc;
  if (d.dtype != ACM_BF16 || L.has_resident || params->residency != 0) return ACM_ERR_UNSUPPORTED;
  const int E = d.n_experts, k = d.top_k;
  cudaStream_t s = static_cast<cudaStream_t>(stream);

  // stage 1 over all rows at once (it is per node); also clears `out` and the FFN kernel's routing inputs
  // early start of the FFN kernel on the union of the blocks' eligible sets (it polls eight words per block)
  const bool early = n_blocks <= kMaxEarlyBlocks && c->early_start;
  int32_t early_epoch = 0;
  if (early) {
    st = next_epoch(c, s, &early_epoch);
    if (st != ACM_OK) return st;
  }
  // ... and on the union of the blocks' anchors (each block's first row is its root) while the selections run
  const bool anchors_first = early && c->anchor_start && params->use_anchors != 0;
  // (on an early call the router kernel's first CTAs work out every block's root ahead of the rest and publish the anchors)
  RootArgs root = {};
  root.rows = early ? n_blocks : 0;
  for (int b = 0; b < root.rows; ++b) root.row[b] = bd.off[b];
  root.words = c->ws.root_words;
  root.tag = static_cast<uint32_t>(early_epoch);
  root.anc_words = c->ws.anc_words;
  root.anc_tag = static_cast<uint32_t>(early_epoch) & 0xffffu;
  root.wait_limit_ns = c->wait_limit_ns;
  ACM_CUDA(launch_router_logits(d.dtype, x, L.w_router, L.bias, c->ws.logits, T, d.hidden, E, out,
                                static_cast<size_t>(T) * d.hidden, c->ws.wtab, c->ffn_in_floats, c->ws.status,
                                nullptr, nullptr, nullptr, k, nullptr, c->pdl, s, nullptr, early ? &root : nullptr));
  // stages 1b-3: one cluster of CTAs per block
  SelectArgs sa;
  sa.probs = nullptr; sa.nat_idx = nullptr; sa.alpha = alpha; sa.anchor_nodes = nullptr;   // (the fused kernel keeps both on chip)
  sa.n_anchor_nodes = 0; sa.resident = nullptr; sa.prm = *params;
  sa.mask_out = c->ws.mask; sa.unpruned_out = c->ws.unpruned; sa.count_out = c->ws.count;
  bool stats_direct = false;
  acm_block_stats* stats_dev = stats_target(c, stats, &stats_direct);
  sa.demand_out = c->ws.demand; sa.stats_out = stats_dev;
  RouteArgs ra = {};
  ra.logits = c->ws.logits; ra.mask = c->ws.mask; ra.idx_out = c->ws.idx; ra.w_out = c->ws.w;
  ra.weighting = d.weighting; ra.routed_scale = d.routed_scale;
  ra.act_mask = c->ws.act_mask; ra.wtab = c->ws.wtab;
  if (early) {
    ra.sel_flag = c->ws.sel_words;
    ra.sel_epoch = early_epoch;
  }
  ACM_CUDA(launch_softmax_select_route(sa, ra, bd, nullptr, E, k, c->pdl, s));
  c->launches += 2;
  // stage 4 once over all rows: an expert activated by several blocks is streamed once
  int widest = 1;
  for (int b = 0; b < n_blocks; ++b) widest = std::max(widest, bd.off[b + 1] - bd.off[b]);
  st = run_ffn_list(c, L, x, T, 0, out, s, nullptr, nullptr, true, early_epoch, nullptr, n_blocks, anchors_first, widest);
  if (st != ACM_OK) return st;

  const size_t tk = static_cast<size_t>(T) * k;
  if (idx_out) ACM_CUDA(cudaMemcpyAsync(idx_out, c->ws.idx, sizeof(int32_t) * tk, cudaMemcpyDeviceToDevice, s));
  if (w_out) ACM_CUDA(cudaMemcpyAsync(w_out, c->ws.w, sizeof(float) * tk, cudaMemcpyDeviceToDevice, s));
  if (mask_out) {
    if (mask_words(E) == kMaskWords) {
      ACM_CUDA(cudaMemcpyAsync(mask_out, c->ws.mask, sizeof(uint32_t) * kMaskWords * n_blocks, cudaMemcpyDeviceToDevice, s));
    } else {
      ACM_CUDA(cudaMemcpy2DAsync(mask_out, sizeof(uint32_t) * mask_words(E), c->ws.mask, sizeof(uint32_t) * kMaskWords,
                                 sizeof(uint32_t) * mask_words(E), n_blocks, cudaMemcpyDeviceToDevice, s));
    }
  }
  if (activated_out)
    ACM_CUDA(cudaMemcpyAsync(activated_out, c->ws.act_mask, sizeof(uint32_t) * mask_words(E), cudaMemcpyDeviceToDevice, s));
  if (stats && !stats_direct)
    ACM_CUDA(cudaMemcpyAsync(stats, c->ws.stats, sizeof(acm_block_stats) * n_blocks, cudaMemcpyDefault, s));
  return ACM_OK;
}

namespace {
acm_status ensure_host_path(acm_ctx* c) {
  if (c->h2d_stream) return ACM_OK;
  const acm_model_desc& d = c->desc;
  const size_t elt = d.dtype == ACM_F32 ? 4 : 2;
  ACM_CUDA(cudaStreamCreateWithFlags(&c->h2d_stream, cudaStreamNonBlocking));
  ACM_CUDA(cudaStreamCreateWithFlags(&c->d2h_stream, cudaStreamNonBlocking));
  for (int b = 0; b < 2; ++b) {
    ACM_CUDA(cudaMalloc(&c->hx_dev[b], static_cast<size_t>(kMaxNodes) * d.hidden * elt));
    ACM_CUDA(cudaMalloc(reinterpret_cast<void**>(&c->halpha_dev[b]), kMaxNodes * sizeof(float)));
    ACM_CUDA(cudaMalloc(reinterpret_cast<void**>(&c->hout_dev[b]), static_cast<size_t>(kMaxNodes) * d.hidden * sizeof(float)));
    ACM_CUDA(cudaMalloc(reinterpret_cast<void**>(&c->hstats_dev[b]), sizeof(acm_block_stats)));
    ACM_CUDA(cudaEventCreateWithFlags(&c->ev_in[b], cudaEventDisableTiming));
    ACM_CUDA(cudaEventCreateWithFlags(&c->ev_done[b], cudaEventDisableTiming));
    ACM_CUDA(cudaEventCreateWithFlags(&c->ev_out[b], cudaEventDisableTiming));
  }
  return ACM_OK;
}
}  // namespace

acm_status acm_moe_verify_host(acm_ctx* c, int layer, const void* x_host, int T, const float* alpha_host,
                               const acm_select_params* params, float* out_host, acm_block_stats* stats_host,
                               acm_stream stream) {
  acm_status st = check_block_args(c, layer, T, true);
  if (st != ACM_OK) return st;
  if (!x_host || !alpha_host || !out_host || !params) return ACM_ERR_INVALID;
  if (c->layers[layer].has_resident) return ACM_ERR_UNSUPPORTED;
  st = ensure_host_path(c);
  if (st != ACM_OK) return st;
  const acm_model_desc& d = c->desc;
  const size_t elt = d.dtype == ACM_F32 ? 4 : 2;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int b = static_cast<int>(c->host_calls & 1ull);
  const bool reused = c->host_calls >= 2;
  // upload into set b once the kernels of the call before last (its previous user) are done with it
  if (reused) ACM_CUDA(cudaStreamWaitEvent(c->h2d_stream, c->ev_done[b], 0));
  ACM_CUDA(cudaMemcpyAsync(c->hx_dev[b], x_host, static_cast<size_t>(T) * d.hidden * elt, cudaMemcpyHostToDevice,
                           c->h2d_stream));
  ACM_CUDA(cudaMemcpyAsync(c->halpha_dev[b], alpha_host, static_cast<size_t>(T) * sizeof(float),
                           cudaMemcpyHostToDevice, c->h2d_stream));
  ACM_CUDA(cudaEventRecord(c->ev_in[b], c->h2d_stream));
  // kernels: after the upload, and after the download that last read this set's output buffer
  ACM_CUDA(cudaStreamWaitEvent(s, c->ev_in[b], 0));
  if (reused) ACM_CUDA(cudaStreamWaitEvent(s, c->ev_out[b], 0));
  st = acm_moe_verify(c, layer, c->hx_dev[b], T, c->halpha_dev[b], params, nullptr, c->hout_dev[b], nullptr, nullptr,
                      nullptr, stats_host ? c->hstats_dev[b] : nullptr, stream);
  if (st != ACM_OK) return st;
  ACM_CUDA(cudaEventRecord(c->ev_done[b], s));
  // download
  ACM_CUDA(cudaStreamWaitEvent(c->d2h_stream, c->ev_done[b], 0));
  ACM_CUDA(cudaMemcpyAsync(out_host, c->hout_dev[b], static_cast<size_t>(T) * d.hidden * sizeof(float),
                           cudaMemcpyDeviceToHost, c->d2h_stream));
  if (stats_host)
    ACM_CUDA(cudaMemcpyAsync(stats_host, c->hstats_dev[b], sizeof(acm_block_stats), cudaMemcpyDeviceToHost,
                             c->d2h_stream));
  ACM_CUDA(cudaEventRecord(c->ev_out[b], c->d2h_stream));
  c->host_calls += 1;
  c->host_h2d += static_cast<size_t>(T) * d.hidden * elt + static_cast<size_t>(T) * sizeof(float);
  c->host_d2h += static_cast<size_t>(T) * d.hidden * sizeof(float) + (stats_host ? sizeof(acm_block_stats) : 0);
  return ACM_OK;
}

acm_status acm_host_synchronize(acm_ctx* c) {
  if (!c) return ACM_ERR_INVALID;
  if (!c->d2h_stream) return ACM_OK;
  ACM_CUDA(cudaStreamSynchronize(c->d2h_stream));
  return ACM_OK;
}


acm_status acm_set_resident(acm_ctx* c, int layer, const uint32_t* resident_mask, const void* host_gate_up,
                            const void* host_down) {
  if (!c || layer < 0 || layer >= c->desc.n_layers) return ACM_ERR_INVALID;
  Layer& L = c->layers[layer];
  if (!resident_mask) {
    L.has_resident = false;
    L.has_pool = false;
    L.host_gate_up = L.host_down = nullptr;
    return ACM_OK;
  }
  if (L.mx) return ACM_ERR_UNSUPPORTED;   // MXFP4 layers: all-resident or behind a pool (acm_set_slot_pool)
  if (L.has_pool) return ACM_ERR_INVALID;      // clear the pool first (NULL mask)
  if (c->desc.dtype != ACM_BF16) return ACM_ERR_UNSUPPORTED;
  if (!host_gate_up || !host_down) return ACM_ERR_INVALID;
  acm_status st = ensure_staging(c);
  if (st != ACM_OK) return st;
  uint32_t words[4] = {0, 0, 0, 0};
  for (int w = 0; w < mask_words(c->desc.n_experts); ++w) words[w] = resident_mask[w];
  ACM_CUDA(cudaMemcpy(c->resident_dev + 4 * layer, words, sizeof words, cudaMemcpyHostToDevice));
  L.has_resident = true;
  L.host_gate_up = host_gate_up;
  L.host_down = host_down;
  return ACM_OK;
}

acm_status acm_set_slot_pool(acm_ctx* c, int layer, int n_slots, void* pool_gate_up, void* pool_down,
                             const void* host_gate_up, const void* host_down, const int32_t* initial_experts,
                             int n_initial) {
  if (!c || layer < 0 || layer >= c->desc.n_layers) return ACM_ERR_INVALID;
  const acm_model_desc& d = c->desc;
  if (d.dtype != ACM_BF16) return ACM_ERR_UNSUPPORTED;
  Layer& L = c->layers[layer];
  if (!L.set) return ACM_ERR_INVALID;
  if (n_slots < d.top_k || n_slots > kMaxSlots || !pool_gate_up || !pool_down || !host_gate_up || !host_down)
    return ACM_ERR_INVALID;
  if (n_initial < 0 || n_initial > n_slots || (n_initial > 0 && !initial_experts)) return ACM_ERR_INVALID;
  if (reinterpret_cast<uintptr_t>(pool_gate_up) % 128 != 0 || reinterpret_cast<uintptr_t>(pool_down) % 128 != 0)
    return ACM_ERR_INVALID;
  acm_status st = ensure_offload_common(c);
  if (st != ACM_OK) return st;
  if (L.mx) {                 // the pool is fed from the host tensors: their scale bytes must be in range
    const size_t rec = static_cast<size_t>(d.n_experts) * ((d.inter / 64) * (d.hidden / 128));
    const size_t rec_dn = static_cast<size_t>(d.n_experts) * ((d.hidden / 128) * (d.inter / 128));
    if (mx_max_scale_host(static_cast<const unsigned char*>(host_gate_up), rec) > kMxMaxScaleByte ||
        mx_max_scale_host(static_cast<const unsigned char*>(host_down), rec_dn) > kMxMaxScaleByte)
      return ACM_ERR_UNSUPPORTED;
  }
  if (!L.mx) {                // (the MXFP4 kernel fetches its tile records with plain bulk copies)
    st = encode_gate_up(c, &L.pool_map_gu, pool_gate_up, n_slots);
    if (st != ACM_OK) return st;
    st = encode_down(c, &L.pool_map_dn, pool_down, n_slots);
    if (st != ACM_OK) return st;
  }
  if (!L.gate_up && !L.mx) {          // no full device tensors: every descriptor the kernel is handed must still be valid
    L.maps.gate_up = L.pool_map_gu;
    L.maps.down = L.pool_map_dn;
    if (d.n_shared == 0) {
      L.maps.shared_gate_up = L.pool_map_gu;
      L.maps.shared_down = L.pool_map_dn;
    }
  }
  const int E = d.n_experts;
  L.n_slots = n_slots;
  L.pool_gate_up = pool_gate_up;
  L.pool_down = pool_down;
  L.host_gate_up = host_gate_up;
  L.host_down = host_down;
  L.slot_expert.assign(n_slots, -1);
  L.expert_slot.assign(E, -1);
  L.last_use.assign(n_slots, 0);
  L.tick = 0;
  L.pool_hits = L.pool_misses = L.pool_h2d = 0;
  size_t gu, dn;
  expert_tensor_bytes(d, L.mx, &gu, &dn);
  for (int i = 0; i < n_initial; ++i) {
    const int e = initial_experts[i];
    if (e < 0 || e >= E || L.expert_slot[e] >= 0) return ACM_ERR_INVALID;
    ACM_CUDA(cudaMemcpy(static_cast<char*>(pool_gate_up) + i * gu, static_cast<const char*>(host_gate_up) + e * gu, gu,
                        cudaMemcpyHostToDevice));
    ACM_CUDA(cudaMemcpy(static_cast<char*>(pool_down) + i * dn, static_cast<const char*>(host_down) + e * dn, dn,
                        cudaMemcpyHostToDevice));
    L.slot_expert[i] = e;
    L.expert_slot[e] = i;
  }
  for (int b = 0; b < 2; ++b) {
    if (!L.slot_of_dev[b]) ACM_CUDA(cudaMalloc(reinterpret_cast<void**>(&L.slot_of_dev[b]), sizeof(int32_t) * kMaxExperts));
    ACM_CUDA(cudaMemcpy(L.slot_of_dev[b], L.expert_slot.data(), sizeof(int32_t) * E, cudaMemcpyHostToDevice));
  }
  L.slot_of_cur = 0;
  uint32_t words[kMaskWords] = {0, 0, 0, 0};
  for (int e = 0; e < E; ++e)
    if (L.expert_slot[e] >= 0) words[e >> 5] |= 1u << (e & 31);
  ACM_CUDA(cudaMemcpy(c->resident_dev + 4 * layer, words, sizeof words, cudaMemcpyHostToDevice));
  L.has_resident = true;
  L.has_pool = true;
  return ACM_OK;
}

acm_status acm_pool_stats(acm_ctx* c, int layer, uint64_t* hits, uint64_t* misses, uint64_t* h2d_bytes,
                          int32_t* slot_expert, int reset) {
  if (!c || layer < 0 || layer >= c->desc.n_layers) return ACM_ERR_INVALID;
  Layer& L = c->layers[layer];
  if (!L.has_pool) return ACM_ERR_INVALID;
  if (hits) *hits = L.pool_hits;
  if (misses) *misses = L.pool_misses;
  if (h2d_bytes) *h2d_bytes = L.pool_h2d;
  if (slot_expert)
    for (int i = 0; i < L.n_slots; ++i) slot_expert[i] = L.slot_expert[i];
  if (reset) L.pool_hits = L.pool_misses = L.pool_h2d = 0;
  return ACM_OK;
}

acm_status acm_pool_plan(int n_experts, int n_slots, int32_t* slot_expert, uint64_t* last_use, uint64_t* tick,
                         const uint32_t* activated_mask, int32_t* load_expert, int32_t* load_slot, int32_t* load_wave,
                         int32_t* n_loads, int32_t* n_hits) {
  if (n_experts < 1 || n_experts > kMaxExperts || n_slots < 1 || n_slots > kMaxExperts || !slot_expert || !last_use ||
      !tick || !activated_mask || !load_expert || !load_slot || !load_wave || !n_loads || !n_hits)
    return ACM_ERR_INVALID;
  std::vector<int32_t> se(slot_expert, slot_expert + n_slots), es(n_experts, -1);
  std::vector<uint64_t> lu(last_use, last_use + n_slots);
  for (int sl = 0; sl < n_slots; ++sl) {
    if (se[sl] < -1 || se[sl] >= n_experts) return ACM_ERR_INVALID;
    if (se[sl] >= 0) {
      if (es[se[sl]] >= 0) return ACM_ERR_INVALID;      // an expert in two slots
      es[se[sl]] = sl;
    }
  }
  uint32_t act[kMaskWords] = {0, 0, 0, 0};
  for (int w = 0; w < mask_words(n_experts); ++w) act[w] = activated_mask[w];
  std::vector<PoolLoad> loads;
  int hits = 0;
  if (!plan_pool_block(n_experts, n_slots, se, es, lu, *tick, act, loads, hits)) return ACM_ERR_INVALID;
  for (size_t i = 0; i < loads.size(); ++i) {
    load_expert[i] = loads[i].expert;
    load_slot[i] = loads[i].slot;
    load_wave[i] = loads[i].wave;
  }
  *n_loads = static_cast<int32_t>(loads.size());
  *n_hits = hits;
  for (int sl = 0; sl < n_slots; ++sl) {
    slot_expert[sl] = se[sl];
    last_use[sl] = lu[sl];
  }
  return ACM_OK;
}

acm_status acm_h2d_bytes(acm_ctx* c, uint64_t* bytes_out, int reset) {
  if (!c || !bytes_out) return ACM_ERR_INVALID;
  *bytes_out = c->h2d_bytes;
  if (reset) c->h2d_bytes = 0;
  return ACM_OK;
}

acm_status acm_ffn_timing(acm_ctx* c, int enable, int capacity) {
  if (!c || capacity < 0) return ACM_ERR_INVALID;
  if (enable < 0) return ACM_ERR_INVALID;
  c->timing = enable != 0;
  c->timing_period = enable > 0 ? enable : 1;
  c->timing_seen = 0;
  c->ev_used = 0;
  while (c->timing && c->ev_pool.size() < static_cast<size_t>(2) * capacity) {
    cudaEvent_t e;
    ACM_CUDA(cudaEventCreate(&e));
    c->ev_pool.push_back(e);
  }
  return ACM_OK;
}

acm_status acm_ffn_time_ms(acm_ctx* c, float* total_ms, int32_t* launches) {
  if (!c || !total_ms || !launches) return ACM_ERR_INVALID;
  float total = 0.f;
  for (size_t i = 0; i + 1 < c->ev_used; i += 2) {
    ACM_CUDA(cudaEventSynchronize(c->ev_pool[i + 1]));
    float ms = 0.f;
    ACM_CUDA(cudaEventElapsedTime(&ms, c->ev_pool[i], c->ev_pool[i + 1]));
    total += ms;
  }
  *total_ms = total;
  *launches = static_cast<int32_t>(c->ev_used / 2);
  return ACM_OK;
}

acm_status acm_offload_timing(acm_ctx* c, int enable, int capacity) {
  if (!c || capacity < 0) return ACM_ERR_INVALID;
  c->off_timing = enable != 0;
  c->off_calls = 0;
  while (c->off_timing && c->off_ev.size() < static_cast<size_t>(5) * capacity) {
    cudaEvent_t e;
    ACM_CUDA(cudaEventCreate(&e));
    c->off_ev.push_back(e);
  }
  c->off_has_copies.assign(c->off_ev.size() / 5 + 1, 0);
  return ACM_OK;
}

acm_status acm_offload_times(acm_ctx* c, double* ms_out, int32_t* calls) {
  if (!c || !ms_out || !calls) return ACM_ERR_INVALID;
  double total = 0.0, resident = 0.0, copies = 0.0, stall = 0.0;
  for (size_t i = 0; i < c->off_calls; ++i) {
    cudaEvent_t* e = c->off_ev.data() + 5 * i;
    ACM_CUDA(cudaEventSynchronize(e[4]));
    float ms = 0.f;
    ACM_CUDA(cudaEventElapsedTime(&ms, e[0], e[4]));
    total += ms;
    ACM_CUDA(cudaEventElapsedTime(&ms, e[0], e[1]));
    resident += ms;
    if (c->off_has_copies[i]) {
      ACM_CUDA(cudaEventElapsedTime(&ms, e[2], e[3]));
      copies += ms;
      ACM_CUDA(cudaEventElapsedTime(&ms, e[1], e[3]));      // negative: the copies were done before the resident part was
      if (ms > 0.f) stall += ms;
    }
  }
  ms_out[0] = total; ms_out[1] = resident; ms_out[2] = copies; ms_out[3] = stall;
  *calls = static_cast<int32_t>(c->off_calls);
  return ACM_OK;
}

acm_status acm_stage_timing(acm_ctx* c, int enable) {
  if (!c) return ACM_ERR_INVALID;
  ACM_CUDA(cudaDeviceSynchronize());
  if (enable) {
    if (!c->trace) {
      const size_t bytes = sizeof(unsigned long long) * (32 * c->sm_count + 32);
      if (cudaMalloc(&c->trace, bytes) != cudaSuccess) return ACM_ERR_NOMEM;
      ACM_CUDA(cudaMemset(c->trace, 0, bytes));
    }
  } else if (c->trace) {
    ACM_CUDA(cudaFree(c->trace));
    c->trace = nullptr;
  }
  return ACM_OK;
}

acm_status acm_stage_times(acm_ctx* c, double* us_out) {
  if (!c || !us_out || !c->trace) return ACM_ERR_INVALID;
  ACM_CUDA(cudaDeviceSynchronize());
  std::vector<unsigned long long> buf(32 * static_cast<size_t>(c->sm_count) + 32);
  ACM_CUDA(cudaMemcpy(buf.data(), c->trace, sizeof(unsigned long long) * buf.size(), cudaMemcpyDeviceToHost));
  const unsigned long long* rt = buf.data() + 32 * static_cast<size_t>(c->sm_count);
  const unsigned long long t_in = rt[13], t_sel0 = rt[0], t_sel1 = rt[2], t_route = rt[3];
  if (t_in == 0 || t_sel0 < t_in || t_sel1 < t_sel0 || t_route < t_sel1) return ACM_ERR_INVALID;   // no fused call seen yet
  unsigned long long ffn0 = ~0ull, ffn1 = 0;
  for (int cta = 0; cta < c->sm_count; ++cta) {
    const unsigned long long* row = buf.data() + 32 * static_cast<size_t>(cta);
    if (row[0] >= t_in && row[0] < ffn0) ffn0 = row[0];          // (older stamps belong to earlier calls)
    for (int slot = 10; slot <= 11; ++slot)
      if (row[slot] >= t_in && row[slot] > ffn1) ffn1 = row[slot];
  }
  if (ffn1 == 0 || ffn0 == ~0ull || ffn1 < ffn0) return ACM_ERR_INVALID;
  us_out[0] = 1e-3 * static_cast<double>(t_sel0 - t_in);
  us_out[1] = 1e-3 * static_cast<double>(t_sel1 - t_sel0);
  us_out[2] = 1e-3 * static_cast<double>(t_route - t_sel1);
  us_out[3] = 1e-3 * static_cast<double>(ffn1 - ffn0);
  us_out[4] = 1e-3 * static_cast<double>(ffn1 - t_in);
  return ACM_OK;
}

acm_status acm_launch_count(acm_ctx* c, uint64_t* launches_out) {
  if (!c || !launches_out) return ACM_ERR_INVALID;
  *launches_out = c->launches;
  return ACM_OK;
}

acm_status acm_ffn_plan(int n_experts_streamed, int n_anchor_first, int hidden, int inter, int grid, int32_t* pieces,
                        int capacity, int32_t* n_pieces, int32_t* n_segments) {
  if (!pieces || !n_pieces || !n_segments || capacity < 0) return ACM_ERR_INVALID;
  if (n_experts_streamed < 1 || n_experts_streamed > kMaxSlots || n_anchor_first < 0 || n_anchor_first > n_experts_streamed ||
      hidden < 128 || hidden % 128 != 0 || inter < 64 || inter % 64 != 0 || grid < 1 || grid > 1024)
    return ACM_ERR_INVALID;
  using namespace acm::plan;
  const int tpe = inter / 64, kc1 = hidden / 128, kpe = (tpe + 1) / 2, h_tiles = hidden / 128;
  if (n_anchor_first * tpe > grid) return ACM_ERR_INVALID;      // the pre-segment gives a CTA at most one tile
  const FastDiv d_grid = make_fastdiv(grid), d_kc1 = make_fastdiv(kc1), d_tpe = make_fastdiv(tpe);
  int n = 0, n_seg = 0;
  for (int cta = 0; cta < grid; ++cta) {
    Plan pl = {};
    int base = 0;
    if (n_anchor_first > 0) {
      const Segment sg0 = Segment{1, 1, 0, n_anchor_first * tpe, 0, 0, 0, d_kc1, 0};
      pl.seg[0] = sg0;
      pl.range[0] = make_range(sg0, cta, d_grid, h_tiles);
      base = 1;
    }
    for (int lane = 3; lane >= 0; --lane)
      plan_lane(pl, lane, cta, n_experts_streamed, tpe, grid, d_kc1, kpe, d_grid, d_tpe, h_tiles, n_anchor_first, base);
    n_seg = pl.n_seg;
    for (int si = 0; si < pl.n_seg; ++si) {
      const Segment& sg = pl.seg[si];
      Sched sc(pl.range[si]);
      int t, k0, k1;
      while (sc.next(t, k0, k1)) {
        if (n < capacity) {
          int32_t* q = pieces + static_cast<size_t>(8) * n;
          q[0] = cta; q[1] = si; q[2] = sg.phase; q[3] = sg.phase == 1 ? sg.whole : 0;
          q[4] = sg.phase == 1 ? sg.t0 + t : t; q[5] = k0; q[6] = k1; q[7] = sg.phase == 1 ? sg.p1_index : sg.a0;
        }
        ++n;
      }
    }
  }
  *n_pieces = n;
  *n_segments = n_seg;
  return n <= capacity ? ACM_OK : ACM_ERR_NOMEM;
}

acm_status acm_set_overlap(acm_ctx* c, int level) {
  if (!c || level < ACM_OVERLAP_NONE || level > ACM_OVERLAP_ANCHORS) return ACM_ERR_INVALID;
  c->overlap = level;
  c->pdl = level >= ACM_OVERLAP_DEPENDENT;
  c->early_start = level >= ACM_OVERLAP_ELIGIBLE;
  c->anchor_start = level >= ACM_OVERLAP_ANCHORS;
  return ACM_OK;
}

acm_status acm_set_wait_limit(acm_ctx* c, uint64_t nanoseconds) {
  if (!c || nanoseconds < 1000ull || nanoseconds > 60ull * 1000000000ull) return ACM_ERR_INVALID;
  c->wait_limit_ns = nanoseconds;
  return ACM_OK;
}

acm_status acm_wait_report(acm_ctx* c, int32_t* site_out, int capacity, int32_t* n_ctas) {
  if (!c || !site_out || !n_ctas || capacity < 0) return ACM_ERR_INVALID;
  ACM_CUDA(cudaDeviceSynchronize());
  std::vector<int32_t> words(c->sm_count);
  ACM_CUDA(cudaMemcpy(words.data(), c->wait_diag, sizeof(int32_t) * c->sm_count, cudaMemcpyDeviceToHost));
  const int n = c->last_ffn_grid;
  *n_ctas = n;
  for (int i = 0; i < n && i < capacity; ++i)
    site_out[i] = (words[i] >> 8) == c->ffn_launch_no ? (words[i] & 0xff) : -1;      // -1: that CTA never started
  return ACM_OK;
}

acm_status acm_inject_unpublished_wait(acm_ctx* c, int layer, const void* x, int T, float* out, acm_stream stream) {
  acm_status st = check_block_args(c, layer, T, true);
  if (st != ACM_OK) return st;
  const Layer& L = c->layers[layer];
  if (!x || !out || (!L.gate_up && !L.mx_gate_up)) return ACM_ERR_INVALID;
  if (reinterpret_cast<uintptr_t>(x) % 16 != 0 || reinterpret_cast<uintptr_t>(out) % 16 != 0) return ACM_ERR_INVALID;
  if (c->desc.dtype != ACM_BF16 || L.has_resident) return ACM_ERR_UNSUPPORTED;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // a tag of its own, which no router or selection kernel is ever launched with
  int32_t epoch = 0;
  st = next_epoch(c, s, &epoch);
  if (st != ACM_OK) return st;
  ACM_CUDA(cudaMemsetAsync(out, 0, sizeof(float) * static_cast<size_t>(T) * c->desc.hidden, s));
  return run_ffn_list(c, L, x, T, 0, out, s, nullptr, nullptr, false, epoch);
}

acm_status acm_device_status(acm_ctx* c, acm_stream stream) {
  if (!c) return ACM_ERR_INVALID;
  ACM_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
  int32_t v = 0;
  ACM_CUDA(cudaMemcpy(&v, c->ws.status, sizeof v, cudaMemcpyDeviceToHost));
  if (v != 0) {
    // a launch that gave up may have left partial sums behind: restore the all-zero state the FFN kernel expects
    ACM_CUDA(cudaMemset(c->ws.status, 0, sizeof v));
    ACM_CUDA(cudaMemset(c->ws.frag, 0, c->frag_bytes));
    ACM_CUDA(cudaMemset(c->ws.frag_flag, 0, c->flag_bytes));
    ACM_CUDA(cudaMemset(c->ws.ticket, 0, 16));
    ACM_CUDA(cudaMemset(c->ws.sel_words, 0, 32 * kMaxEarlyBlocks));
    ACM_CUDA(cudaMemset(c->ws.anc_words, 0, 32 * kMaxEarlyBlocks));
    ACM_CUDA(cudaMemset(c->ws.root_words, 0, sizeof(unsigned long long) * kMaxExperts * kMaxEarlyBlocks));
    c->epoch = 0;
    ACM_CUDA(cudaMemset(c->ws.tile_done, 0, sizeof(int32_t) * kMaxNodes));
  }
  return static_cast<acm_status>(v);
}

}  // extern "C"
