// AcceptMoE verifier-side MoE layer -- CPU ORACLE.  TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, obviously-correct restatement of what the hot path computes for
// one verification block and one MoE layer: router + softmax + natural top-k
// (Section 3.1, Eq. 1), commitment-weighted demand (Eq. 3, Eq. 4), root anchor
// (Eq. 5), self-sized eligible set (Eq. 6), residency-aware pruning (Eq. 7),
// restricted top-k routing (Eq. 2) and the SwiGLU expert FFN with weighted
// combine.  It shares no code, header, table or constant generator with the CUDA
// library; only tests, the smoke check and the benchmark's CPU-baseline leg may
// call it.  The product path never does.
//
// Precision.  Every quantity that decides a set member, a count or an index
// (logits, softmax, demand, entropy, effective rank) is computed in IEEE
// binary32 in a fixed, documented order, so that an independent implementation
// can reproduce the decision bit for bit.  Quantities that are only compared
// within a tolerance (routing weights, FFN outputs) are computed in binary64.
//
// Pins (see tests/test_oracle_*.py): exp/log series against libm in double;
// router against a double dot product; demand, effective rank and pruning
// against closed forms and brute force on tiny inputs; the FFN against a
// double-precision dense matmul chain.  Whole-method outputs on real models:
// parity unpinned (the paper prints no per-block set).
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -fno-fast-math -mfma -fopenmp -shared -fPIC

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

constexpr int kMaxExperts = 128;   // padded length of every sum over the expert axis

inline float bf16_bits_to_float(uint16_t b) {
  uint32_t u = static_cast<uint32_t>(b) << 16;
  float f;
  std::memcpy(&f, &u, sizeof f);
  return f;
}

// element (row, col) of a row-major matrix stored as fp32 (dtype 0) or bf16 bits (dtype 1)
inline float load_elem(const void* base, int dtype, size_t index) {
  if (dtype == 0) return static_cast<const float*>(base)[index];
  return bf16_bits_to_float(static_cast<const uint16_t*>(base)[index]);
}

// ---------------------------------------------------------------------------
// Elementary functions with a fixed arithmetic recipe (binary32 throughout).
// exp: range reduction x = n ln2 + r with a two-term ln2, degree-7 Taylor
// polynomial in Horner form, scaling by 2^n through the exponent field.
// ---------------------------------------------------------------------------
float series_expf(float x) {
  x = std::fmin(std::fmax(x, -87.0f), 88.0f);
  const float n = std::rint(x * 0x1.715476p+0f);
  float r = std::fmaf(n, -0x1.62e400p-1f, x);
  r = std::fmaf(n, -0x1.7f7d1cp-20f, r);
  float p = 0x1.a01a02p-13f;            // 1/7!
  p = std::fmaf(p, r, 0x1.6c16c2p-10f); // 1/6!
  p = std::fmaf(p, r, 0x1.111112p-7f);  // 1/5!
  p = std::fmaf(p, r, 0x1.555556p-5f);  // 1/4!
  p = std::fmaf(p, r, 0x1.555556p-3f);  // 1/3!
  p = std::fmaf(p, r, 0.5f);
  p = std::fmaf(p, r, 1.0f);
  p = std::fmaf(p, r, 1.0f);
  const int32_t ni = static_cast<int32_t>(n);
  const uint32_t bits = static_cast<uint32_t>(ni + 127) << 23;
  float scale;
  std::memcpy(&scale, &bits, sizeof scale);
  return p * scale;
}

// log of a positive normal number: q = m 2^e with m in (sqrt(1/2), sqrt(2)],
// log m = 2 atanh(s), s = (m-1)/(m+1), odd series up to s^11.
float series_logf(float q) {
  uint32_t bits;
  std::memcpy(&bits, &q, sizeof bits);
  int32_t e = static_cast<int32_t>((bits >> 23) & 0xffu) - 127;
  const uint32_t mbits = (bits & 0x007fffffu) | 0x3f800000u;
  float m;
  std::memcpy(&m, &mbits, sizeof m);
  if (m > 0x1.6a09e6p+0f) {
    m = m * 0.5f;
    e += 1;
  }
  const float s = (m - 1.0f) / (m + 1.0f);
  const float s2 = s * s;
  float p = 0x1.745d18p-4f;             // 1/11
  p = std::fmaf(p, s2, 0x1.c71c72p-4f); // 1/9
  p = std::fmaf(p, s2, 0x1.24924ap-3f); // 1/7
  p = std::fmaf(p, s2, 0x1.99999ap-3f); // 1/5
  p = std::fmaf(p, s2, 0x1.555556p-2f); // 1/3
  p = std::fmaf(p, s2, 1.0f);
  const float lm = 2.0f * (s * p);
  return std::fmaf(static_cast<float>(e), 0x1.62e430p-1f, lm);
}

// Sum over the expert axis: values sit in their own slot of a 128-long array
// (unused slots +0), then a halving tree a[i] += a[i+s], s = 64, 32, ..., 1.
float tree_sum_128(const float* v, int n) {
  float a[kMaxExperts];
  for (int i = 0; i < kMaxExperts; ++i) a[i] = (i < n) ? v[i] : 0.0f;
  for (int s = kMaxExperts / 2; s >= 1; s /= 2)
    for (int i = 0; i < s; ++i) a[i] = a[i] + a[i + s];
  return a[0];
}

inline bool mask_has(const uint32_t* mask, int e) { return (mask[e >> 5] >> (e & 31)) & 1u; }
inline void mask_set(uint32_t* mask, int e) { mask[e >> 5] |= (1u << (e & 31)); }
inline void mask_clear(uint32_t* mask, int e) { mask[e >> 5] &= ~(1u << (e & 31)); }

// indices of `cand` ordered by (score descending, index ascending)
std::vector<int> order_desc(const std::vector<int>& cand, const float* score) {
  std::vector<int> o(cand);
  std::stable_sort(o.begin(), o.end(), [&](int a, int b) {
    if (score[a] != score[b]) return score[a] > score[b];
    return a < b;
  });
  return o;
}

}  // namespace

extern "C" {

struct orc_select_params {
  int32_t demand;        // 0: Eq. 4 (mass inside natural top-k); 1: full router mass; 2: natural votes
  int32_t use_anchors;   // 1: Eq. 5 anchors kept unconditionally
  int32_t fixed_budget;  // 0: self-sized (Eq. 6); B > 0: total set size held at B
  float ceil_guard;      // tau in ceil(exp(H) - tau)
  int32_t residency;     // 0 off; 1: Eq. 7; 2: (S intersect resident) union anchors
  int32_t max_remove;    // optional cap on Eq. 7 removals (E = nonbinding)
};

struct orc_select_stats {
  int32_t n_anchor, n_er, n_eligible, n_eligible_pruned, n_natural_union, displaced_aS, pruned_m;
  float residual_mass, entropy, perplexity;
};

float orc_expf(float x) { return series_expf(x); }
float orc_logf(float x) { return series_logf(x); }
void orc_expf_array(const float* x, float* y, int64_t n) { for (int64_t i = 0; i < n; ++i) y[i] = series_expf(x[i]); }
void orc_logf_array(const float* x, float* y, int64_t n) { for (int64_t i = 0; i < n; ++i) y[i] = series_logf(x[i]); }
float orc_tree_sum(const float* v, int n) { return tree_sum_128(v, n); }

// Eq. 3: alpha_t = p_hat[d_t]^beta * N_{d_t}^{-1/2}; evaluated in double, rounded once.
int orc_node_weights(const int32_t* depth, int T, const float* p_table, int n_depths, float beta,
                     int width_norm, float* alpha_out) {
  std::vector<int> width(n_depths, 0);
  for (int t = 0; t < T; ++t) {
    if (depth[t] < 0 || depth[t] >= n_depths) return 1;
    width[depth[t]] += 1;
  }
  for (int t = 0; t < T; ++t) {
    const int d = depth[t];
    double a = std::pow(static_cast<double>(p_table[d]), static_cast<double>(beta));
    if (width_norm) a = a / std::sqrt(static_cast<double>(width[d]));
    alpha_out[t] = static_cast<float>(a);
  }
  return 0;
}

// Section 3.1: z_t = W_r x_t (+ bias), r_t = softmax(z_t), K_t = TopK_k.
// The dot product keeps 32 interleaved partial sums (partial l takes h = l, l+32, ...
// in ascending order with fused multiply-add) and folds them with a halving tree.
int orc_router(const void* x, const void* w_router, const float* bias, int T, int H, int E, int k,
               int dtype, float* logits, float* probs, int32_t* nat_idx) {
  if (E > kMaxExperts || k > E) return 1;
  for (int t = 0; t < T; ++t) {
    float* z = logits + static_cast<size_t>(t) * E;
    for (int e = 0; e < E; ++e) {
      float part[32];
      for (int l = 0; l < 32; ++l) part[l] = 0.0f;
      for (int h = 0; h < H; ++h) {
        const float xv = load_elem(x, dtype, static_cast<size_t>(t) * H + h);
        const float wv = load_elem(w_router, dtype, static_cast<size_t>(e) * H + h);
        part[h & 31] = std::fmaf(xv, wv, part[h & 31]);
      }
      for (int s = 16; s >= 1; s /= 2)
        for (int i = 0; i < s; ++i) part[i] = part[i] + part[i + s];
      float v = part[0];
      if (bias) v = v + bias[e];
      z[e] = v;
    }
    // softmax over the expert axis
    float zmax = z[0];
    for (int e = 1; e < E; ++e) zmax = std::fmax(zmax, z[e]);
    float y[kMaxExperts];
    for (int e = 0; e < E; ++e) y[e] = series_expf(z[e] - zmax);
    const float denom = tree_sum_128(y, E);
    for (int e = 0; e < E; ++e) probs[static_cast<size_t>(t) * E + e] = y[e] / denom;
    // natural top-k, ranked on the logits: (z descending, index ascending)
    std::vector<int> all(E);
    for (int e = 0; e < E; ++e) all[e] = e;
    const std::vector<int> ord = order_desc(all, z);
    for (int j = 0; j < k; ++j) nat_idx[static_cast<size_t>(t) * k + j] = ord[j];
  }
  return 0;
}

// Sections 3.2-3.4: demand (Eq. 4), anchors (Eq. 5), self-sizing (Eq. 6), pruning (Eq. 7).
int orc_select_eligible(const float* probs, const int32_t* nat_idx, int T, int E, int k,
                        const float* alpha, const int32_t* anchor_nodes, int n_anchor_nodes,
                        const orc_select_params* prm, const uint32_t* resident_mask,
                        uint32_t* eligible_mask, uint32_t* unpruned_mask, int32_t* eligible_count,
                        float* demand_out, orc_select_stats* stats) {
  if (E > kMaxExperts || k > E || T < 1) return 1;
  const int words = (E + 31) / 32;

  // natural votes v_e and membership e in K_t
  std::vector<int> votes(E, 0);
  std::vector<uint8_t> in_topk(static_cast<size_t>(T) * E, 0);
  for (int t = 0; t < T; ++t)
    for (int j = 0; j < k; ++j) {
      const int e = nat_idx[static_cast<size_t>(t) * k + j];
      if (e < 0 || e >= E) return 1;
      in_topk[static_cast<size_t>(t) * E + e] = 1;
      votes[e] += 1;
    }

  // demand u_e, nodes in ascending order, fused multiply-add in binary32
  float u[kMaxExperts];
  for (int e = 0; e < E; ++e) {
    float acc = 0.0f;
    if (prm->demand == 2) {
      acc = static_cast<float>(votes[e]);
    } else {
      for (int t = 0; t < T; ++t) {
        const bool take = (prm->demand == 1) || in_topk[static_cast<size_t>(t) * E + e];
        if (take) acc = std::fmaf(alpha[t], probs[static_cast<size_t>(t) * E + e], acc);
      }
    }
    u[e] = acc;
    if (demand_out) demand_out[e] = acc;
  }

  // anchor set A
  uint32_t A[4] = {0, 0, 0, 0};
  int nA = 0;
  if (prm->use_anchors) {
    const int32_t root = 0;
    const int32_t* nodes = anchor_nodes ? anchor_nodes : &root;
    const int n_nodes = anchor_nodes ? n_anchor_nodes : 1;
    for (int a = 0; a < n_nodes; ++a) {
      const int t = nodes[a];
      if (t < 0 || t >= T) return 1;
      for (int j = 0; j < k; ++j) {
        const int e = nat_idx[static_cast<size_t>(t) * k + j];
        if (!mask_has(A, e)) { mask_set(A, e); ++nA; }
      }
    }
  }

  // residual experts R, their positive parts, total mass Z
  std::vector<int> R;
  float upos[kMaxExperts];
  int n_positive = 0;
  for (int e = 0; e < E; ++e) {
    upos[e] = 0.0f;
    if (!mask_has(A, e)) {
      R.push_back(e);
      upos[e] = std::fmax(u[e], 0.0f);
      if (u[e] > 0.0f) ++n_positive;
    }
  }
  const float Z = tree_sum_128(upos, E);

  float entropy = 0.0f, perp = 0.0f;
  int n_er = 0;
  int n_keep;
  const int floor_keep = std::max(0, k - nA);   // |S| >= k
  if (prm->fixed_budget > 0) {
    n_keep = std::max(0, prm->fixed_budget - nA);
    n_keep = std::max(n_keep, floor_keep);
  } else if (Z > 0.0f) {
    float hterm[kMaxExperts];
    for (int e = 0; e < E; ++e) {
      const float q = upos[e] / Z;
      hterm[e] = (q >= 0x1p-126f) ? q * series_logf(q) : 0.0f;
    }
    entropy = -tree_sum_128(hterm, E);
    perp = series_expf(entropy);
    n_er = static_cast<int>(std::ceil(perp - prm->ceil_guard));
    n_er = std::min(std::max(n_er, 1), n_positive);
    n_keep = std::max(n_er, floor_keep);
  } else {
    n_keep = floor_keep;
  }
  n_keep = std::min(n_keep, static_cast<int>(R.size()));

  uint32_t S[4] = {A[0], A[1], A[2], A[3]};
  const std::vector<int> ranked = order_desc(R, u);
  for (int j = 0; j < n_keep; ++j) mask_set(S, ranked[j]);
  const int nS = nA + n_keep;

  // natural union K and displaced assignments a(S)
  int n_union = 0, aS = 0;
  for (int e = 0; e < E; ++e)
    if (votes[e] > 0) {
      ++n_union;
      if (!mask_has(S, e)) aS += votes[e];
    }

  uint32_t Sp[4] = {S[0], S[1], S[2], S[3]};
  int nSp = nS, m_star = 0;
  if (prm->residency == 1 && resident_mask) {
    std::vector<int> C;
    for (int e = 0; e < E; ++e)
      if (mask_has(S, e) && !mask_has(resident_mask, e)) C.push_back(e);
    std::stable_sort(C.begin(), C.end(), [&](int a, int b) {
      if (u[a] != u[b]) return u[a] < u[b];
      return a < b;
    });
    int moved = 0;
    for (size_t j = 0; j < C.size(); ++j) {
      const int m = static_cast<int>(j) + 1;
      moved += votes[C[j]];
      if (moved > aS || nS - m < k || m > prm->max_remove) break;
      m_star = m;
    }
    for (int j = 0; j < m_star; ++j) mask_clear(Sp, C[j]);
    nSp = nS - m_star;
  } else if (prm->residency == 2 && resident_mask) {
    nSp = 0;
    for (int w = 0; w < 4; ++w) Sp[w] = 0;
    for (int e = 0; e < E; ++e)
      if ((mask_has(S, e) && mask_has(resident_mask, e)) || mask_has(A, e)) { mask_set(Sp, e); ++nSp; }
    m_star = nS - nSp;
  }

  for (int w = 0; w < words; ++w) {
    eligible_mask[w] = Sp[w];
    if (unpruned_mask) unpruned_mask[w] = S[w];
  }
  *eligible_count = nSp;
  if (stats) {
    stats->n_anchor = nA;
    stats->n_er = n_er;
    stats->n_eligible = nS;
    stats->n_eligible_pruned = nSp;
    stats->n_natural_union = n_union;
    stats->displaced_aS = aS;
    stats->pruned_m = m_star;
    stats->residual_mass = Z;
    stats->entropy = entropy;
    stats->perplexity = perp;
  }
  return 0;
}

// Eq. 2: top-k of z_t over the eligible experts, (z descending, index ascending); slots
// beyond the number of eligible experts hold -1 with weight 0.  Weights (double):
// 0 renormalised over the selected experts, 1 unmasked softmax probability,
// 2 softmax over the eligible experts only; each times routed_scale.
int orc_route_restricted(const float* logits, const uint32_t* eligible_mask, int T, int E, int k,
                         int weighting, double routed_scale, int32_t* idx, double* w) {
  if (E > kMaxExperts) return 1;
  for (int t = 0; t < T; ++t) {
    const float* z = logits + static_cast<size_t>(t) * E;
    std::vector<int> cand;
    for (int e = 0; e < E; ++e)
      if (mask_has(eligible_mask, e)) cand.push_back(e);
    const std::vector<int> ord = order_desc(cand, z);
    const int n_sel = std::min<int>(k, static_cast<int>(ord.size()));
    double zmax = z[0];
    for (int e = 1; e < E; ++e) zmax = std::max(zmax, static_cast<double>(z[e]));
    double sum_all = 0.0, sum_elig = 0.0, sum_sel = 0.0;
    for (int e = 0; e < E; ++e) {
      const double y = std::exp(static_cast<double>(z[e]) - zmax);
      sum_all += y;
      if (mask_has(eligible_mask, e)) sum_elig += y;
    }
    for (int j = 0; j < n_sel; ++j) sum_sel += std::exp(static_cast<double>(z[ord[j]]) - zmax);
    for (int j = 0; j < k; ++j) {
      if (j >= n_sel) {
        idx[static_cast<size_t>(t) * k + j] = -1;
        w[static_cast<size_t>(t) * k + j] = 0.0;
        continue;
      }
      const int e = ord[j];
      const double y = std::exp(static_cast<double>(z[e]) - zmax);
      const double den = (weighting == 0) ? sum_sel : (weighting == 1) ? sum_all : sum_elig;
      idx[static_cast<size_t>(t) * k + j] = e;
      w[static_cast<size_t>(t) * k + j] = routed_scale * y / den;
    }
  }
  return 0;
}

// y_t = sum_{e in K~_t} w_{t,e} W_down_e ( silu(W_gate_e x_t) * (W_up_e x_t) )  (+ shared experts, weight 1)
// gate_up: [E, 2I, H] rows 0..I-1 gate, I..2I-1 up; down: [E, H, I].  Double accumulation.
int orc_expert_ffn(const void* x, int T, int H, int I, int E, int k, int dtype, const int32_t* idx,
                   const double* w, const void* gate_up, const void* down, int n_shared,
                   const void* shared_gate_up, const void* shared_down, double* out) {
  (void)E;
#pragma omp parallel for schedule(dynamic, 1)
  for (int t = 0; t < T; ++t) {
    std::vector<double> y(H, 0.0), act(I);
    const size_t xoff = static_cast<size_t>(t) * H;
    for (int j = 0; j < k + n_shared; ++j) {
      const void* gu;
      const void* dn;
      int e;
      double weight;
      if (j < k) {
        e = idx[static_cast<size_t>(t) * k + j];
        if (e < 0) continue;
        weight = w[static_cast<size_t>(t) * k + j];
        gu = gate_up;
        dn = down;
      } else {
        e = j - k;
        weight = 1.0;
        gu = shared_gate_up;
        dn = shared_down;
      }
      const size_t gu_base = static_cast<size_t>(e) * 2 * I * H;
      for (int i = 0; i < I; ++i) {
        double g = 0.0, u = 0.0;
        const size_t grow = gu_base + static_cast<size_t>(i) * H;
        const size_t urow = gu_base + static_cast<size_t>(I + i) * H;
        for (int h = 0; h < H; ++h) {
          const double xv = load_elem(x, dtype, xoff + h);
          g += static_cast<double>(load_elem(gu, dtype, grow + h)) * xv;
          u += static_cast<double>(load_elem(gu, dtype, urow + h)) * xv;
        }
        act[i] = (g / (1.0 + std::exp(-g))) * u;
      }
      const size_t dn_base = static_cast<size_t>(e) * H * I;
      for (int h = 0; h < H; ++h) {
        double acc = 0.0;
        const size_t drow = dn_base + static_cast<size_t>(h) * I;
        for (int i = 0; i < I; ++i) acc += static_cast<double>(load_elem(dn, dtype, drow + i)) * act[i];
        y[h] += weight * acc;
      }
    }
    for (int h = 0; h < H; ++h) out[xoff + h] = y[h];
  }
  return 0;
}

}  // extern "C"
