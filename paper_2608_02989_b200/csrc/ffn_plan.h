// Work plan of one launch of the expert-FFN kernel: which CTA streams which part of which weight tile, in what
// order.  Pure integer logic, compiled for the device (the kernel works its plan out in its prologue, four lanes
// side by side) and for the host (acm_ffn_plan lists a plan so that its coverage can be checked without a GPU).
//
// Units of work.  A gate/up tile = 64 gate rows + the 64 matching up rows of one activated expert over the
// whole hidden dimension (kc1 pipeline stages of 128 K); tile number = slot * tiles_per_expert + sub-tile, slot =
// position of the expert in the launch's work list.  It needs the complete sum over K before its activation can
// be formed, so it is either given whole to one CTA or cut along K, the pieces' partial sums then meeting in the
// CTA that holds the tile's first chunk.  A down unit = one stage (128 K of one expert's intermediate features)
// of one 128-row output tile; down work is linear in K and is always cut evenly (partial output tiles are added
// in L2).  The down projection of an expert can start once all its gate/up tiles are finalised and stored.
//
// A launch that knows its whole work list at the start (G CTAs, n_tiles gate/up tiles):
//   with at least one tile per CTA:
//     1. the n_tiles mod G tiles that do not fill a round, cut evenly over all CTAs (their cross-CTA exchange
//        then hides behind the next segment)
//     2. whole tiles, one per CTA and round
//     3. down projection of the experts that were complete before the last round
//     4. down projection of the rest -- by then their activations have been stored
//   with fewer tiles than CTAs: gate/up of the first half of the experts, gate/up of the second half (both cut
//   evenly), then down of the first half, down of the second half.
// A launch that started on the anchors (n_pre experts, P = n_pre * tiles_per_expert tiles, one per CTA for CTAs
// [0, P), as segment 0) learns the rest of its list later; the CTAs [P, G) have been idle until then, while the
// others are still in their anchor tile:
//   fewer rest tiles than CTAs: they are dealt whole, one per CTA, to the idle CTAs first (no exchange at all);
//   else as above.  The anchors' experts are complete early: their down projection comes first.
// (Measured and dropped: every tile whole with the CTAs that get one tile less taking down work early -- the last
// round's experts then start their down projection too late; the leftover tiles after the whole rounds instead of
// before them; the leftover tiles cut over the idle CTAs only.)
#pragma once

#include <stdint.h>

#if defined(__CUDACC__)
#define ACM_PLAN_FN __host__ __device__ __forceinline__
#else
#define ACM_PLAN_FN inline
#endif

namespace acm {
namespace plan {

// Division by a launch constant through a precomputed 64-bit reciprocal (exact for n < 2^32): the schedules are
// walked by ONE thread per role, for which a hardware-less integer division is a chain of dozens of dependent
// instructions.
struct FastDiv {
  unsigned long long M;   // ceil(2^64 / d) for d >= 2; 0 = divide the plain way
  unsigned d;
};
inline FastDiv make_fastdiv(unsigned d) {
  FastDiv f;
  f.d = d;
  f.M = d > 1 ? 0xffffffffffffffffull / d + 1ull : 0ull;
  return f;
}
ACM_PLAN_FN FastDiv plain_div(unsigned d) {
  FastDiv f;
  f.d = d;
  f.M = 0ull;
  return f;
}
ACM_PLAN_FN unsigned fdiv(unsigned n, const FastDiv& f) {
  if (f.M == 0ull) return f.d == 1 ? n : n / f.d;
#if defined(__CUDA_ARCH__)
  return static_cast<unsigned>(__umul64hi(static_cast<unsigned long long>(n), f.M));
#else
  return static_cast<unsigned>((static_cast<unsigned __int128>(n) * f.M) >> 64);
#endif
}

struct Segment {
  int phase;      // 1 = gate/up, 2 = down
  int whole;      // gate/up only: 1 = whole tiles dealt round-robin, 0 = tiles cut evenly over the CTAs
  int t0, nt;     // gate/up: first tile and number of tiles
  int a0, a1;     // down: activated-expert slots [a0, a1)
  int p1_index;   // gate/up: which fragment buffer a cut segment uses
  FastDiv chunks; // K-chunks per tile: the per-tile constant for gate/up, (a1 - a0) * chunks per expert for down
  int rot;        // gate/up whole: tile i of the segment goes to CTA (rot + i) mod G
};
// This CTA's share of one segment.  Cut segments: a contiguous range of (tile, K-chunk) units; whole-tile
// segments: tiles u, u + G, u + 2G, ...  The divisions are done once per launch and every role then walks its
// share with additions only.
struct SegRange {
  unsigned u, u_end;     // cut: the CTA's unit range; whole: first tile and tile count of the segment
  int tile0, k00;        // cut: tile and chunk of unit u
  int kc;                // chunks per tile
  int stride;            // whole: the grid size (tile step); 0 for a cut segment
  unsigned n_stages;     // pipeline stages this CTA runs in the segment
};
struct Plan {
  Segment seg[5];      // [0] may be the anchors' pre-segment, then up to four
  SegRange range[5];   // this CTA's share of each segment
  volatile int n_seg;
  int n_pre;           // experts whose gate/up tiles the pre-segment covers (the first slots of the work list)
};

struct Sched {
  unsigned u, u_end;
  int tile, k0n, kc, stride;
  ACM_PLAN_FN explicit Sched(const SegRange& r) : u(r.u), u_end(r.u_end), tile(r.tile0), k0n(r.k00), kc(r.kc), stride(r.stride) {}
  ACM_PLAN_FN bool next(int& t, int& k0, int& k1) {
    if (stride > 0) {            // whole tiles: u counts tiles
      if (u >= u_end) return false;
      t = static_cast<int>(u);
      k0 = 0;
      k1 = kc;
      u += static_cast<unsigned>(stride);
      return true;
    }
    if (u >= u_end) return false;
    t = tile;
    k0 = k0n;
    const int rem = static_cast<int>(u_end - u);
    k1 = rem < kc - k0 ? k0 + rem : kc;
    u += static_cast<unsigned>(k1 - k0);
    ++tile;
    k0n = 0;
    return true;
  }
};

// First (tile, K-chunk) unit of CTA `cta` in a cut gate/up segment (cta = G gives the number of units).
ACM_PLAN_FN unsigned cut_begin(const Segment& sg, int cta, const FastDiv& d_grid) {
  return fdiv(static_cast<unsigned>(sg.nt) * sg.chunks.d * static_cast<unsigned>(cta), d_grid);
}

// Range of one segment for CTA `cta` (see SegRange).  (tiles * chunks * grid fits 32 bits: the launcher checks.)
ACM_PLAN_FN SegRange make_range(const Segment& sg, int cta, const FastDiv& d_grid, int h_tiles) {
  SegRange r;
  r.kc = static_cast<int>(sg.chunks.d);
  if (sg.phase == 1 && sg.whole) {
    const int first = cta >= sg.rot ? cta - sg.rot : cta - sg.rot + static_cast<int>(d_grid.d);
    r.u = static_cast<unsigned>(first);
    r.u_end = static_cast<unsigned>(sg.nt);
    r.tile0 = 0; r.k00 = 0;
    r.stride = static_cast<int>(d_grid.d);
    r.n_stages = r.u < r.u_end ? fdiv(r.u_end - r.u + d_grid.d - 1u, d_grid) * sg.chunks.d : 0u;
    return r;
  }
  r.stride = 0;
  const unsigned tiles = sg.phase == 1 ? static_cast<unsigned>(sg.nt) : static_cast<unsigned>(h_tiles);
  const unsigned total = tiles * sg.chunks.d;
  r.u = fdiv(total * static_cast<unsigned>(cta), d_grid);
  r.u_end = fdiv(total * static_cast<unsigned>(cta + 1), d_grid);
  r.tile0 = static_cast<int>(fdiv(tiles * static_cast<unsigned>(cta), d_grid));   // = floor(u / chunks): floors nest
  r.k00 = static_cast<int>(r.u - static_cast<unsigned>(r.tile0) * sg.chunks.d);
  r.n_stages = r.u_end - r.u;
  return r;
}

// The plan behind the optional pre-segment: lane i of four works out the i-th segment and this CTA's range in it
// (the candidates in order, each present or not), so nothing waits for a serial pass; lane 0 publishes the count
// last.  n_act counts every slot of the work list (the n_pre pre-streamed experts first); base = 1 when segment 0
// is the pre-segment.
ACM_PLAN_FN void plan_lane(Plan& pl, int lane, int cta, int n_act, int tpe, int grid, const FastDiv& d_kc1, int kpe,
                           const FastDiv& d_grid, const FastDiv& d_tpe, int h_tiles, int n_pre = 0, int base = 0) {
  const int t_pre = n_pre * tpe;                   // tiles (= CTAs) of the pre-segment
  const int n_t = (n_act - n_pre) * tpe;
  const int rounds = static_cast<int>(fdiv(static_cast<unsigned>(n_t), d_grid)), rem = n_t - rounds * grid;
  // candidates in execution order: two gate/up segments, two down segments
  Segment c0 = {}, c1 = {}, c2 = {}, c3 = {};
  bool h0 = false, h1 = false, h2 = false, h3 = false;
  int a_split;
  if (rounds == 0 && n_pre > 0) {
    // behind the anchors, fewer tiles than CTAs: dealt whole, the idle CTAs [t_pre, G) first
    a_split = n_pre;
    c0 = Segment{1, 1, t_pre, n_t, 0, 0, 0, d_kc1, t_pre < grid ? t_pre : 0};             h0 = n_t > 0;
  } else if (rounds == 0) {
    const int nA = (n_act + 1) / 2;
    a_split = nA;
    c0 = Segment{1, 0, 0, nA * tpe, 0, 0, 0, d_kc1, 0};                                   h0 = nA > 0;
    c1 = Segment{1, 0, nA * tpe, (n_act - nA) * tpe, 0, 0, 1, d_kc1, 0};                  h1 = n_act > nA;
  } else {
    a_split = n_pre + static_cast<int>(fdiv(static_cast<unsigned>(rem + (rounds - 1) * grid), d_tpe));
    c0 = Segment{1, 0, t_pre, rem, 0, 0, 0, d_kc1, 0};                                    h0 = rem > 0;
    c1 = Segment{1, 1, t_pre + rem, rounds * grid, 0, 0, 1, d_kc1, 0};                    h1 = true;
  }
  c2 = Segment{2, 0, 0, 0, 0, a_split, 0, plain_div(static_cast<unsigned>(a_split * kpe)), 0};                 h2 = a_split > 0;
  c3 = Segment{2, 0, 0, 0, a_split, n_act, 1, plain_div(static_cast<unsigned>((n_act - a_split) * kpe)), 0};   h3 = n_act > a_split;
  const int i0 = 0, i1 = i0 + h0, i2 = i1 + h1, i3 = i2 + h2, n = i3 + h3;
  Segment mine = c0;
  bool have = false;
  if (h0 && i0 == lane) { mine = c0; have = true; }
  if (h1 && i1 == lane) { mine = c1; have = true; }
  if (h2 && i2 == lane) { mine = c2; have = true; }
  if (h3 && i3 == lane) { mine = c3; have = true; }
  if (have) {
    pl.seg[base + lane] = mine;
    pl.range[base + lane] = make_range(mine, cta, d_grid, h_tiles);
  }
#if defined(__CUDA_ARCH__)
  __syncwarp(0xfu);            // (called by lanes 0..3: the segments are in place before their count is)
#endif
  if (lane == 0) pl.n_seg = base + n;
}

}  // namespace plan
}  // namespace acm
