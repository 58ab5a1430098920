// Work decomposition of one verification-attention call, shared by host and device code.
//
// Rows.  For KV head g the G = Hq/Hkv query heads that read it are stacked with the T tree
// nodes into G*T query rows, row r = t*G + i  <->  (node t, head g*G + i).  Rows are cut into
// row blocks of RB (128 or 256) rows; a (KV head, row block) pair is a "problem".
//
// Units.  The prefix is cut into key tiles of 128 tokens; the tree keys form one more tile.  A
// problem therefore has UPP = ceil(L/128) + 1 units, the last one being the tree tile.  All
// units of all problems are laid out in one line (problem-major) and cut into n_cta contiguous
// ranges; worker c (a CTA, or a cluster of two CTAs for the paired kernel) owns units
// [unit_start(c), unit_start(c+1)).  With cpp > 0 every problem gets the same whole number cpp of
// workers and its units are spread evenly over them, so that no worker straddles two problems;
// with cpp == 0 the whole line is cut into n_cta nearly equal ranges.  The part of a worker's
// range that lies inside one problem is a "segment" and yields one partial result (unnormalised
// output, running maximum, row sum) in slot c + problem.  Slots are unique because both c and the
// problem index are non-decreasing along the line.
#ifndef SPECEXT_PLAN_H_
#define SPECEXT_PLAN_H_

#include <stdint.h>

#if defined(__CUDACC__)
#define SPX_HD __host__ __device__ __forceinline__
#else
#define SPX_HD inline
#endif

#define SPX_TILE_KEYS 128

struct AttnPlan {
  int Hq, Hkv, G, D, L, T, C;
  int rows;        // G*T query rows per KV head
  int RB;          // rows per row block (128 or 256)
  int n_rblk;      // row blocks per KV head
  int NP;          // problems = Hkv * n_rblk
  int TPH;         // prefix key tiles per problem = ceil(L/128)
  int UPP;         // units per problem = TPH + 1 (tree tile last)
  int U;           // total units
  int n_cta;       // workers of the attention kernel (<= U)
  int kernel;      // 1 CUDA-core kernel, 2 one-CTA tensor-core kernel, 3 paired-CTA tensor-core kernel
  int cpp;         // workers per problem, or 0 when the line of units is cut without regard to problems
  int q, rem;      // cpp > 0: UPP = q*cpp + rem;  cpp == 0: U = q*n_cta + rem
  int n_slots;     // n_cta + NP - 1 partial slots
  int max_segs;    // upper bound on segments per problem
  int CPT;         // chunks per key tile = 128 / C
  int NC;          // ceil(L/C)
  int want_score;
  float scale2;    // softmax_scale * log2(e)
  // workspace offsets in floats
  long long off_part_o, off_part_m, off_part_l, off_mass, off_mref, total_floats;
};

SPX_HD int spx_unit_start(const AttnPlan& p, int c) {
  if (p.cpp > 0) {
    const int prob = c / p.cpp, k = c - prob * p.cpp;
    return prob * p.UPP + k * p.q + (k < p.rem ? k : p.rem);
  }
  return c * p.q + (c < p.rem ? c : p.rem);
}

// Worker that owns unit u.
SPX_HD int spx_unit_owner(const AttnPlan& p, int u) {
  const int big = p.rem * (p.q + 1);
  if (p.cpp > 0) {
    const int prob = u / p.UPP, w = u - prob * p.UPP;
    return prob * p.cpp + (w < big ? w / (p.q + 1) : p.rem + (w - big) / p.q);
  }
  return u < big ? u / (p.q + 1) : p.rem + (u - big) / p.q;
}

// The part of a worker's unit range that lies inside one problem is a run of `n_units` units starting
// at tile `tile_lo`.  When the prefix length is only known on the device (Ld <= L, the planned
// capacity), just the first tph_eff = ceil(Ld/128) prefix tiles exist; the tree tile (unit TPH, the
// last of the problem) always does.  n = n_pref + has_tree tiles are processed: tile_lo + j for
// j < n_pref, then the tree tile.  With tph_eff == TPH this is the planned run itself.
struct SpxSeg {
  int n_pref, has_tree, n;
};
SPX_HD SpxSeg spx_segment(const AttnPlan& p, int tile_lo, int n_units, int tph_eff) {
  SpxSeg s;
  const int end = tile_lo + n_units;                 // exclusive, <= UPP
  s.has_tree = end == p.UPP ? 1 : 0;
  int pref_end = end - s.has_tree;                   // <= TPH
  if (pref_end > tph_eff) pref_end = tph_eff;
  s.n_pref = pref_end > tile_lo ? pref_end - tile_lo : 0;
  s.n = s.n_pref + s.has_tree;
  return s;
}
SPX_HD int spx_seg_tile(const AttnPlan& p, const SpxSeg& s, int tile_lo, int j) {
  return j < s.n_pref ? tile_lo + j : p.TPH;
}

#endif  // SPECEXT_PLAN_H_
