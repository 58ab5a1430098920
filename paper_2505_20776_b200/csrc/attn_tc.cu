// Hybrid Tree Attention on the sm_100a tensor cores: split-over-KV partial attention of the stacked
// (query head x tree node) rows of one KV head against 128-key tiles of the prefix and the tree.
//
// CTA = 3 warpgroups (384 threads), one CTA per SM, persistent over its range of (problem, key
// tile) units:
//   warps 0-3   softmax of row tile 0, one thread per query row: one tcgen05.ld of the whole
//               128-column S row into registers, maximum with lazy rescaling of O, exp2 in fp32,
//               row and per-chunk sums from the unrounded exponentials, P rounded to bf16 back into
//               the columns S occupied.  Warps 4-7: the same for row tile 1.
//   warp 8      TMA producer: Q tile of the segment (once), then K and V tiles into a shared-memory
//               ring (128-byte swizzle, 64-element column blocks), completion on mbarriers.
//   warp 9      MMA issuer: S = Q K^T (both operands K-major in shared memory) into tensor memory,
//               O += P V with P read from tensor memory and V as an MN-major shared-memory operand.
//   warps 10-11 build the ancestor masks of the tree, then idle.
// Registers are moved from the third warpgroup to the two softmax warpgroups (setmaxnreg).
// Tensor memory (512 columns): O tile 0 | O tile 1 | S/P tile 0 | S/P tile 1, 128 columns each.
// The two row tiles are interleaved on the tensor pipe (S0 S1 | PV0 S0' PV1 S1' | ...) so that
// the softmax of one tile runs under the MMAs of the other.
//
// Every mbarrier wait is bounded; on expiry the CTA raises SPECEXT_ERR_TIMEOUT, drains its copies
// and MMAs (bounded again), frees tensor memory and returns.
#include "common.cuh"
#include "sm100.cuh"

using namespace sm100;

struct TcMaps {
  CUtensorMap q, kp, vp, kt, vt;
};

namespace {

constexpr int kThreads = 384;
constexpr int kProducerWarp = 8, kMmaWarp = 9;
// Register hand-over between warpgroups.  The kernel is compiled for 168 registers per thread
// (65536 / 384, rounded down to a multiple of 8); the third warpgroup shrinks to kRegsOther and
// the two softmax warpgroups grow to kRegsSoftmax.  setmaxnreg.inc blocks until the registers it
// asks for have been released inside the CTA's own allocation, so the release must cover the request.
constexpr int kRegsLaunch = 168, kRegsOther = 64, kRegsSoftmax = 216;
static_assert(128 * (kRegsLaunch - kRegsOther) >= 256 * (kRegsSoftmax - kRegsLaunch),
              "setmaxnreg.inc would wait for registers that are never released");
constexpr int kSubTileBytes = 128 * 128;        // 128 rows x 64 bf16
constexpr float kRescaleThreshold = 8.0f;       // log2 units

template <int D>
struct Cfg {
  static constexpr int DS = D / 64;                           // 64-element column blocks
  static constexpr int kStageBytes = DS * kSubTileBytes;      // one K or V tile
  static constexpr int kQBytes = 2 * DS * kSubTileBytes;      // two row tiles
  static constexpr int kStages = D == 128 ? 5 : 8;
  static constexpr int kBarOffset = kQBytes + kStages * kStageBytes;
  // Trees of more than 64 nodes need two mask words per node.  With head_dim 128 the rings leave only 1 KB
  // for the control block, and such a tree with at most 128 stacked rows (one query head per KV head) is sent
  // to the paired kernel by the plan; with head_dim 64 there is room for the full 128 nodes.
  static constexpr int kTreeMax = D == 128 ? 64 : kSpxMaxTree;
  static constexpr int kCtrlBytes = D == 128 ? 1024 : 3072;
  static constexpr int kSmemBytes = kBarOffset + kCtrlBytes + 1024; // + control block + alignment slack
};

template <int D>
struct CtrlT {
  uint64_t q_full, q_free, drain;
  uint64_t v_rag;                 // a V tile whose tail rows must be cleared has landed (device-side length)
  uint64_t s_full[2], p_full[2], o_done[2], o_free[2];
  uint64_t kv_full[8], kv_empty[8];
  unsigned long long anc[Cfg<D>::kTreeMax][Cfg<D>::kTreeMax / 64];
  int parent[Cfg<D>::kTreeMax];
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(CtrlT<128>) <= Cfg<128>::kCtrlBytes && sizeof(CtrlT<64>) <= Cfg<64>::kCtrlBytes,
              "control block too large");

// DEVLEN: the prefix length is read from device memory (a.L_dev) and may be shorter than the planned
// capacity p.L; the instantiation without it carries none of that code.
template <int D, bool SCORE, bool DEVLEN>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ AttnArgs a, const __grid_constant__ TcMaps maps) {
  using C = Cfg<D>;
  constexpr int DS = C::DS;
  constexpr int NS = C::kStages;
  const AttnPlan& p = a.plan;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                                         ~static_cast<uintptr_t>(1023));
  unsigned char* Qs = base;
  unsigned char* ring = base + C::kQBytes;
  using Ctrl = CtrlT<D>;
  constexpr int kTreeMax = C::kTreeMax;
  Ctrl* ctl = reinterpret_cast<Ctrl*>(base + C::kBarOffset);
  volatile int* abort_flag = &ctl->abort_flag;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_mt = p.RB / 128;
  const int cta = blockIdx.x;
  const int unit_lo = spx_unit_start(p, cta), unit_hi = spx_unit_start(p, cta + 1);

  if (warp == kProducerWarp && lane == 0) {
    mbar_init(&ctl->q_full, 1);
    mbar_init(&ctl->q_free, 1);
    mbar_init(&ctl->drain, 1);
    mbar_init(&ctl->v_rag, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&ctl->s_full[i], 1);
      mbar_init(&ctl->p_full[i], 128);
      mbar_init(&ctl->o_done[i], 1);
      mbar_init(&ctl->o_free[i], 128);
    }
    for (int i = 0; i < NS; ++i) {
      mbar_init(&ctl->kv_full[i], 1);
      mbar_init(&ctl->kv_empty[i], 1);
    }
    ctl->abort_flag = 0;
    fence_mbar_init();
    prefetch_tensormap(&maps.q);
    prefetch_tensormap(&maps.kp);
    prefetch_tensormap(&maps.vp);
    prefetch_tensormap(&maps.kt);
    prefetch_tensormap(&maps.vt);
  }
  __syncthreads();                       // barriers are initialised; the producer may start at once
  bool ok = true;

  if (warp == kProducerWarp) {
    // ================================ TMA producer ==========================================
    setmaxnreg_dec<kRegsOther>();
    if (lane == 0) {
      uint32_t kvp = 0, n_rag = 0;
      int seg = 0;
      bool q_armed = false;
      constexpr bool dev_len = DEVLEN;
      const int L_eff = DEVLEN ? spx_prefix_len(a) : p.L;
      const int tph_eff = DEVLEN ? (L_eff + SPX_TILE_KEYS - 1) / SPX_TILE_KEYS : p.TPH;
      for (int u = unit_lo; u < unit_hi && ok;) {
        const int prob = u / p.UPP;
        const int tile_lo = u - prob * p.UPP;
        const int n_units = min(p.UPP - tile_lo, unit_hi - u);
        SpxSeg sg;
        if (DEVLEN) {
          sg = spx_segment(p, tile_lo, n_units, tph_eff);
        } else {
          sg.n_pref = n_units;                 // (the tree tile, if any, is simply the last of the run)
          sg.has_tree = 0;
          sg.n = n_units;
        }
        u += n_units;
        if (DEVLEN && sg.n == 0) continue;     // nothing of this run exists at the device-side length
        const int g = prob / p.n_rblk, rblk = prob - g * p.n_rblk;
        if (seg > 0) ok = mbar_wait(&ctl->q_free, (seg - 1) & 1, abort_flag);
        if (!ok) break;
        mbar_arrive_expect_tx(&ctl->q_full, n_mt * DS * kSubTileBytes);
        q_armed = true;
        for (int mt = 0; mt < n_mt; ++mt)
          for (int ds = 0; ds < DS; ++ds)
            tma_load_3d(Qs + (mt * DS + ds) * kSubTileBytes, &maps.q, &ctl->q_full, ds * 64, g * p.G,
                        (rblk * n_mt + mt) * (128 / p.G));
        for (int j = 0; j < sg.n && ok; ++j) {
          const int tile = DEVLEN ? spx_seg_tile(p, sg, tile_lo, j) : tile_lo + j;
          const bool is_tree = tile == p.TPH;
          const int nk = is_tree ? SPX_TILE_KEYS : L_eff - tile * SPX_TILE_KEYS;
          for (int which = 0; which < 2; ++which) {
            const int stage = kvp % NS;
            ok = mbar_wait(&ctl->kv_empty[stage], ((kvp / NS) & 1) ^ 1, abort_flag);
            if (!ok) break;
            const CUtensorMap* m = is_tree ? (which ? &maps.vt : &maps.kt) : (which ? &maps.vp : &maps.kp);
            unsigned char* dst = ring + stage * C::kStageBytes;
            if (which == 1 && dev_len && nk < SPX_TILE_KEYS) {
              // Device-side length: the tensor map spans the whole capacity, so the rows of this V tile
              // past the length hold whatever the cache holds (their probabilities are zero, but zero
              // times a NaN is a NaN).  The tile lands on a barrier of its own, its tail rows are
              // cleared (a row of a 64-column block is 128 bytes whatever the swizzle), and only then
              // is the stage handed to the MMA issuer.
              mbar_arrive_expect_tx(&ctl->v_rag, C::kStageBytes);
              for (int ds = 0; ds < DS; ++ds)
                tma_load_3d(dst + ds * kSubTileBytes, m, &ctl->v_rag, ds * 64, g, tile * SPX_TILE_KEYS);
              ok = mbar_wait(&ctl->v_rag, n_rag & 1, abort_flag);
              if (!ok) break;
              ++n_rag;
              for (int ds = 0; ds < DS; ++ds) {
                uint4* tail = reinterpret_cast<uint4*>(dst + ds * kSubTileBytes + nk * 128);
                for (int i = 0; i < (SPX_TILE_KEYS - nk) * 8; ++i) tail[i] = make_uint4(0u, 0u, 0u, 0u);
              }
              asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
              mbar_arrive(&ctl->kv_full[stage]);
            } else {
              mbar_arrive_expect_tx(&ctl->kv_full[stage], C::kStageBytes);
              for (int ds = 0; ds < DS; ++ds)
                tma_load_3d(dst + ds * kSubTileBytes, m, &ctl->kv_full[stage], ds * 64, g,
                            is_tree ? 0 : tile * SPX_TILE_KEYS);
            }
            ++kvp;
          }
        }
        ++seg;
      }
      if (!ok) {
        // give the copies already issued a bounded chance to land before the CTA's memory is released
        const uint32_t lo = kvp > (uint32_t)NS ? kvp - NS : 0;
        for (uint32_t f = lo; f < kvp; ++f)
          for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(&ctl->kv_full[f % NS], (f / NS) & 1); ++spin) {}
        if (q_armed)
          for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(&ctl->q_full, (seg > 0 ? seg - 1 : 0) & 1); ++spin) {}
      }
    }
  } else {
    // tensor memory (MMA warp) and ancestor masks (warps 10, 11), then everybody but the producer meets
    if (warp == kMmaWarp) {
      tmem_alloc(&ctl->tmem_base, 512);
      tmem_relinquish();
    } else if (warp > kMmaWarp) {
      const int t64 = tid - (kMmaWarp + 1) * 32;                // 0..63
      for (int t = t64; t < kTreeMax; t += 64) ctl->parent[t] = t < p.T ? a.parent[t] : -1;
      named_bar_sync(2, 64);
      bool bad = false;
      for (int t = t64; t < kTreeMax; t += 64) {
        SpxMask128 m = {0ull, 0ull};
        if (t < p.T) m = spx_walk_up(ctl->parent, p.T, t, bad);
        ctl->anc[t][0] = m.lo;
        if (kTreeMax > 64) ctl->anc[t][kTreeMax / 64 - 1] = m.hi;
      }
      if (bad && cta == 0) spx_raise(a.status, SPECEXT_ERR_BAD_TREE);
    }
    tc_fence_before();
    named_bar_sync(1, kThreads - 32);
    tc_fence_after();
    const uint32_t tmem = ctl->tmem_base;

    if (warp == kMmaWarp) {
      // ================================ MMA issuer ==========================================
      setmaxnreg_dec<kRegsOther>();
      if (lane == 0) {
        const uint32_t idesc_s = idesc_bf16_f32(128, SPX_TILE_KEYS, false, false);
        const uint32_t idesc_o = idesc_bf16_f32(128, D, false, true);
        constexpr uint32_t hi = desc_hi(1024);
        const uint32_t q_lo = desc_lo(smem_u32(Qs), 16);
        const uint32_t k_lo0 = desc_lo(smem_u32(ring), 16);
        const uint32_t v_lo0 = desc_lo(smem_u32(ring), kSubTileBytes);
        uint32_t kvc = 0, it = 0;
        int seg = 0;

        auto issue_s = [&](int mt, int stage) {
          const uint32_t kb = k_lo0 + stage * (C::kStageBytes >> 4);
          const uint32_t qb = q_lo + mt * (DS * kSubTileBytes >> 4);
          const uint32_t d = tmem + 256 + mt * 128;
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = (kk >> 2) * (kSubTileBytes >> 4) + (kk & 3) * 2;
            mma_ss2(d, qb + off, hi, kb + off, hi, idesc_s, kk > 0 ? 1u : 0u);
          }
          mma_commit(&ctl->s_full[mt]);
        };
        auto issue_pv = [&](int mt, int stage, uint32_t accumulate) {
          const uint32_t vb = v_lo0 + stage * (C::kStageBytes >> 4);
          const uint32_t d = tmem + mt * 128;
          const uint32_t pa = tmem + 256 + mt * 128;
          mma_ts2(d, pa, vb, hi, idesc_o, accumulate);
#pragma unroll
          for (int kk = 1; kk < SPX_TILE_KEYS / 16; ++kk) mma_ts2(d, pa + kk * 8, vb + kk * 128, hi, idesc_o, 1u);
        };

        const int tph_eff = DEVLEN ? (spx_prefix_len(a) + SPX_TILE_KEYS - 1) / SPX_TILE_KEYS : p.TPH;
        for (int u = unit_lo; u < unit_hi && ok;) {
          const int prob = u / p.UPP;
          const int tile_lo = u - prob * p.UPP;
          const int n_units = min(p.UPP - tile_lo, unit_hi - u);
          const int n = DEVLEN ? spx_segment(p, tile_lo, n_units, tph_eff).n : n_units;
          u += n_units;
          if (DEVLEN && n == 0) continue;
          ok = mbar_wait(&ctl->q_full, seg & 1, abort_flag);
          if (!ok) break;
          {
            const int ks = kvc % NS;
            ok = mbar_wait(&ctl->kv_full[ks], (kvc / NS) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            for (int mt = 0; mt < n_mt; ++mt) issue_s(mt, ks);
            mma_commit(&ctl->kv_empty[ks]);
            ++kvc;
          }
          for (int i = 0; i < n && ok; ++i) {
            const bool has_next = i + 1 < n, last = !has_next;
            const int vs = kvc % NS;
            const uint32_t vph = (kvc / NS) & 1;
            ++kvc;
            const int ks = kvc % NS;
            const uint32_t kph = (kvc / NS) & 1;
            ok = mbar_wait(&ctl->kv_full[vs], vph, abort_flag);
            for (int mt = 0; mt < n_mt && ok; ++mt) {
              ok = mbar_wait(&ctl->p_full[mt], it & 1, abort_flag);
              if (ok && i == 0 && seg > 0) ok = mbar_wait(&ctl->o_free[mt], (seg - 1) & 1, abort_flag);
              if (!ok) break;
              tc_fence_after();
              issue_pv(mt, vs, i > 0 ? 1u : 0u);
              if (last) mma_commit(&ctl->o_done[mt]);
              if (mt == n_mt - 1) mma_commit(&ctl->kv_empty[vs]);
              if (has_next) {
                if (mt == 0) {
                  ok = mbar_wait(&ctl->kv_full[ks], kph, abort_flag);
                  if (!ok) break;
                  tc_fence_after();
                }
                issue_s(mt, ks);
                if (mt == n_mt - 1) mma_commit(&ctl->kv_empty[ks]);
              }
            }
            if (has_next) ++kvc;
            ++it;
          }
          if (ok) mma_commit(&ctl->q_free);
          ++seg;
        }
        // drain: all MMAs issued so far must have completed before tensor memory is released
        mma_commit(&ctl->drain);
        for (int spin = 0; spin < (1 << 22) && !mbar_try_wait(&ctl->drain, 0); ++spin) {}
      }
    } else if (warp > kMmaWarp) {
      setmaxnreg_dec<kRegsOther>();
    } else {
      // ================================ softmax warps =======================================
      setmaxnreg_inc<kRegsSoftmax>();
      const int mt = warp >> 2;
      if (mt < n_mt) {
        const int quarter = warp & 3;
        const int row_t = quarter * 32 + lane;
        const int rr = mt * 128 + row_t;
        const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
        const uint32_t s_addr = tmem + lane_addr + 256 + mt * 128;
        const uint32_t o_addr = tmem + lane_addr + mt * 128;
        const float scale2 = p.scale2;
        uint32_t it = 0;
        int seg = 0;
        const int L_eff = DEVLEN ? spx_prefix_len(a) : p.L;
        const int tph_eff = DEVLEN ? (L_eff + SPX_TILE_KEYS - 1) / SPX_TILE_KEYS : p.TPH;
        for (int u = unit_lo; u < unit_hi && ok;) {
          const int prob = u / p.UPP;
          const int tile_lo = u - prob * p.UPP;
          const int n_units = min(p.UPP - tile_lo, unit_hi - u);
          SpxSeg sg;
          if (DEVLEN) sg = spx_segment(p, tile_lo, n_units, tph_eff);
          const int n_seg = DEVLEN ? sg.n : n_units;
          const int g = prob / p.n_rblk, rblk = prob - g * p.n_rblk;
          const int r = rblk * p.RB + rr;
          const bool valid = r < p.rows;
          if (DEVLEN && n_seg == 0) {
            // No tile of this run exists at the device-side length: its slot gets the neutral partial
            // (weight zero in the merge), and no barrier of the pipeline is touched.
            const int slot = cta + prob;
            float* po = a.ws + p.off_part_o + (long long)slot * (D / 4) * p.RB * 4;
            for (int q4 = 0; q4 < D / 4; ++q4)
              *reinterpret_cast<float4*>(po + ((long long)q4 * p.RB + rr) * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
            a.ws[p.off_part_m + (long long)slot * p.RB + rr] = -1e30f;      // finite: see the merge
            a.ws[p.off_part_l + (long long)slot * p.RB + rr] = 0.f;
            u += n_units;
            continue;
          }
          const int t_node = valid ? r / p.G : 0;
          float m_used = -INFINITY, l = 0.f;

          for (int jt = 0; jt < n_seg; ++jt, ++it) {
            const int tile = DEVLEN ? spx_seg_tile(p, sg, tile_lo, jt) : tile_lo + jt;
            const bool is_tree = tile == p.TPH;
            const int nkeys = is_tree ? p.T : min(SPX_TILE_KEYS, (DEVLEN ? L_eff : p.L) - tile * SPX_TILE_KEYS);
            const bool need_mask = is_tree || nkeys < SPX_TILE_KEYS;
            ok = mbar_wait(&ctl->s_full[mt], it & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();

            // the whole S row of this thread: 128 fp32 scores in registers
            uint32_t s0[32], s1[32], s2[32], s3[32];
            tmem_ld32(s_addr, s0);
            tmem_ld32(s_addr + 32, s1);
            tmem_ld32(s_addr + 64, s2);
            tmem_ld32(s_addr + 96, s3);
            tmem_wait_ld();
            if (need_mask) {
              unsigned long long vis_lo, vis_hi;
              if (is_tree) {               // this node and its ancestors (a padding row sees key 0)
                vis_lo = valid ? ctl->anc[t_node][0] : 1ull;
                vis_hi = (kTreeMax > 64 && valid) ? ctl->anc[t_node][kTreeMax / 64 - 1] : 0ull;
              } else {
                vis_lo = nkeys >= 64 ? ~0ull : ((1ull << nkeys) - 1ull);
                vis_hi = nkeys <= 64 ? 0ull : ((1ull << (nkeys - 64)) - 1ull);
              }
              const uint32_t b0 = static_cast<uint32_t>(vis_lo), b1 = static_cast<uint32_t>(vis_lo >> 32);
              const uint32_t b2 = static_cast<uint32_t>(vis_hi), b3 = static_cast<uint32_t>(vis_hi >> 32);
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                if (!((b0 >> j) & 1u)) s0[j] = 0xff800000u;    // -inf
                if (!((b1 >> j) & 1u)) s1[j] = 0xff800000u;
                if (!((b2 >> j) & 1u)) s2[j] = 0xff800000u;
                if (!((b3 >> j) & 1u)) s3[j] = 0xff800000u;
              }
            }
            float t0 = -INFINITY, t1 = -INFINITY, t2 = -INFINITY, t3 = -INFINITY;
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
              t0 = fmax3(t0, __uint_as_float(s0[j]), __uint_as_float(s0[j + 1]));
              t1 = fmax3(t1, __uint_as_float(s1[j]), __uint_as_float(s1[j + 1]));
              t2 = fmax3(t2, __uint_as_float(s2[j]), __uint_as_float(s2[j + 1]));
              t3 = fmax3(t3, __uint_as_float(s3[j]), __uint_as_float(s3[j + 1]));
            }
            const float tmax = fmaxf(fmaxf(t0, t1), fmaxf(t2, t3));
            const float m_tile = tmax * scale2;
            float alpha = 1.f;
            bool rescale = false;
            if (m_tile > m_used + kRescaleThreshold || m_used == -INFINITY) {
              alpha = (m_used == -INFINITY) ? 0.f : ex2_approx(m_used - m_tile);
              rescale = jt > 0;
              m_used = m_tile;
              l *= alpha;
            }
            if (__any_sync(0xffffffffu, rescale)) {
              // S(tile) has been committed after PV(tile-1), so O is complete and not being written
#pragma unroll
              for (int c = 0; c < D / 32; ++c) {
                uint32_t v[32];
                tmem_ld32(o_addr + c * 32, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * alpha);
                tmem_st32(o_addr + c * 32, v);
              }
            }

            // exponentials against the reference maximum, sums, P in bf16 back to tensor memory
            const float neg_m = -m_used;
            const bool score = SCORE && !is_tree;
            float* mass = nullptr;
            if (score) {
              const long long rowbase = ((long long)prob * p.TPH + tile) * p.RB + rr;
              mass = a.ws + p.off_mass + rowbase * p.CPT;
              a.ws[p.off_mref + rowbase] = m_used;
            }
            float csum = 0.f;
            auto exp_chunk = [&](uint32_t (&v)[32], int c) {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                v[j] = __float_as_uint(ex2_approx(fmaf(__uint_as_float(v[j]), scale2, neg_m)));
              float gs0 = 0.f, gs1 = 0.f, gs2 = 0.f, gs3 = 0.f;
#pragma unroll
              for (int j = 0; j < 32; j += 4) {
                gs0 += __uint_as_float(v[j]);
                gs1 += __uint_as_float(v[j + 1]);
                gs2 += __uint_as_float(v[j + 2]);
                gs3 += __uint_as_float(v[j + 3]);
              }
              const float gs = (gs0 + gs1) + (gs2 + gs3);
              l += gs;
              if (score) {
                if (p.C >= 32) {
                  csum += gs;
                  if ((((c + 1) * 32) & (p.C - 1)) == 0) {
                    mass[((c + 1) * 32) / p.C - 1] = csum;
                    csum = 0.f;
                  }
                } else {
                  float acc = 0.f;
#pragma unroll
                  for (int j = 0; j < 32; ++j) {
                    acc += __uint_as_float(v[j]);
                    if (((j + 1) & (p.C - 1)) == 0) {
                      mass[(c * 32 + j) / p.C] = acc;
                      acc = 0.f;
                    }
                  }
                }
              }
              uint32_t pk[16];
#pragma unroll
              for (int j = 0; j < 16; ++j) pk[j] = pack_bf16x2(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
              tmem_st16(s_addr + c * 16, pk);
            };
            exp_chunk(s0, 0);
            exp_chunk(s1, 1);
            exp_chunk(s2, 2);
            exp_chunk(s3, 3);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&ctl->p_full[mt]);
          }
          if (!ok) break;

          // epilogue of the segment: unnormalised O, reference maximum and row sum to the partial slot
          ok = mbar_wait(&ctl->o_done[mt], seg & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          {
            const int slot = cta + prob;
            float* po = a.ws + p.off_part_o + (long long)slot * (D / 4) * p.RB * 4;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
              uint32_t v[32];
              tmem_ld32(o_addr + c * 32, v);
              tmem_wait_ld();
#pragma unroll
              for (int q4 = 0; q4 < 8; ++q4) {
                const float4 x = make_float4(__uint_as_float(v[q4 * 4]), __uint_as_float(v[q4 * 4 + 1]),
                                             __uint_as_float(v[q4 * 4 + 2]), __uint_as_float(v[q4 * 4 + 3]));
                *reinterpret_cast<float4*>(po + ((long long)(c * 8 + q4) * p.RB + rr) * 4) = x;
              }
            }
            a.ws[p.off_part_m + (long long)slot * p.RB + rr] = m_used;
            a.ws[p.off_part_l + (long long)slot * p.RB + rr] = l;
          }
          tc_fence_before();
          mbar_arrive(&ctl->o_free[mt]);
          u += n_units;
          ++seg;
        }
      }
    }
  }

  if (!ok && lane == 0) spx_raise(a.status, SPECEXT_ERR_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    tmem_dealloc(ctl->tmem_base, 512);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// bf16 tensor [n2][n1][D] with element strides (s2, s1, 1); box = 64 x b1 x b2, 128-byte swizzle,
// out-of-range elements read as zero.
bool encode_map(CUtensorMap* m, const void* ptr, int D, long long n1, long long s1, long long n2, long long s2,
                int b1, int b2) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)n1, (cuuint64_t)n2};
  const cuuint64_t strides[2] = {(cuuint64_t)s1 * 2, (cuuint64_t)s2 * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)b1, (cuuint32_t)b2};
  const cuuint32_t es[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, bool SCORE, bool DEVLEN>
cudaError_t launch(const AttnArgs& a, const TcMaps& maps, cudaStream_t st) {
  static SpxOncePerDevice once;
  const cudaError_t ec = spx_opt_in_smem(attn_tc_kernel<D, SCORE, DEVLEN>, Cfg<D>::kSmemBytes, &once);
  if (ec != cudaSuccess) return ec;
  attn_tc_kernel<D, SCORE, DEVLEN><<<a.plan.n_cta, kThreads, Cfg<D>::kSmemBytes, st>>>(a, maps);
  return cudaGetLastError();
}

}  // namespace

cudaError_t spx_launch_attn_tc(const AttnArgs& a, cudaStream_t st, int* n_launches) {
  const AttnPlan& p = a.plan;
  TcMaps maps;
  const int tok_per_tile = 128 / p.G;
  bool ok = encode_map(&maps.q, a.Q, p.D, p.Hq, a.q_sh, p.T, a.q_st, p.G, tok_per_tile);
  ok = ok && encode_map(&maps.kt, a.Kt, p.D, p.Hkv, a.tkv_sh, p.T, a.tkv_st, 1, SPX_TILE_KEYS);
  ok = ok && encode_map(&maps.vt, a.Vt, p.D, p.Hkv, a.tkv_sh, p.T, a.tkv_st, 1, SPX_TILE_KEYS);
  if (p.L > 0) {
    ok = ok && encode_map(&maps.kp, a.Kp, p.D, p.Hkv, a.kv_sh, p.L, a.kv_sl, 1, SPX_TILE_KEYS);
    ok = ok && encode_map(&maps.vp, a.Vp, p.D, p.Hkv, a.kv_sh, p.L, a.kv_sl, 1, SPX_TILE_KEYS);
  } else {
    maps.kp = maps.kt;
    maps.vp = maps.vt;
  }
  if (!ok) return cudaErrorInvalidValue;
  cudaError_t e;
  if (a.L_dev)                                  // never with chunk sums
    e = p.D == 128 ? launch<128, false, true>(a, maps, st) : launch<64, false, true>(a, maps, st);
  else if (p.D == 128)
    e = p.want_score ? launch<128, true, false>(a, maps, st) : launch<128, false, false>(a, maps, st);
  else
    e = p.want_score ? launch<64, true, false>(a, maps, st) : launch<64, false, false>(a, maps, st);
  *n_launches += 1;
  return e;
}
