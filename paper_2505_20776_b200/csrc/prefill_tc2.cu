// Prefill (causal self-attention of the prompt) on pairs of SMs: the inner loop of the paired Hybrid
// Tree Attention kernel (attn_tc2.cu) with whole problems instead of key splits.
//
// A problem is one KV head and one block of tb = 256 / G consecutive prompt tokens: the block's
// G * tb = 256 stacked query rows (row = token * G + head in group) attend to the keys 0 .. end of the
// block.  Keys are taken in 128-key tiles aligned at multiples of 128; the tiles that end at or before
// the block's first token are fully visible, the last one or two ("diagonal") tiles are masked per row
// (key j is visible to token i iff j <= i).  A problem is processed from its first to its last tile by
// one cluster, so its result is final: O = sum / row sum and lse are written by the kernel itself; there
// are no partial results and no merge.  Problems are dealt to the clusters longest first, in
// boustrophedon order, which balances the triangular work to within one problem.
//
// Roles, tensor-memory layout, rings and barriers are those of attn_tc2.cu (see there): warps 0-3 and
// 4-7 are the two softmax warpgroups that alternate key tiles of the same 128 rows, warp 8 the TMA
// producer, warps 9 and 10 (leader CTA) the issuers of S = Q K^T and O += P V.  Every wait is bounded.
#include "common.cuh"
#include "pair.cuh"

using namespace sm100;
using namespace pair;

namespace {

constexpr int kThreads = 384;
constexpr int kProducerWarp = 8, kMmaWarp = 9, kPvWarp = 10;
constexpr int kRegsLaunch = 168, kRegsOther = 64, kRegsSoftmax = 216;
static_assert(128 * (kRegsLaunch - kRegsOther) >= 256 * (kRegsSoftmax - kRegsLaunch),
              "setmaxnreg.inc would wait for registers that are never released");
constexpr int D = 128;
constexpr int kStageBytes = 16384;             // half of a K tile (64 keys x 128) or of a V tile (128 keys x 64)
constexpr int kStages = 6;
constexpr int kCtrlOffset = 2 * kStages * kStageBytes;
constexpr int kSmemBytes = kCtrlOffset + 3072 + 1024;
constexpr float kRescaleThreshold = 8.0f;      // log2 units
constexpr uint32_t kColO = 0, kColS = 128, kColQ = 384, kColP = 448;
constexpr float kLn2 = 0.693147180559945309417f;

struct PrefillArgs {
  const __nv_bfloat16* Q;
  __nv_bfloat16* O;
  float* lse;
  int32_t* status;
  long long q_st, q_sh, o_st, o_sh;
  int L, Hq, Hkv, G;
  int tb;          // tokens per block = 256 / G
  int nb;          // blocks = ceil(L / tb)
  int n_prob;      // nb * Hkv
  int W;           // clusters
  float scale2;    // softmax_scale * log2(e)
};

struct PrefillMaps {
  CUtensorMap k, v;      // [L][Hkv][128], boxes 64 x 1 x 64 (K halves) and 64 x 1 x 128 (V halves)
};

struct Ctrl {
  uint64_t k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
  uint64_t q_ready;             // leader: 16 arrivals (every softmax warp of both CTAs)
  uint64_t s_full[2], s_free[2];
  uint64_t p_full;
  uint64_t pv_done[2];
  uint64_t o_done;
  uint64_t m_pub[2];
  uint64_t drain;
  uint64_t epi[2];
  float m_row[128];
  float l_x[2][128];            // epilogue: each warpgroup's row sums, for the other one
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(Ctrl) <= 3072, "control block too large");

// Problem number `rnd` of cluster `cl`: problems are numbered longest first and dealt out back and forth.
__device__ __forceinline__ bool problem_of(const PrefillArgs& a, int cl, int rnd, int& b, int& g, int& n_tiles) {
  const int pos = rnd * a.W + ((rnd & 1) ? a.W - 1 - cl : cl);
  if (pos >= a.n_prob) return false;
  b = a.nb - 1 - pos / a.Hkv;
  g = pos % a.Hkv;
  n_tiles = ((b + 1) * a.tb + SPX_TILE_KEYS - 1) / SPX_TILE_KEYS;
  const int all = (a.L + SPX_TILE_KEYS - 1) / SPX_TILE_KEYS;          // the last block may be short
  if (n_tiles > all) n_tiles = all;
  return true;
}

__global__ void __launch_bounds__(kThreads, 1)
prefill_tc2_kernel(const __grid_constant__ PrefillArgs a, const __grid_constant__ PrefillMaps maps) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                                         ~static_cast<uintptr_t>(1023));
  unsigned char* ring = base;
  Ctrl* ctl = reinterpret_cast<Ctrl*>(base + kCtrlOffset);
  volatile int* abort_flag = &ctl->abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (warp == kProducerWarp) {
    if (lane < kStages) {
      mbar_init(&ctl->k_full[lane], 2);
      mbar_init(&ctl->k_empty[lane], 1);
      mbar_init(&ctl->v_full[lane], 2);
      mbar_init(&ctl->v_empty[lane], 1);
    } else if (lane < kStages + 2) {
      const int i = lane - kStages;
      mbar_init(&ctl->s_full[i], 1);
      mbar_init(&ctl->s_free[i], 8);
      mbar_init(&ctl->pv_done[i], 1);
      mbar_init(&ctl->m_pub[i], 4);
      mbar_init(&ctl->epi[i], 8);
    } else if (lane == kStages + 2) {
      mbar_init(&ctl->q_ready, 16);
      mbar_init(&ctl->p_full, 8);
      mbar_init(&ctl->o_done, 1);
      mbar_init(&ctl->drain, 2);
      ctl->abort_flag = 0;
    }
    fence_mbar_init();
  }
  cluster_arrive();
  pdl_launch_dependents();
  if (warp != kMmaWarp) pdl_wait();

  const uint32_t rank = cluster_rank();
  const int cl = blockIdx.x >> 1;
  const int n_rounds = (a.n_prob + a.W - 1) / a.W;

  if (warp == kProducerWarp && lane == 0) {
    prefetch_tensormap(&maps.k);
    prefetch_tensormap(&maps.v);
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    pdl_wait();
  }
  bool ok = true;

  if (warp == kProducerWarp) {
    // ================================ TMA producer (each CTA loads its halves) ===============
    setmaxnreg_dec<kRegsOther>();
    cluster_wait();
    if (lane == 0) {
      uint32_t kp = 0, vp = 0;
      const uint32_t kfull0 = map_to_cta(smem_u32(&ctl->k_full[0]), 0);
      const uint32_t vfull0 = map_to_cta(smem_u32(&ctl->v_full[0]), 0);
      for (int rnd = 0; rnd < n_rounds && ok; ++rnd) {
        int b, g, n;
        if (!problem_of(a, cl, rnd, b, g, n)) continue;
        for (int tile = 0; tile < n && ok; ++tile) {
          {
            const int stage = kp % kStages;
            ok = wait_c(&ctl->k_empty[stage], ((kp / kStages) & 1) ^ 1, abort_flag);
            if (!ok) break;
            const uint32_t bar = kfull0 + stage * 8;
            const uint32_t dst = smem_u32(ring + stage * kStageBytes);
            const int key0 = tile * SPX_TILE_KEYS + 64 * rank;
            arrive_expect_tx_cluster(bar, kStageBytes);
            tma_load_3d_pair(dst, &maps.k, bar, 0, g, key0);
            tma_load_3d_pair(dst + 8192, &maps.k, bar, 64, g, key0);
            ++kp;
          }
          {
            const int stage = vp % kStages;
            ok = wait_c(&ctl->v_empty[stage], ((vp / kStages) & 1) ^ 1, abort_flag);
            if (!ok) break;
            const uint32_t bar = vfull0 + stage * 8;
            arrive_expect_tx_cluster(bar, kStageBytes);
            tma_load_3d_pair(smem_u32(ring + (kStages + stage) * kStageBytes), &maps.v, bar, 64 * rank, g,
                             tile * SPX_TILE_KEYS);
            ++vp;
          }
        }
      }
    }
  } else {
    if (warp == 11) setmaxnreg_dec<kRegsOther>();        // registers first: the softmax warpgroups wait for them
    tc_fence_before();
    if (warp != 11) named_bar_sync(1, kThreads - 64);    // the tensor-memory base address is visible
    cluster_wait();                                      // both CTAs' barriers exist
    tc_fence_after();
    const uint32_t tmem = ctl->tmem_base;

    if (warp == kMmaWarp) {
      // ================================ issuer of S = Q K^T (leader CTA) =====================
      setmaxnreg_dec<kRegsOther>();
      if (lane == 0 && rank == 0) {
        const uint32_t idesc_s = idesc_bf16_f32(256, SPX_TILE_KEYS, false, false);
        constexpr uint32_t hi = desc_hi(1024);
        const uint32_t ring_lo = desc_lo(smem_u32(ring), 16);
        uint32_t kc = 0, n_w[2] = {0, 0};
        int seg = 0;
        for (int rnd = 0; rnd < n_rounds && ok; ++rnd) {
          int b, g, n;
          if (!problem_of(a, cl, rnd, b, g, n)) continue;
          ok = wait_c(&ctl->q_ready, seg & 1, abort_flag);
          for (int j = 0; j < n && ok; ++j) {
            const int w = j & 1;
            if (n_w[w] > 0) ok = wait_c(&ctl->s_free[w], (n_w[w] - 1) & 1, abort_flag);
            const int stage = kc % kStages;
            if (ok) ok = wait_c(&ctl->k_full[stage], (kc / kStages) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t kb = ring_lo + stage * (kStageBytes >> 4);
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk)
              mma_ts_pair(tmem + kColS + w * 128, tmem + kColQ + kk * 8, kb + (kk >> 2) * 512 + (kk & 3) * 2, hi,
                          idesc_s, kk > 0 ? 1u : 0u);
            commit_pair(&ctl->s_full[w]);
            commit_pair(&ctl->k_empty[stage]);
            ++kc;
            ++n_w[w];
          }
          ++seg;
        }
        commit_pair(&ctl->drain);
      }
    } else if (warp == kPvWarp) {
      // ================================ issuer of O += P V (leader CTA) ======================
      setmaxnreg_dec<kRegsOther>();
      if (lane == 0 && rank == 0) {
        const uint32_t idesc_o = idesc_bf16_f32(256, D, false, true);
        constexpr uint32_t hi = desc_hi(1024);
        const uint32_t ring_lo = desc_lo(smem_u32(ring + kStages * kStageBytes), 16);
        uint32_t vc = 0;
        int seg = 0;
        for (int rnd = 0; rnd < n_rounds && ok; ++rnd) {
          int b, g, n;
          if (!problem_of(a, cl, rnd, b, g, n)) continue;
          ok = wait_c(&ctl->q_ready, seg & 1, abort_flag);       // every thread is done reading the previous O
          for (int j = 0; j < n && ok; ++j) {
            const int w = j & 1;
            const int stage = vc % kStages;
            ok = wait_c(&ctl->v_full[stage], (vc / kStages) & 1, abort_flag);
            if (ok) ok = wait_c(&ctl->p_full, vc & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t vb = ring_lo + stage * (kStageBytes >> 4);
            const uint32_t pa = tmem + kColP;
            mma_ts_pair(tmem + kColO, pa, vb, hi, idesc_o, j > 0 ? 1u : 0u);
#pragma unroll
            for (int kk = 1; kk < SPX_TILE_KEYS / 16; ++kk)
              mma_ts_pair(tmem + kColO, pa + kk * 8, vb + kk * 128, hi, idesc_o, 1u);
            commit_pair(&ctl->v_empty[stage]);
            commit_pair(&ctl->pv_done[w]);
            if (j == n - 1) commit_pair(&ctl->o_done);
            ++vc;
          }
          ++seg;
        }
        commit_pair(&ctl->drain);
        for (int spin = 0; spin < (1 << 22) && !mbar_test_wait(&ctl->drain, 0); ++spin) {}
      }
    } else if (warp == 11) {
      // nothing to do
    } else {
      // ================================ softmax warps =======================================
      setmaxnreg_inc<kRegsSoftmax>();
      const int wg = warp >> 2;                          // 0: even tiles, 1: odd tiles
      const int quarter = warp & 3;
      const int row_t = quarter * 32 + lane;             // row inside this CTA's 128-row tile
      const int rr = rank * 128 + row_t;                 // row inside the 256-row block
      const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
      const uint32_t s_addr = tmem + lane_addr + kColS + wg * 128;
      const uint32_t p_addr = tmem + lane_addr + kColP;
      const uint32_t o_addr = tmem + lane_addr + kColO;
      const uint32_t q_ready_l = map_to_cta(smem_u32(&ctl->q_ready), 0);
      const uint32_t p_full_l = map_to_cta(smem_u32(&ctl->p_full), 0);
      const uint32_t s_free_l = map_to_cta(smem_u32(&ctl->s_free[wg]), 0);
      const float scale2 = a.scale2;
      uint32_t n_mine = 0, n_other = 0, n_oth = 0;
      int seg = 0;
      for (int rnd = 0; rnd < n_rounds && ok; ++rnd) {
        int b, g, n;
        if (!problem_of(a, cl, rnd, b, g, n)) continue;
        const int tok = b * a.tb + rr / a.G;             // this row's token
        const bool valid = tok < a.L;
        const int head = g * a.G + rr % a.G;
        const int tok_eff = valid ? tok : a.L - 1;       // a padding row repeats the last token; it is not stored
        const int block_lo = b * a.tb;                   // tiles that end at or before this key are fully visible
        // Q row of this thread -> tensor memory (warpgroup 0: first 64 elements, warpgroup 1: the rest)
        {
          uint32_t qv[32];
          if (valid) {
            const uint4* qp = reinterpret_cast<const uint4*>(a.Q + (long long)tok * a.q_st + (long long)head * a.q_sh +
                                                             wg * 64);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const uint4 x = __ldg(qp + j);
              qv[j * 4] = x.x; qv[j * 4 + 1] = x.y; qv[j * 4 + 2] = x.z; qv[j * 4 + 3] = x.w;
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) qv[j] = 0u;
          }
          tmem_st32(tmem + lane_addr + kColQ + wg * 32, qv);
          tmem_wait_st();
          tc_fence_before();
          warp_arrive_cluster(q_ready_l, lane);
        }

        float m_loc = -INFINITY, l = 0.f;        // l is relative to m_loc
        for (int j = wg; j < n && ok; j += 2) {
          const int key_lo = j * SPX_TILE_KEYS;
          const bool need_mask = key_lo + SPX_TILE_KEYS > block_lo;      // a diagonal tile
          ok = wait_c(&ctl->s_full[wg], n_mine & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          uint32_t s0[32], s1[32], s2[32], s3[32];
          tmem_ld32(s_addr, s0);
          tmem_ld32(s_addr + 32, s1);
          tmem_ld32(s_addr + 64, s2);
          tmem_ld32(s_addr + 96, s3);
          // the row's reference maximum after the previous tile is fetched while the scores are on their way
          float m_cur = -INFINITY;
          if (j > 0) {
            ok = mbar_wait(&ctl->m_pub[wg ^ 1], n_other & 1, abort_flag);
            if (!ok) break;
            ++n_other;
            m_cur = ctl->m_row[row_t];
          }
          tmem_wait_ld();
          tc_fence_before();
          warp_arrive_cluster(s_free_l, lane);
          if (need_mask) {
            // keys key_lo .. key_lo + nvis - 1 are visible to this row (none when the tile lies past its token)
            int nvis = tok_eff - key_lo + 1;
            nvis = nvis < 0 ? 0 : (nvis > SPX_TILE_KEYS ? SPX_TILE_KEYS : nvis);
            const unsigned long long vis_lo = nvis >= 64 ? ~0ull : ((1ull << nvis) - 1ull);
            const unsigned long long vis_hi = nvis <= 64 ? 0ull : (nvis >= 128 ? ~0ull : ((1ull << (nvis - 64)) - 1ull));
            const uint32_t b0 = static_cast<uint32_t>(vis_lo), b1 = static_cast<uint32_t>(vis_lo >> 32);
            const uint32_t b2 = static_cast<uint32_t>(vis_hi), b3 = static_cast<uint32_t>(vis_hi >> 32);
#pragma unroll
            for (int k = 0; k < 32; ++k) {
              if (!((b0 >> k) & 1u)) s0[k] = 0xff800000u;    // -inf
              if (!((b1 >> k) & 1u)) s1[k] = 0xff800000u;
              if (!((b2 >> k) & 1u)) s2[k] = 0xff800000u;
              if (!((b3 >> k) & 1u)) s3[k] = 0xff800000u;
            }
          }
          float t0 = -INFINITY, t1 = -INFINITY, t2 = -INFINITY, t3 = -INFINITY;
#pragma unroll
          for (int k = 0; k < 32; k += 2) {
            t0 = fmax3(t0, __uint_as_float(s0[k]), __uint_as_float(s0[k + 1]));
            t1 = fmax3(t1, __uint_as_float(s1[k]), __uint_as_float(s1[k + 1]));
            t2 = fmax3(t2, __uint_as_float(s2[k]), __uint_as_float(s2[k + 1]));
            t3 = fmax3(t3, __uint_as_float(s3[k]), __uint_as_float(s3[k + 1]));
          }
          const float m_tile = fmaxf(fmaxf(t0, t1), fmaxf(t2, t3)) * scale2;     // -inf when the row sees nothing here

          float m_new = m_cur;
          bool rescale = false;
          if (m_tile > m_cur + kRescaleThreshold || m_cur == -INFINITY) {
            m_new = m_tile;                      // (tile 0 always shows key 0, so m_new is finite from the start)
            rescale = j > 0;
          }
          ctl->m_row[row_t] = m_new;
          warp_arrive(&ctl->m_pub[wg], lane);
          if (m_loc != m_new) {
            l *= (m_loc == -INFINITY) ? 0.f : ex2_approx(m_loc - m_new);
            m_loc = m_new;
          }
          const uint32_t n_prev_other = n_oth + ((j + 1) >> 1);
          bool pv_seen = false;
          auto wait_prev_pv = [&]() -> bool {
            if (pv_seen) return true;
            pv_seen = true;
            // (one parity test suffices: the other warpgroup's barrier is either one completion short of the
            // one asked for or at it, and the PVs complete in order)
            if (n_prev_other > 0 && !wait_c(&ctl->pv_done[wg ^ 1], (n_prev_other - 1) & 1, abort_flag)) return false;
            tc_fence_after();
            return true;
          };
          if (__any_sync(0xffffffffu, rescale)) {
            ok = wait_prev_pv();
            if (!ok) break;
            const float alpha = rescale ? ex2_approx(m_cur - m_new) : 1.f;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
              uint32_t v[32];
              tmem_ld32(o_addr + c * 32, v);
              tmem_wait_ld();
#pragma unroll
              for (int k = 0; k < 32; ++k) v[k] = __float_as_uint(__uint_as_float(v[k]) * alpha);
              tmem_st32(o_addr + c * 32, v);
            }
          }

          const float neg_m = -m_new;
          const uint64_t scale2x2 = pack_f32x2(scale2, scale2), neg_mx2 = pack_f32x2(neg_m, neg_m);
          uint32_t pk0[16], pk1[16], pk2[16], pk3[16];
          auto exp_chunk = [&](uint32_t (&v)[32], uint32_t (&pk)[16]) {
            uint64_t acc01 = 0ull, acc23 = 0ull;
#pragma unroll
            for (int k = 0; k < 32; k += 4) {
              float e0, e1, e2, e3;
              unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(v[k]), __uint_as_float(v[k + 1])), scale2x2, neg_mx2), e0, e1);
              unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(v[k + 2]), __uint_as_float(v[k + 3])), scale2x2, neg_mx2), e2, e3);
              e0 = ex2_approx(e0);
              e1 = ex2_approx(e1);
              e2 = ex2_approx(e2);
              e3 = ex2_approx(e3);
              acc01 = add_f32x2(acc01, pack_f32x2(e0, e1));
              acc23 = add_f32x2(acc23, pack_f32x2(e2, e3));
              v[k] = __float_as_uint(e0);
              v[k + 1] = __float_as_uint(e1);
              v[k + 2] = __float_as_uint(e2);
              v[k + 3] = __float_as_uint(e3);
            }
            float gs0, gs1, gs2, gs3;
            unpack_f32x2(acc01, gs0, gs1);
            unpack_f32x2(acc23, gs2, gs3);
            l += (gs0 + gs1) + (gs2 + gs3);
#pragma unroll
            for (int k = 0; k < 16; ++k) pk[k] = pack_bf16x2(__uint_as_float(v[2 * k]), __uint_as_float(v[2 * k + 1]));
          };
          exp_chunk(s0, pk0);
          exp_chunk(s1, pk1);
          exp_chunk(s2, pk2);
          exp_chunk(s3, pk3);
          ok = wait_prev_pv();
          if (!ok) break;
          tmem_st16(p_addr, pk0);
          tmem_st16(p_addr + 16, pk1);
          tmem_st16(p_addr + 32, pk2);
          tmem_st16(p_addr + 48, pk3);
          tmem_wait_st();
          tc_fence_before();
          warp_arrive_cluster(p_full_l, lane);
          ++n_mine;
        }
        if (!ok) break;

        // ---- epilogue of the problem: the result is final ------------------------------------
        if (((n - 1) & 1) != wg) {
          ok = mbar_wait(&ctl->m_pub[wg ^ 1], n_other & 1, abort_flag);
          if (!ok) break;
          ++n_other;
        }
        const float m_fin = ctl->m_row[row_t];
        if (m_loc != m_fin) l *= (m_loc == -INFINITY) ? 0.f : ex2_approx(m_loc - m_fin);
        ctl->l_x[wg][row_t] = l;
        ok = wait_c(&ctl->o_done, seg & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        n_oth += wg == 0 ? (n >> 1) : ((n + 1) >> 1);
        warp_arrive(&ctl->epi[0], lane);                 // both warpgroups' row sums are visible
        ok = mbar_wait(&ctl->epi[0], seg & 1, abort_flag);
        if (!ok) break;
        {
          const float l_tot = l + ctl->l_x[wg ^ 1][row_t];
          const float inv = 1.f / l_tot;
          __nv_bfloat16* out = a.O + (long long)tok * a.o_st + (long long)head * a.o_sh + wg * 64;
#pragma unroll
          for (int c = 0; c < 2; ++c) {                  // this warpgroup's 64 of the 128 columns
            uint32_t v[32];
            tmem_ld32(o_addr + wg * 64 + c * 32, v);
            tmem_wait_ld();
            if (valid) {
#pragma unroll
              for (int q8 = 0; q8 < 4; ++q8) {
                uint4 x;
                x.x = pack_bf16x2(__uint_as_float(v[q8 * 8]) * inv, __uint_as_float(v[q8 * 8 + 1]) * inv);
                x.y = pack_bf16x2(__uint_as_float(v[q8 * 8 + 2]) * inv, __uint_as_float(v[q8 * 8 + 3]) * inv);
                x.z = pack_bf16x2(__uint_as_float(v[q8 * 8 + 4]) * inv, __uint_as_float(v[q8 * 8 + 5]) * inv);
                x.w = pack_bf16x2(__uint_as_float(v[q8 * 8 + 6]) * inv, __uint_as_float(v[q8 * 8 + 7]) * inv);
                *reinterpret_cast<uint4*>(out + c * 32 + q8 * 8) = x;
              }
            }
          }
          if (wg == 0 && valid) a.lse[(long long)head * a.L + tok] = (m_fin + log2f(l_tot)) * kLn2;
        }
        warp_arrive(&ctl->epi[1], lane);                 // l_x and m_row may be reused
        ok = mbar_wait(&ctl->epi[1], seg & 1, abort_flag);
        ++seg;
      }
    }
  }

  if (!ok && lane == 0) spx_raise(a.status, SPECEXT_ERR_TIMEOUT);
  tc_fence_before();
  cluster_sync_relaxed();
  if (warp == kMmaWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(ctl->tmem_base), "r"(512u) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 tensor [L][Hkv][128] with element strides (s_l, s_h, 1); box = 64 x 1 x keys, 128-byte swizzle,
// out-of-range elements read as zero.
bool encode_kv(CUtensorMap* m, const void* ptr, long long Hkv, long long s_h, long long L, long long s_l, int keys) {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr_fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr_fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr_fn);
  }
  if (!fn) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)Hkv, (cuuint64_t)L};
  const cuuint64_t strides[2] = {(cuuint64_t)s_h * 2, (cuuint64_t)s_l * 2};
  const cuuint32_t box[3] = {64, 1, (cuuint32_t)keys};
  const cuuint32_t es[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// Causal self-attention of L prompt tokens; head_dim 128 and G = Hq / Hkv a power of two <= 256.
cudaError_t spx_launch_prefill_tc2(const void* Q, const void* K, const void* V, void* O, float* lse, int L, int Hq,
                                   int Hkv, float scale2, long long q_st, long long q_sh, long long kv_sl,
                                   long long kv_sh, long long o_st, long long o_sh, int n_sm, int32_t* status,
                                   cudaStream_t st) {
  PrefillArgs a;
  a.Q = static_cast<const __nv_bfloat16*>(Q);
  a.O = static_cast<__nv_bfloat16*>(O);
  a.lse = lse;
  a.status = status;
  a.q_st = q_st; a.q_sh = q_sh; a.o_st = o_st; a.o_sh = o_sh;
  a.L = L; a.Hq = Hq; a.Hkv = Hkv; a.G = Hq / Hkv;
  a.tb = 256 / a.G;
  a.nb = (L + a.tb - 1) / a.tb;
  a.n_prob = a.nb * Hkv;
  int W = n_sm / 2;
  if (W > a.n_prob) W = a.n_prob;
  if (W < 1) W = 1;
  a.W = W;
  a.scale2 = scale2;
  PrefillMaps maps;
  if (!encode_kv(&maps.k, K, Hkv, kv_sh, L, kv_sl, 64) || !encode_kv(&maps.v, V, Hkv, kv_sh, L, kv_sl, SPX_TILE_KEYS))
    return cudaErrorInvalidValue;
  static SpxOncePerDevice once;
  const cudaError_t ec = spx_opt_in_smem(prefill_tc2_kernel, kSmemBytes, &once);
  if (ec != cudaSuccess) return ec;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * W);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, prefill_tc2_kernel, a, maps);
}
