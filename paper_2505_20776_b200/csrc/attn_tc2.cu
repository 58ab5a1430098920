// Hybrid Tree Attention on pairs of SMs (tcgen05 cta_group::2), head dimension 128, row blocks of
// 256 stacked query rows.
//
// A cluster of two CTAs works on one range of (problem, 128-key tile) units.  CTA r of the pair
// owns the 128 query rows r*128.. of the row block: its Q rows, its S tiles, its P and its O
// accumulator live in its own tensor memory.  Each CTA stages only half of every K/V tile in its
// shared memory (K: 64 of the 128 keys; V: 64 of the 128 value columns); the pair's MMAs
// (M = 256, issued by one thread of the leader CTA) read both halves.  Compared with one CTA doing
// both row tiles this halves the shared-memory traffic per MMA, removes the re-reading of Q from
// shared memory (Q is the tensor-memory A operand), and frees tensor memory for P buffers of their own:
//
//   tensor memory per CTA: O [0,128) | S0 [128,256) | S1 [256,384) | Q [384,448) | P [448,512)
//
// A softmax thread pulls its whole S row into registers and releases its S buffer at once, so the
// S tiles run two key tiles ahead of the exponentials; P is kept in registers until the previous
// PV has consumed the P buffer, and the PV of a tile is issued whenever its P is complete.  The two
// softmax warpgroups of a CTA take alternate key tiles of the same 128 rows (one thread per row each); the running reference maximum of a
// row is handed from tile to tile through shared memory, each warpgroup keeps its own partial row
// sum, and O is rescaled lazily by whichever warpgroup raises the maximum by more than 2^8.
//
// Warps: 0-3 softmax of even tiles, 4-7 softmax of odd tiles, 8 TMA producer (own halves),
// 9 issuer of the S = Q K^T MMAs and 10 issuer of the O += P V MMAs (leader CTA only; two issuers
// so that neither kind waits behind the other's barriers), 11 ancestor masks.
// Barriers with arrivals from both CTAs live in the leader CTA; MMA completion is multicast to
// both CTAs.  Every wait is bounded; an expired wait raises SPECEXT_ERR_TIMEOUT, and both CTAs
// always reach the final cluster barrier before tensor memory is freed.
//
// The kernel is launched with programmatic stream serialization: barrier set-up, tensor-memory
// allocation and the start-up cluster barrier run while the kernel before it in the stream finishes;
// global memory is touched only after griddepcontrol.wait.
#include "common.cuh"
#include "pair.cuh"

using namespace sm100;
using namespace pair;

struct Tc2Maps {
  CUtensorMap kp, vp, kt, vt;
  CUtensorMap q;      // Q as [T][Hq][128] with boxes of 64 x G x 128/G: the 128 stacked rows of one CTA
};

namespace {

constexpr int kThreads = 384;
constexpr int kProducerWarp = 8, kMmaWarp = 9, kPvWarp = 10, kTreeWarp = 11;
constexpr int kRegsLaunch = 168, kRegsOther = 64, kRegsSoftmax = 216;
static_assert(128 * (kRegsLaunch - kRegsOther) >= 256 * (kRegsSoftmax - kRegsLaunch),
              "setmaxnreg.inc would wait for registers that are never released");
constexpr int D = 128;
constexpr int kStageBytes = 16384;             // half of a K tile (64 keys x 128) or of a V tile (128 keys x 64)
constexpr int kStages = 6;                     // per ring; one ring for K halves, one for V halves
constexpr int kCtrlOffset = 2 * kStages * kStageBytes;
constexpr int kSmemBytes = kCtrlOffset + 4096 + 1024;
constexpr float kRescaleThreshold = 8.0f;      // log2 units
constexpr uint32_t kColO = 0, kColS = 128, kColQ = 384, kColP = 448;

struct Ctrl {
  uint64_t k_full[kStages];     // leader: 2 arrivals (one producer per CTA) + bytes of both halves
  uint64_t k_empty[kStages];    // each CTA: MMA completion, multicast
  uint64_t v_full[kStages];
  uint64_t v_empty[kStages];
  uint64_t q_ready;             // leader: 16 arrivals (every softmax warp of both CTAs)
  uint64_t s_full[2];           // each CTA: multicast commit; S buffer w holds a tile for warpgroup w
  uint64_t s_free[2];           // leader: 8 arrivals; warpgroup w of both CTAs has its S tile in registers
  uint64_t p_full;              // leader: 8 arrivals (the warpgroup of each CTA that produced this tile's P)
  uint64_t pv_done[2];          // each CTA: multicast commit after the PV of a tile of warpgroup w
  uint64_t o_done;              // each CTA: multicast commit after the last PV of a segment
  uint64_t m_pub[2];            // this CTA: 4 arrivals, reference maxima of the tile are published
  uint64_t drain;
  uint64_t anc_ready;           // this CTA: the ancestor masks are in shared memory
  uint64_t q_land;              // this CTA: the first segment's Q rows have landed in the scratch (TMA)
  uint64_t v_rag;               // this CTA: a V half whose tail rows must be cleared has landed (device-side length)
  uint64_t epi[2];              // this CTA: 8 arrivals, the two meeting points of a segment's epilogue
  unsigned long long anc[kSpxMaxTree][2];
  int parent[kSpxMaxTree];
  float m_row[128];             // reference maximum of each row after the latest tile
  float l_x[128];               // epilogue: warpgroup 1 hands its row sums to warpgroup 0
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(Ctrl) <= 4096, "control block too large");

// SCORE: 0 no chunk sums; otherwise the class of the chunk size, so that each variant carries only the
// code it runs (the loop of the exponentials is instruction-cache sensitive): 1 chunks of 32 keys,
// 2 chunks of 64 or 128 keys, 3 chunks of fewer than 32 keys.
// DEVLEN: the prefix length is read from device memory (a.L_dev) and may be shorter than the planned
// capacity p.L; the instantiation without it carries none of that code.
template <int SCORE, bool DEVLEN>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc2_kernel(const __grid_constant__ AttnArgs a, const __grid_constant__ Tc2Maps maps) {
  const AttnPlan& p = a.plan;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                                         ~static_cast<uintptr_t>(1023));
  unsigned char* ring = base;
  Ctrl* ctl = reinterpret_cast<Ctrl*>(base + kCtrlOffset);
  volatile int* abort_flag = &ctl->abort_flag;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // The cluster barrier that makes both CTAs' mbarriers visible is split: the producer warp
  // initialises the barriers and arrives, every other warp arrives at once, and each warp waits just
  // before it first touches a barrier.  What needs no barrier (the Q copies, the tensor-memory
  // allocation, the ancestor masks) runs in between.
  if (warp == kProducerWarp) {
    // one barrier per lane (the four ring arrays first), so that the set-up is not 40 serial inits
    if (lane < kStages) {
      mbar_init(&ctl->k_full[lane], 2);
      mbar_init(&ctl->k_empty[lane], 1);
      mbar_init(&ctl->v_full[lane], 2);
      mbar_init(&ctl->v_empty[lane], 1);
    } else if (lane < kStages + 2) {
      const int i = lane - kStages;
      mbar_init(&ctl->s_full[i], 1);
      mbar_init(&ctl->s_free[i], 8);    // one arrival per warp: 4 warps of the warpgroup x 2 CTAs
      mbar_init(&ctl->pv_done[i], 1);
      mbar_init(&ctl->m_pub[i], 4);
      mbar_init(&ctl->epi[i], 8);
    } else if (lane == kStages + 2) {
      mbar_init(&ctl->q_ready, 16);     // one arrival per softmax warp of both CTAs
      mbar_init(&ctl->p_full, 8);
      mbar_init(&ctl->o_done, 1);
      mbar_init(&ctl->drain, 2);
      mbar_init(&ctl->anc_ready, 1);
      mbar_init(&ctl->q_land, 1);
      mbar_init(&ctl->v_rag, 1);
      ctl->abort_flag = 0;
    }
    fence_mbar_init();
  }
  cluster_arrive();
  // The kernel after this one (the merge) may be set up while this one runs; this one touches global
  // memory only once the kernel before it has completed (its set-up so far has used none).
  pdl_launch_dependents();
  if (warp != kMmaWarp) pdl_wait();

  const uint32_t rank = cluster_rank();
  const int cl = blockIdx.x >> 1;                        // the plan's "CTA" index is the cluster index
  const int unit_lo = spx_unit_start(p, cl), unit_hi = spx_unit_start(p, cl + 1);

  // The first segment's Q rows are requested before anything else, into a shared-memory scratch, so
  // that their latency runs under the set-up instead of delaying the first S MMA.  The scratch holds
  // the CTA's 128 rows twice 64 elements (warpgroup 0 reads the first 64 elements of a row, warpgroup
  // 1 the rest), 128 bytes per row with the 16-byte chunks XOR-swizzled by the row (the TMA 128-byte
  // swizzle), so that the per-row reads are conflict-free.  It is the tail of the V ring, which the
  // producer leaves alone until the first S MMA is done.  One thread fetches it with two TMA boxes
  // of 64 elements x G heads x 128/G nodes: exactly the stacked rows (G is a power of two), rows
  // past the tree zero-filled.
  // (With a device-side prefix length the first segment may turn out to be empty; its Q rows then
  // come by plain loads like those of every later segment.)
  constexpr bool dev_len = DEVLEN;
  if (warp == kProducerWarp && lane == 0 && unit_lo < unit_hi && !dev_len) {
    const int prob = unit_lo / p.UPP;
    const int g = prob / p.n_rblk, rblk = prob - g * p.n_rblk;
    const int t0 = (rblk * p.RB + (int)rank * 128) / p.G;
    unsigned char* scratch = ring + (2 * kStages - 2) * kStageBytes;
    mbar_arrive_expect_tx(&ctl->q_land, 2 * kStageBytes);
    tma_load_3d(scratch, &maps.q, &ctl->q_land, 0, g * p.G, t0);
    tma_load_3d(scratch + kStageBytes, &maps.q, &ctl->q_land, 64, g * p.G, t0);
    // The first K/V tiles can only be loaded once the pair's barriers are known to exist (a cluster
    // barrier away); until then their halves are at least pulled into L2.
    const int tile = unit_lo - prob * p.UPP;
    const bool is_tree = tile == p.TPH;
    const int key0 = is_tree ? 0 : tile * SPX_TILE_KEYS;
    const CUtensorMap* mk = is_tree ? &maps.kt : &maps.kp;
    tma_prefetch_3d(mk, 0, g, key0 + 64 * rank);
    tma_prefetch_3d(mk, 64, g, key0 + 64 * rank);
    tma_prefetch_3d(is_tree ? &maps.vt : &maps.vp, 64 * rank, g, key0);
  }

  if (warp == kProducerWarp && lane == 0) {
    prefetch_tensormap(&maps.q);
    prefetch_tensormap(&maps.kp);
    prefetch_tensormap(&maps.vp);
    prefetch_tensormap(&maps.kt);
    prefetch_tensormap(&maps.vt);
  }
  if (warp == kMmaWarp) {
    // tensor memory for the pair: both CTAs' warps with this index allocate all 512 columns
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
    cluster_wait();                        // both CTAs' barriers exist
    if (lane == 0) {
      uint32_t kp = 0, vp = 0;
      const uint64_t stream_once = policy_evict_first();
      const uint32_t kfull0 = map_to_cta(smem_u32(&ctl->k_full[0]), 0);      // leader's barriers
      const uint32_t vfull0 = map_to_cta(smem_u32(&ctl->v_full[0]), 0);
      if constexpr (!DEVLEN) {
        // position in the line of units
        struct Cursor {
          int unit, tile, prob, g;
        };
        auto step = [&](Cursor& c) {
          ++c.unit;
          if (++c.tile == p.UPP) {
            c.tile = 0;
            ++c.prob;
            c.g = c.prob / p.n_rblk;
          }
        };
        // K half of a unit: keys [64*rank, 64*rank+64) of the tile, two 64-column blocks
        auto load_k = [&](const Cursor& c) -> bool {
          const int tile = c.tile, g = c.g;
          const bool is_tree = tile == p.TPH;
          const int stage = kp % kStages;
          if (!wait_c(&ctl->k_empty[stage], ((kp / kStages) & 1) ^ 1, abort_flag)) return false;
          const uint32_t bar = kfull0 + stage * 8;
          const uint32_t dst = smem_u32(ring + stage * kStageBytes);
          const CUtensorMap* m = is_tree ? &maps.kt : &maps.kp;
          const int key0 = (is_tree ? 0 : tile * SPX_TILE_KEYS) + 64 * rank;
          arrive_expect_tx_cluster(bar, kStageBytes);
          tma_load_3d_pair_hint(dst, m, bar, 0, g, key0, stream_once);
          tma_load_3d_pair_hint(dst + 8192, m, bar, 64, g, key0, stream_once);
          ++kp;
          return true;
        };
        // V half of a unit: value columns [64*rank, 64*rank+64) of all 128 keys
        auto load_v = [&](const Cursor& c) -> bool {
          const int tile = c.tile, g = c.g;
          const bool is_tree = tile == p.TPH;
          const int stage = vp % kStages;
          if (!wait_c(&ctl->v_empty[stage], ((vp / kStages) & 1) ^ 1, abort_flag)) return false;
          const uint32_t bar = vfull0 + stage * 8;
          const uint32_t dst = smem_u32(ring + (kStages + stage) * kStageBytes);
          arrive_expect_tx_cluster(bar, kStageBytes);
          tma_load_3d_pair_hint(dst, is_tree ? &maps.vt : &maps.vp, bar, 64 * rank, g, is_tree ? 0 : tile * SPX_TILE_KEYS,
                              stream_once);
          ++vp;
          return true;
        };
        // Start-up: only two tiles are requested until the first S MMA has consumed K tile 0.  A full
        // ring requested at once by every SM sits in the memory system's queues in no particular order,
        // and tile 0 would arrive last as often as first.
        Cursor ck;
        ck.unit = unit_lo;
        ck.prob = unit_lo / p.UPP;
        ck.tile = unit_lo - ck.prob * p.UPP;
        ck.g = ck.prob / p.n_rblk;
        Cursor cv = ck;
        for (int i = 0; i < 2 && ck.unit < unit_hi && ok; ++i) {
          ok = load_k(ck);
          step(ck);
          if (ok) ok = load_v(cv);
          step(cv);
        }
        if (ok && unit_lo < unit_hi) ok = wait_c(&ctl->k_empty[0], 0, abort_flag);
        while (ok && ck.unit < unit_hi) {
          ok = load_k(ck);
          step(ck);
          if (ok) ok = load_v(cv);
          step(cv);
        }
      } else {
        const int L_eff = spx_prefix_len(a);
        const int tph_eff = (L_eff + SPX_TILE_KEYS - 1) / SPX_TILE_KEYS;
        uint32_t n_rag = 0;
        // position in the line of units: the run of units inside one problem and the tile inside the run
        struct Cursor {
          int u, g, tile_lo, n_units, j;
          SpxSeg sg;
        };
        auto enter = [&](Cursor& c) {                 // moves to the next run that has tiles to process
          while (c.u < unit_hi) {
            const int prob = c.u / p.UPP;
            c.tile_lo = c.u - prob * p.UPP;
            c.n_units = min(p.UPP - c.tile_lo, unit_hi - c.u);
            c.sg = spx_segment(p, c.tile_lo, c.n_units, tph_eff);
            c.g = prob / p.n_rblk;
            c.j = 0;
            if (c.sg.n > 0) return;
            c.u += c.n_units;
          }
        };
        auto step = [&](Cursor& c) {
          if (++c.j == c.sg.n) {
            c.u += c.n_units;
            enter(c);
          }
        };
        // K half of a unit: keys [64*rank, 64*rank+64) of the tile, two 64-column blocks
        auto load_k = [&](const Cursor& c) -> bool {
          const int tile = spx_seg_tile(p, c.sg, c.tile_lo, c.j), g = c.g;
          const bool is_tree = tile == p.TPH;
          const int stage = kp % kStages;
          if (!wait_c(&ctl->k_empty[stage], ((kp / kStages) & 1) ^ 1, abort_flag)) return false;
          const uint32_t bar = kfull0 + stage * 8;
          const uint32_t dst = smem_u32(ring + stage * kStageBytes);
          const CUtensorMap* m = is_tree ? &maps.kt : &maps.kp;
          const int key0 = (is_tree ? 0 : tile * SPX_TILE_KEYS) + 64 * rank;
          arrive_expect_tx_cluster(bar, kStageBytes);
          tma_load_3d_pair(dst, m, bar, 0, g, key0);       // (no eviction hint: a compact cache is read again at the next draft step)
          tma_load_3d_pair(dst + 8192, m, bar, 64, g, key0);
          ++kp;
          return true;
        };
        // V half of a unit: value columns [64*rank, 64*rank+64) of all 128 keys
        auto load_v = [&](const Cursor& c) -> bool {
          const int tile = spx_seg_tile(p, c.sg, c.tile_lo, c.j), g = c.g;
          const bool is_tree = tile == p.TPH;
          const int stage = vp % kStages;
          if (!wait_c(&ctl->v_empty[stage], ((vp / kStages) & 1) ^ 1, abort_flag)) return false;
          const uint32_t bar = vfull0 + stage * 8;
          unsigned char* dstp = ring + (kStages + stage) * kStageBytes;
          const int nk = is_tree ? SPX_TILE_KEYS : L_eff - tile * SPX_TILE_KEYS;
          if (dev_len && nk < SPX_TILE_KEYS) {
            // Device-side length: the tensor map spans the whole capacity, so the rows of this tile past the
            // length hold whatever the cache holds (their probabilities are zero, but zero times a NaN is
            // a NaN).  The half lands on a barrier of this CTA, its tail rows are cleared (a row is 128
            // bytes whatever the swizzle), and only then is the stage handed to the MMA issuer.
            mbar_arrive_expect_tx(&ctl->v_rag, kStageBytes);
            tma_load_3d(dstp, &maps.vp, &ctl->v_rag, 64 * rank, g, tile * SPX_TILE_KEYS);
            if (!mbar_wait(&ctl->v_rag, n_rag & 1, abort_flag)) return false;
            ++n_rag;
            uint4* tail = reinterpret_cast<uint4*>(dstp + nk * 128);
            for (int i = 0; i < (SPX_TILE_KEYS - nk) * 8; ++i) tail[i] = make_uint4(0u, 0u, 0u, 0u);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            arrive_release_cluster(bar);
          } else {
            arrive_expect_tx_cluster(bar, kStageBytes);
            tma_load_3d_pair(smem_u32(dstp), is_tree ? &maps.vt : &maps.vp, bar, 64 * rank, g,
                             is_tree ? 0 : tile * SPX_TILE_KEYS);
          }
          ++vp;
          return true;
        };
        // Start-up: only two tiles are requested until the first S MMA has consumed K tile 0.  A full
        // ring requested at once by every SM sits in the memory system's queues in no particular order,
        // and tile 0 would arrive last as often as first.
        Cursor ck;
        ck.u = unit_lo;
        enter(ck);
        Cursor cv = ck;
        const bool any = ck.u < unit_hi;
        for (int i = 0; i < 2 && ck.u < unit_hi && ok; ++i) {
          ok = load_k(ck);
          step(ck);
          if (ok) ok = load_v(cv);
          step(cv);
        }
        if (ok && any) ok = wait_c(&ctl->k_empty[0], 0, abort_flag);
        while (ok && ck.u < unit_hi) {
          ok = load_k(ck);
          step(ck);
          if (ok) ok = load_v(cv);
          step(cv);
        }
      }
    }
  } else {
    if (warp == kTreeWarp) {
      // registers first: the softmax warpgroups cannot grow until every warp of this warpgroup has shrunk
      setmaxnreg_dec<kRegsOther>();
#pragma unroll
      for (int q = 0; q < kSpxMaxTree / 32; ++q) ctl->parent[lane + 32 * q] = lane + 32 * q < p.T ? a.parent[lane + 32 * q] : -1;
      __syncwarp();
      bool bad = false;
#pragma unroll 1
      for (int q = 0; q < kSpxMaxTree / 32; ++q) {
        const int t = lane + 32 * q;
        SpxMask128 m = {0ull, 0ull};
        if (t < p.T) m = spx_walk_up(ctl->parent, p.T, t, bad);
        ctl->anc[t][0] = m.lo;
        ctl->anc[t][1] = m.hi;
      }
      if (bad && blockIdx.x == 0) spx_raise(a.status, SPECEXT_ERR_BAD_TREE);
      cluster_wait();                      // this CTA's barriers exist
      warp_arrive(&ctl->anc_ready, lane);
    }
    // the tensor-memory base address is visible to everybody who uses it (not the producer, not the tree warp)
    tc_fence_before();
    if (warp != kTreeWarp) {
      named_bar_sync(1, kThreads - 64);
      cluster_wait();                      // both CTAs' barriers exist
    }
    tc_fence_after();
    const uint32_t tmem = ctl->tmem_base;

    if (warp == kMmaWarp) {
      // ================================ issuer of S = Q K^T (leader CTA) =====================
      setmaxnreg_dec<kRegsOther>();
      if (lane == 0 && rank == 0) {
        const uint32_t idesc_s = idesc_bf16_f32(256, SPX_TILE_KEYS, false, false);
        constexpr uint32_t hi = desc_hi(1024);
        const uint32_t ring_lo = desc_lo(smem_u32(ring), 16);
        uint32_t kc = 0, n_w[2] = {0, 0};          // n_w[w]: S tiles issued so far for warpgroup w
        int seg = 0;
        const int tph_eff = DEVLEN ? (spx_prefix_len(a) + SPX_TILE_KEYS - 1) / SPX_TILE_KEYS : p.TPH;
        for (int u = unit_lo; u < unit_hi && ok;) {
          const int prob = u / p.UPP;
          const int tile_lo = u - prob * p.UPP;
          const int n_units = min(p.UPP - tile_lo, unit_hi - u);
          const int n = DEVLEN ? spx_segment(p, tile_lo, n_units, tph_eff).n : n_units;
          u += n_units;
          if (DEVLEN && n == 0) continue;          // nothing of this run exists at the device-side length
          ok = wait_c(&ctl->q_ready, seg & 1, abort_flag);
          for (int j = 0; j < n && ok; ++j) {
            const int w = j & 1;
            // S buffer w is free once warpgroup w holds its previous tile in registers
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
        uint32_t vc = 0;                           // V tiles consumed = PVs issued
        int seg = 0;
        const int tph_eff = DEVLEN ? (spx_prefix_len(a) + SPX_TILE_KEYS - 1) / SPX_TILE_KEYS : p.TPH;
        for (int u = unit_lo; u < unit_hi && ok;) {
          const int prob = u / p.UPP;
          const int tile_lo = u - prob * p.UPP;
          const int n_units = min(p.UPP - tile_lo, unit_hi - u);
          const int n = DEVLEN ? spx_segment(p, tile_lo, n_units, tph_eff).n : n_units;
          u += n_units;
          if (DEVLEN && n == 0) continue;
          ok = wait_c(&ctl->q_ready, seg & 1, abort_flag);      // every thread is done reading the previous O
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
        // everything issued by both issuers must be complete before tensor memory is released
        for (int spin = 0; spin < (1 << 22) && !try_wait_cluster(&ctl->drain, 0, 0u); ++spin) {}
      }
    } else if (warp == kTreeWarp) {
      // nothing left to do
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
      const float scale2 = p.scale2;
      uint32_t n_mine = 0;       // tiles this warpgroup has processed (phase of s_full[wg], m_pub[wg])
      uint32_t n_other = 0;      // tiles of the other warpgroup whose maxima this one has consumed
      uint32_t n_oth = 0;        // tiles the other warpgroup had been given before the current segment
      int seg = 0;
      bool anc_seen = false;
      const int L_eff = DEVLEN ? spx_prefix_len(a) : p.L;
      const int tph_eff = DEVLEN ? (L_eff + SPX_TILE_KEYS - 1) / SPX_TILE_KEYS : p.TPH;
      for (int u = unit_lo; u < unit_hi && ok;) {
        const int prob = u / p.UPP;
        const int tile_lo = u - prob * p.UPP;
        const int n_units = min(p.UPP - tile_lo, unit_hi - u);
        SpxSeg sg;
        if (DEVLEN) sg = spx_segment(p, tile_lo, n_units, tph_eff);
        const int n = DEVLEN ? sg.n : n_units;
        const int g = prob / p.n_rblk, rblk = prob - g * p.n_rblk;
        const int r = rblk * p.RB + rr;
        const bool valid = r < p.rows;
        const int t_node = valid ? r / p.G : 0;
        if (DEVLEN && n == 0) {
          // No tile of this run exists at the device-side length: its slot gets the neutral partial
          // (weight zero in the merge), and no barrier of the pipeline is touched.
          const int slot = cl + prob;
          if (valid) {
            float* po = a.ws + p.off_part_o + (long long)slot * (D / 4) * p.RB * 4;
#pragma unroll 4
            for (int q4 = 0; q4 < 16; ++q4)
              *reinterpret_cast<float4*>(po + ((long long)(wg * 16 + q4) * p.RB + rr) * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
            if (wg == 0) {
              a.ws[p.off_part_m + (long long)slot * p.RB + rr] = -1e30f;      // finite: see the merge
              a.ws[p.off_part_l + (long long)slot * p.RB + rr] = 0.f;
            }
          }
          u += n_units;
          continue;
        }
        // Q row of this thread -> tensor memory (warpgroup 0: first 64 elements, warpgroup 1: the rest)
        {
          uint32_t qv[32];
          const __nv_bfloat16* qbase = a.Q + (long long)(g * p.G) * a.q_sh + wg * 64;
          if (seg == 0 && !dev_len) {
            // requested at kernel start (see above)
            const unsigned char* scratch = ring + (2 * kStages - 2) * kStageBytes + warp * 4096;
            ok = mbar_wait(&ctl->q_land, 0, abort_flag);
            if (!ok) break;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const uint4 y = *reinterpret_cast<const uint4*>(scratch + lane * 128 + ((j ^ (lane & 7)) << 4));
              qv[j * 4] = y.x; qv[j * 4 + 1] = y.y; qv[j * 4 + 2] = y.z; qv[j * 4 + 3] = y.w;
            }
            // the scratch goes back to the V ring, which the TMA unit writes
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          } else if (valid) {
            const uint4* qp = reinterpret_cast<const uint4*>(qbase + (long long)t_node * a.q_st +
                                                             (long long)(r % p.G) * a.q_sh);
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
        if (DEVLEN ? !anc_seen : seg == 0) {
          ok = mbar_wait(&ctl->anc_ready, 0, abort_flag);
          if (!ok) break;
          anc_seen = true;
        }

        float m_loc = -INFINITY, l = 0.f;        // l is relative to m_loc
        for (int j = wg; j < n && ok; j += 2) {
          const int tile = DEVLEN ? spx_seg_tile(p, sg, tile_lo, j) : tile_lo + j;
          const bool is_tree = tile == p.TPH;
          const int nkeys = is_tree ? p.T : min(SPX_TILE_KEYS, (DEVLEN ? L_eff : p.L) - tile * SPX_TILE_KEYS);
          const bool need_mask = is_tree || nkeys < SPX_TILE_KEYS;
          ok = wait_c(&ctl->s_full[wg], n_mine & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          uint32_t s0[32], s1[32], s2[32], s3[32];
          tmem_ld32(s_addr, s0);
          tmem_ld32(s_addr + 32, s1);
          tmem_ld32(s_addr + 64, s2);
          tmem_ld32(s_addr + 96, s3);
          // The row's reference maximum after the previous tile (handled by the other warpgroup) is fetched
          // while the scores are on their way from tensor memory: it was published long before, as a rule.
          float m_cur = -INFINITY;
          if (j > 0) {
            ok = mbar_wait(&ctl->m_pub[wg ^ 1], n_other & 1, abort_flag);
            if (!ok) break;
            ++n_other;
            m_cur = ctl->m_row[row_t];
          }
          tmem_wait_ld();
          tc_fence_before();
          warp_arrive_cluster(s_free_l, lane);          // the S buffer may take the next tile
          if (need_mask) {
            unsigned long long vis_lo, vis_hi;
            if (is_tree) {                 // this node and its ancestors (a padding row sees key 0)
              vis_lo = valid ? ctl->anc[t_node][0] : 1ull;
              vis_hi = valid ? ctl->anc[t_node][1] : 0ull;
            } else {
              vis_lo = nkeys >= 64 ? ~0ull : ((1ull << nkeys) - 1ull);
              vis_hi = nkeys <= 64 ? 0ull : ((1ull << (nkeys - 64)) - 1ull);
            }
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
          const float m_tile = fmaxf(fmaxf(t0, t1), fmaxf(t2, t3)) * scale2;

          float m_new = m_cur;
          bool rescale = false;
          if (m_tile > m_cur + kRescaleThreshold || m_cur == -INFINITY) {
            m_new = m_tile;
            rescale = j > 0;
          }
          ctl->m_row[row_t] = m_new;
          warp_arrive(&ctl->m_pub[wg], lane);
          if (m_loc != m_new) {
            l *= (m_loc == -INFINITY) ? 0.f : ex2_approx(m_loc - m_new);
            m_loc = m_new;
          }
          // Completion of the PV of tile j-1 (the other warpgroup's) is needed before O may be
          // rescaled and before the P buffer may be overwritten; the PVs complete in order, so every
          // earlier one is complete then too.  One parity test on the other warpgroup's barrier is
          // enough: its previous completion (tile j-3) was waited for at this warpgroup's previous tile,
          // or lies in a segment whose end every thread has seen, and its next one (tile j+1) needs this
          // tile's P, so the barrier is either one completion short of the one asked for or at it.
          const uint32_t n_prev_other = n_oth + ((j + 1) >> 1);      // tiles given to the other warpgroup before j
          bool pv_seen = false;
          auto wait_prev_pv = [&]() -> bool {
            if (pv_seen) return true;
            pv_seen = true;
            if (n_prev_other > 0 && !wait_c(&ctl->pv_done[wg ^ 1], (n_prev_other - 1) & 1, abort_flag)) return false;
            tc_fence_after();
            return true;
          };
          if (__any_sync(0xffffffffu, rescale)) {
            // O must hold the sum up to tile j-1 and nothing may be accumulating into it
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
          const bool score = SCORE != 0 && !is_tree;
          float* mass = nullptr;
          if (score) {
            const long long rowbase = ((long long)prob * p.TPH + tile) * p.RB + rr;
            mass = a.ws + p.off_mass + rowbase * p.CPT;
            a.ws[p.off_mref + rowbase] = m_new;
          }
          float csum = 0.f;
          float cg[4] = {0.f, 0.f, 0.f, 0.f};      // chunk size 32: the tile's four chunk sums, stored as one float4
          uint32_t pk0[16], pk1[16], pk2[16], pk3[16];
          auto exp_chunk = [&](uint32_t (&v)[32], uint32_t (&pk)[16], int c) {
            // two elements per fma and per add (packed fp32 pairs); the exponential itself is per element
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
            const float gs = (gs0 + gs1) + (gs2 + gs3);
            l += gs;
            if (score) {
              if (SCORE == 1) {
                cg[c] = gs;
              } else if (SCORE == 2) {
                csum += gs;
                if ((((c + 1) * 32) & (p.C - 1)) == 0) {
                  mass[((c + 1) * 32) / p.C - 1] = csum;
                  csum = 0.f;
                }
              } else {
                float acc = 0.f;
#pragma unroll
                for (int k = 0; k < 32; ++k) {
                  acc += __uint_as_float(v[k]);
                  if (((k + 1) & (p.C - 1)) == 0) {
                    mass[(c * 32 + k) / p.C] = acc;
                    acc = 0.f;
                  }
                }
              }
            }
#pragma unroll
            for (int k = 0; k < 16; ++k) pk[k] = pack_bf16x2(__uint_as_float(v[2 * k]), __uint_as_float(v[2 * k + 1]));
          };
          exp_chunk(s0, pk0, 0);
          exp_chunk(s1, pk1, 1);
          exp_chunk(s2, pk2, 2);
          exp_chunk(s3, pk3, 3);
          if (SCORE == 1 && score) *reinterpret_cast<float4*>(mass) = make_float4(cg[0], cg[1], cg[2], cg[3]);
          // the P buffer is shared by all tiles: the PV of the previous tile must have read it
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

        // ---- epilogue of the segment --------------------------------------------------------
        // final reference maximum: published by the warpgroup that handled the last tile
        if (((n - 1) & 1) != wg) {
          ok = mbar_wait(&ctl->m_pub[wg ^ 1], n_other & 1, abort_flag);
          if (!ok) break;
          ++n_other;
        }
        const float m_fin = ctl->m_row[row_t];
        if (m_loc != m_fin) l *= (m_loc == -INFINITY) ? 0.f : ex2_approx(m_loc - m_fin);
        if (wg == 1) ctl->l_x[row_t] = l;
        ok = wait_c(&ctl->o_done, seg & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        n_oth += wg == 0 ? (n >> 1) : ((n + 1) >> 1);
        warp_arrive(&ctl->epi[0], lane);                 // l_x visible; both warpgroups past their last tile
        ok = mbar_wait(&ctl->epi[0], seg & 1, abort_flag);
        if (!ok) break;
        {
          const int slot = cl + prob;
          float* po = a.ws + p.off_part_o + (long long)slot * (D / 4) * p.RB * 4;
#pragma unroll
          for (int c = 0; c < 2; ++c) {                  // this warpgroup's 64 of the 128 columns
            uint32_t v[32];
            tmem_ld32(o_addr + wg * 64 + c * 32, v);
            tmem_wait_ld();
#pragma unroll
            for (int q4 = 0; q4 < 8; ++q4) {
              const float4 x = make_float4(__uint_as_float(v[q4 * 4]), __uint_as_float(v[q4 * 4 + 1]),
                                           __uint_as_float(v[q4 * 4 + 2]), __uint_as_float(v[q4 * 4 + 3]));
              if (valid) *reinterpret_cast<float4*>(po + ((long long)(wg * 16 + c * 8 + q4) * p.RB + rr) * 4) = x;
            }
          }
          if (wg == 0 && valid) {                        // rows past the last stacked row are never read
            a.ws[p.off_part_m + (long long)slot * p.RB + rr] = m_fin;
            a.ws[p.off_part_l + (long long)slot * p.RB + rr] = l + ctl->l_x[row_t];
          }
        }
        u += n_units;
        if (u < unit_hi) {
          warp_arrive(&ctl->epi[1], lane);               // l_x and m_row may be reused
          ok = mbar_wait(&ctl->epi[1], seg & 1, abort_flag);
        }
        ++seg;
      }
    }
  }

  if (!ok && lane == 0) spx_raise(a.status, SPECEXT_ERR_TIMEOUT);
  tc_fence_before();
  // The peer may still signal this CTA's barriers or read its halves, and tensor memory is freed by one
  // warp for all: everybody meets once more.  The partial results written above need no ordering here.
  cluster_sync_relaxed();
  if (warp == kMmaWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(ctl->tmem_base), "r"(512u) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn2() {
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

// bf16 tensor [n2][n1][128] with element strides (s2, s1, 1); box = 64 x 1 x b2, 128-byte swizzle,
// out-of-range elements read as zero.
bool encode_map2(CUtensorMap* m, const void* ptr, long long n1, long long s1, long long n2, long long s2, int b2) {
  EncodeTiledFn fn = encode_fn2();
  if (!fn) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)n1, (cuuint64_t)n2};
  const cuuint64_t strides[2] = {(cuuint64_t)s1 * 2, (cuuint64_t)s2 * 2};
  const cuuint32_t box[3] = {64, 1, (cuuint32_t)b2};
  const cuuint32_t es[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Q [T][Hq][128] (element strides q_st, q_sh, 1) with boxes of 64 elements x G heads x 128/G nodes.
bool encode_q_map(CUtensorMap* m, const void* ptr, int T, int Hq, int G, long long q_st, long long q_sh) {
  EncodeTiledFn fn = encode_fn2();
  if (!fn || G > 128 || 128 % G != 0) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)Hq, (cuuint64_t)T};
  const cuuint64_t strides[2] = {(cuuint64_t)q_sh * 2, (cuuint64_t)q_st * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)G, (cuuint32_t)(128 / G)};
  const cuuint32_t es[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int SCORE, bool DEVLEN>
cudaError_t launch2(const AttnArgs& a, const Tc2Maps& maps, cudaStream_t st) {
  static SpxOncePerDevice once;
  const cudaError_t ec = spx_opt_in_smem(attn_tc2_kernel<SCORE, DEVLEN>, kSmemBytes, &once);
  if (ec != cudaSuccess) return ec;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * a.plan.n_cta);
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
  return cudaLaunchKernelEx(&cfg, attn_tc2_kernel<SCORE, DEVLEN>, a, maps);
}

}  // namespace

// Requires head_dim 128 and 256-row blocks (plan.RB == 256); plan.n_cta counts clusters of two CTAs.
cudaError_t spx_launch_attn_tc2(const AttnArgs& a, cudaStream_t st, int* n_launches) {
  const AttnPlan& p = a.plan;
  if (p.D != D || p.RB != 256) return cudaErrorInvalidValue;
  Tc2Maps maps;
  bool ok = encode_map2(&maps.kt, a.Kt, p.Hkv, a.tkv_sh, p.T, a.tkv_st, 64);
  ok = ok && encode_map2(&maps.vt, a.Vt, p.Hkv, a.tkv_sh, p.T, a.tkv_st, SPX_TILE_KEYS);
  if (p.L > 0) {
    ok = ok && encode_map2(&maps.kp, a.Kp, p.Hkv, a.kv_sh, p.L, a.kv_sl, 64);
    ok = ok && encode_map2(&maps.vp, a.Vp, p.Hkv, a.kv_sh, p.L, a.kv_sl, SPX_TILE_KEYS);
  } else {
    maps.kp = maps.kt;
    maps.vp = maps.vt;
  }
  ok = ok && encode_q_map(&maps.q, a.Q, p.T, p.Hq, p.G, a.q_st, a.q_sh);
  if (!ok) return cudaErrorInvalidValue;
  const cudaError_t e = a.L_dev       ? launch2<0, true>(a, maps, st)       // never with chunk sums
                        : !p.want_score ? launch2<0, false>(a, maps, st)
                        : p.C == 32   ? launch2<1, false>(a, maps, st)
                        : p.C > 32    ? launch2<2, false>(a, maps, st)
                                      : launch2<3, false>(a, maps, st);
  *n_launches += 1;
  return e;
}
