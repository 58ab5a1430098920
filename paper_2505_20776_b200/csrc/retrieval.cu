// SelectChunks and UpdateDraftCache kernels.
//
// select_kernel (one CTA): the ranking key of chunk c is score[c] / len_c, a non-negative fp32
// whose bit pattern orders like the value.  A most-significant-digit radix select (4 passes of
// 8 bits, warp-aggregated shared-memory histograms) finds the k-th largest key exactly; every
// chunk with a larger key is kept, and of the chunks equal to it the lowest-indexed are kept
// until k are chosen.  A block-wide ballot/popcount scan in index order then emits the kept
// chunks in ascending order, which also implements the tie rule.
//
// gather_kernel: 16-byte vector copy of the kept chunks of the draft K and V into the compact cache.
#include "common.cuh"
#include "sm100.cuh"

namespace {

constexpr int kSelThreads = 1024;
constexpr int kFusedThreads = 256;
constexpr int kFusedMaxK = 1024;           // selected indices a fused block keeps in shared memory
constexpr int kFusedMaxChunks = 8192;      // above this every block repeating the selection costs more than a launch

// Shape of one selection: chunk count, prefix length, chunk size, and the forced chunks (the first n_sink
// and the last n_recent chunks are kept whatever their score; 0 and 0 = the plain top-k).
struct SelShape {
  int NC, L, C, n_sink, n_recent;
};

__device__ __forceinline__ uint32_t chunk_key(const float* __restrict__ score, int c, const SelShape& sh) {
  if (c < sh.n_sink || c >= sh.NC - sh.n_recent) return 0x7F800000u;     // +inf: above every finite key, ties by index
  const int len = (c == sh.NC - 1) ? (sh.L - c * sh.C) : sh.C;
  float x = score[c] / (float)len;
  if (!(x > 0.f)) x = 0.f;                 // -0, negative or NaN rank lowest
  if (x > 3.0e38f) x = 3.0e38f;            // a finite score never reaches the forced chunks' key
  return __float_as_uint(x);
}

constexpr int kKeyCache = 2048;            // ranking keys kept in shared memory (more chunks: recomputed per pass)

template <int NT>
struct SelectSmem {
  uint32_t hist[4][256];                   // one histogram per radix pass: cleared once, no barrier in between
  uint32_t s_prefix[4], s_need[4];
  uint32_t warp_eq[2][NT / 32], warp_keep[2][NT / 32];     // per batch of NT chunks, double-buffered
  uint32_t keys[kKeyCache];
};

// Selection by one block of NT threads: writes the keff = min(k, NC) kept chunk indices, ascending,
// to idx_out (global or shared memory).  Every thread of the block must call it.  Two block barriers per
// radix pass and two per batch of NT chunks in the emission.
template <int NT>
__device__ __forceinline__ void select_block(SelectSmem<NT>& sm, const float* __restrict__ score, const SelShape& sh,
                                             int keff, int32_t* idx_out) {
  const int NC = sh.NC;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int NW = NT / 32;
  // one load and one division per chunk when the keys fit in shared memory
  const bool cached = NC <= kKeyCache;
  if (cached)
    for (int c = tid; c < NC; c += NT) sm.keys[c] = chunk_key(score, c, sh);
  auto key_of = [&](int c) -> uint32_t { return cached ? sm.keys[c] : chunk_key(score, c, sh); };
  for (int i = tid; i < 4 * 256; i += NT) (&sm.hist[0][0])[i] = 0;
  __syncthreads();

  // ---- radix select of the keff-th largest key --------------------------------------------
  uint32_t prefix = 0, need = keff;        // `need` keys still to take among those matching prefix
#pragma unroll 1
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    const uint32_t himask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
    for (int c = tid; c < NC; c += NT) {
      const uint32_t key = key_of(c);
      if ((key & himask) == prefix) atomicAdd(&sm.hist[pass][(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (warp == 0) {
      // bins from high to low: lane owns bins 255-8*lane .. 248-8*lane
      uint32_t local[8], tot = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        local[i] = sm.hist[pass][255 - (lane * 8 + i)];
        tot += local[i];
      }
      uint32_t incl = tot;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      uint32_t before = incl - tot;       // keys in strictly higher bins than this lane's
      if (before < need && need <= incl) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (before < need && need <= before + local[i]) {
            sm.s_prefix[pass] = prefix | ((uint32_t)(255 - (lane * 8 + i)) << shift);
            sm.s_need[pass] = need - before;
          }
          before += local[i];
        }
      }
    }
    __syncthreads();
    prefix = sm.s_prefix[pass];
    need = sm.s_need[pass];
  }
  const uint32_t theta = prefix;           // the keff-th largest key
  const uint32_t need_eq = need;           // how many keys equal to theta are kept (lowest indices)

  // ---- emit in ascending index order --------------------------------------------------------
  uint32_t carry_eq = 0, carry_keep = 0;   // totals of the batches before this one (the same in every thread)
  int buf = 0;
  for (int base = 0; base < NC; base += NT, buf ^= 1) {
    const int c = base + tid;
    uint32_t key = 0;
    const bool in = c < NC;
    if (in) key = key_of(c);
    const bool eq = in && key == theta;
    const bool gt = in && key > theta;
    const uint32_t beq = __ballot_sync(0xffffffffu, eq);
    if (lane == 0) sm.warp_eq[buf][warp] = __popc(beq);
    __syncthreads();
    uint32_t eq_before = carry_eq + __popc(beq & ((1u << lane) - 1u)), eq_all = 0;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const uint32_t x = sm.warp_eq[buf][w];
      eq_all += x;
      if (w < warp) eq_before += x;
    }
    const bool keep = gt || (eq && eq_before < need_eq);
    const uint32_t bk = __ballot_sync(0xffffffffu, keep);
    if (lane == 0) sm.warp_keep[buf][warp] = __popc(bk);
    __syncthreads();
    uint32_t pos = carry_keep + __popc(bk & ((1u << lane) - 1u)), keep_all = 0;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const uint32_t x = sm.warp_keep[buf][w];
      keep_all += x;
      if (w < warp) pos += x;
    }
    if (keep && pos < (uint32_t)keff) idx_out[pos] = c;
    carry_eq += eq_all;
    carry_keep += keep_all;
  }
}

template <int NT>
__global__ void __launch_bounds__(NT) select_kernel(const float* __restrict__ score, const SelShape sh, int k,
                                                    int32_t* __restrict__ idx, int32_t* __restrict__ n_selected) {
  __shared__ SelectSmem<NT> sm;
  sm100::pdl_launch_dependents();
  sm100::pdl_wait();                       // the scores are complete
  const int keff = min(k, sh.NC);
  select_block<NT>(sm, score, sh, keff, idx);
  if (threadIdx.x == 0) *n_selected = keff;
}

struct GatherArgs {
  const __nv_bfloat16* src[2];
  __nv_bfloat16* dst[2];
  const int32_t* idx;
  const int32_t* n_selected;
  int32_t* n_tokens_out;
  int32_t* status;
  int n_layers, H, D, L, C, NC, max_selected, sub;
  long long s_layer, s_l, s_h;
  // fused selection (select_gather_kernel only)
  const float* score;
  int32_t* idx_out;
  int32_t* n_selected_out;
  int k, n_sink, n_recent;
};

// Copies the tokens [o_lo, o_hi) of kept chunk number i (chunk index c) of one layer of K or V.
__device__ __forceinline__ void gather_part(const GatherArgs& g, int i, int c, int part, int layer, int which) {
  const int len = min(g.C, g.L - c * g.C);
  const int tok_per_part = (g.C + g.sub - 1) / g.sub;
  const int o_lo = part * tok_per_part, o_hi = min(len, o_lo + tok_per_part);
  const int vpr = g.D / 8;                            // 16-byte vectors per head row
  const int vpt = g.H * vpr;                          // per token
  const __nv_bfloat16* src = g.src[which] + (long long)layer * g.s_layer;
  __nv_bfloat16* dst = g.dst[which] + ((long long)layer * g.max_selected * g.C + (long long)i * g.C) * g.H * g.D;
  const int nvec = max(0, o_hi - o_lo) * vpt;
  if (g.s_h == g.D && g.s_l == (long long)g.H * g.D) {
    // tokens are contiguous in the source as they are in the compact cache: a plain copy of one range,
    // four vectors per thread and round, all loads issued before the first store
    const uint4* sp = reinterpret_cast<const uint4*>(src + (long long)(c * g.C + o_lo) * g.s_l);
    uint4* dp = reinterpret_cast<uint4*>(dst + (long long)o_lo * g.H * g.D);
    for (int v0 = threadIdx.x; v0 < nvec; v0 += 4 * blockDim.x) {
      uint4 x[4];
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (v0 + q * (int)blockDim.x < nvec) x[q] = __ldg(sp + v0 + q * blockDim.x);
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (v0 + q * (int)blockDim.x < nvec) dp[v0 + q * blockDim.x] = x[q];
    }
    return;
  }
  // strided source: four vectors per thread and round, all loads issued before the first store
  for (int v0 = threadIdx.x; v0 < nvec; v0 += 4 * blockDim.x) {
    uint4 x[4];
    long long off[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int v = v0 + q * blockDim.x;
      if (v < nvec) {
        const int o = o_lo + v / vpt;
        const int w = v - (v / vpt) * vpt;
        const int hh = w / vpr, dv = w - hh * vpr;
        x[q] = *reinterpret_cast<const uint4*>(src + (long long)(c * g.C + o) * g.s_l + (long long)hh * g.s_h + dv * 8);
        off[q] = ((long long)o * g.H + hh) * g.D + dv * 8;
      }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q)
      if (v0 + q * blockDim.x < nvec) *reinterpret_cast<uint4*>(dst + off[q]) = x[q];
  }
}

__global__ void __launch_bounds__(256) gather_kernel(const __grid_constant__ GatherArgs g) {
  const int i = blockIdx.x / g.sub;                  // which selected chunk
  const int part = blockIdx.x - i * g.sub;           // which slice of its tokens
  const int layer = blockIdx.y;
  const int which = blockIdx.z;                      // 0 = K, 1 = V
  sm100::pdl_launch_dependents();
  sm100::pdl_wait();                                 // idx and n_selected are complete
  int nsel = *g.n_selected;
  nsel = max(0, min(nsel, g.max_selected));
  if (blockIdx.x == 0 && layer == 0 && which == 0 && threadIdx.x == 0) {
    int ntok = 0;
    if (nsel > 0) {
      const int last = g.idx[nsel - 1];
      if (last >= 0 && last < g.NC) ntok = (nsel - 1) * g.C + min(g.C, g.L - last * g.C);
    }
    *g.n_tokens_out = ntok;
  }
  if (i >= nsel) return;
  const int c = g.idx[i];
  if (c < 0 || c >= g.NC) {
    if (threadIdx.x == 0 && part == 0) spx_raise(g.status, SPECEXT_ERR_INVALID_ARG);
    return;
  }
  gather_part(g, i, c, part, layer, which);
}

// SelectChunks and UpdateDraftCache in one launch: every block repeats the (deterministic) selection
// in its own shared memory and then copies its share of the kept chunks, so no block waits for
// another; block (0, 0, 0) also writes idx, n_selected and n_tokens.
__global__ void __launch_bounds__(kFusedThreads) select_gather_kernel(const __grid_constant__ GatherArgs g) {
  __shared__ SelectSmem<kFusedThreads> sm;
  __shared__ int32_t s_idx[kFusedMaxK];
  const int i = blockIdx.x / g.sub;
  const int part = blockIdx.x - i * g.sub;
  const int layer = blockIdx.y;
  const int which = blockIdx.z;
  sm100::pdl_launch_dependents();
  sm100::pdl_wait();                                 // the scores are complete
  const int keff = min(g.k, g.NC);
  if (i >= keff) return;                             // uniform for the block
  const SelShape sh = {g.NC, g.L, g.C, g.n_sink, g.n_recent};
  select_block<kFusedThreads>(sm, g.score, sh, keff, s_idx);
  __syncthreads();
  if (blockIdx.x == 0 && layer == 0 && which == 0) {
    for (int j = threadIdx.x; j < keff; j += kFusedThreads) g.idx_out[j] = s_idx[j];
    if (threadIdx.x == 0) {
      *g.n_selected_out = keff;
      const int last = s_idx[keff - 1];
      *g.n_tokens_out = (keff - 1) * g.C + min(g.C, g.L - last * g.C);
    }
  }
  gather_part(g, i, s_idx[i], part, layer, which);
}

cudaError_t launch_pdl(const void* kernel, dim3 grid, dim3 block, void** args, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelExC(&cfg, kernel, args);
}

void fill_gather_args(GatherArgs& g, const void* dK, const void* dV, int n_layers, int H, int D, int L, int C,
                      long long s_layer, long long s_l, long long s_h, int max_selected, void* K_out, void* V_out,
                      int32_t* n_tokens_out, int32_t* status) {
  g.src[0] = static_cast<const __nv_bfloat16*>(dK);
  g.src[1] = static_cast<const __nv_bfloat16*>(dV);
  g.dst[0] = static_cast<__nv_bfloat16*>(K_out);
  g.dst[1] = static_cast<__nv_bfloat16*>(V_out);
  g.n_tokens_out = n_tokens_out;
  g.status = status;
  g.n_layers = n_layers; g.H = H; g.D = D; g.L = L; g.C = C;
  g.NC = (L + C - 1) / C;
  g.max_selected = max_selected;
  // aim for ~16 KB per CTA
  const long long chunk_bytes = (long long)C * H * D * 2;
  int sub = (int)((chunk_bytes + 16383) / 16384);
  sub = max(1, min(sub, C));
  g.sub = sub;
  g.s_layer = s_layer; g.s_l = s_l; g.s_h = s_h;
  g.idx = nullptr; g.n_selected = nullptr;
  g.score = nullptr; g.idx_out = nullptr; g.n_selected_out = nullptr; g.k = 0; g.n_sink = 0; g.n_recent = 0;
}

}  // namespace

cudaError_t spx_launch_select(const float* score_row, int NC, int L, int C, int k, int n_sink, int n_recent,
                              int32_t* idx, int32_t* n_selected, cudaStream_t st) {
  SelShape sh = {NC, L, C, n_sink, n_recent};
  void* args[] = {&score_row, &sh, &k, &idx, &n_selected};
  // few chunks: a small block, whose barriers are cheap; many: the widest one
  if (NC <= 2048)
    return launch_pdl(reinterpret_cast<const void*>(select_kernel<kFusedThreads>), dim3(1), dim3(kFusedThreads), args, st);
  return launch_pdl(reinterpret_cast<const void*>(select_kernel<kSelThreads>), dim3(1), dim3(kSelThreads), args, st);
}

cudaError_t spx_launch_gather(const void* dK, const void* dV, int n_layers, int H, int D, int L, int C,
                              long long s_layer, long long s_l, long long s_h, const int32_t* idx,
                              const int32_t* n_selected, int max_selected, void* K_out, void* V_out,
                              int32_t* n_tokens_out, int32_t* status, cudaStream_t st) {
  GatherArgs g;
  fill_gather_args(g, dK, dV, n_layers, H, D, L, C, s_layer, s_l, s_h, max_selected, K_out, V_out, n_tokens_out,
                   status);
  g.idx = idx;
  g.n_selected = n_selected;
  void* args[] = {&g};
  return launch_pdl(reinterpret_cast<const void*>(gather_kernel), dim3(max_selected * g.sub, n_layers, 2), dim3(256),
                    args, st);
}

// True when SelectChunks + UpdateDraftCache of this size run as one launch.
bool spx_select_gather_fusable(int NC, int k) { return NC >= 1 && NC <= kFusedMaxChunks && k <= kFusedMaxK; }

cudaError_t spx_launch_select_gather(const float* score_row, int k, int n_sink, int n_recent, const void* dK,
                                     const void* dV, int n_layers,
                                     int H, int D, int L, int C, long long s_layer, long long s_l, long long s_h,
                                     int32_t* idx, int32_t* n_selected, void* K_out, void* V_out,
                                     int32_t* n_tokens_out, int32_t* status, cudaStream_t st) {
  GatherArgs g;
  fill_gather_args(g, dK, dV, n_layers, H, D, L, C, s_layer, s_l, s_h, k, K_out, V_out, n_tokens_out, status);
  g.score = score_row;
  g.idx_out = idx;
  g.n_selected_out = n_selected;
  g.k = k;
  g.n_sink = n_sink;
  g.n_recent = n_recent;
  void* args[] = {&g};
  const int keff = k < g.NC ? k : g.NC;
  return launch_pdl(reinterpret_cast<const void*>(select_gather_kernel), dim3(keff * g.sub, n_layers, 2),
                    dim3(kFusedThreads), args, st);
}
