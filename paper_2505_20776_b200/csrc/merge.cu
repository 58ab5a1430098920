// Log-sum-exp merge of the per-segment partial results, and the normalisation of the per-chunk
// sums into the head-averaged chunk scores that retrieval ranks.
//
// merge_kernel: for each query row: M = max_s m_s,
// Z = sum_s l_s 2^(m_s - M), lse = (M + log2 Z) ln 2, O = sum_s O~_s 2^(m_s - M) / Z.
//
// score_kernel: for every (tree node, chunk) sums over all query heads the chunk's exponential sum
// rescaled from its tile's reference maximum to the row's final lse, i.e. the exactly normalised
// probability mass, and divides by Hq.
#include "common.cuh"
#include "sm100.cuh"

namespace {

constexpr float kLn2 = 0.693147180559945309417f;
constexpr int kMergeSmemCap = 200 * 1024;          // bytes of dynamic shared memory requested only to limit residency
constexpr float kLog2e = 1.44269504088896340736f;

// Block = 8 warps; warp w handles two 16-byte column groups (d4, d4 + 1) for 32 consecutive rows of
// one problem, so every partial read is a 512-byte coalesced segment, all reads of a thread are
// independent of each other, and the segment weights are computed once for eight output columns.
template <int B>
__device__ __forceinline__ void merge_batch(const float* __restrict__ pm, const float* __restrict__ pl,
                                            const float* __restrict__ po, long long ostride, int RB, int s, int n,
                                            float& M, float& Z, float4& acc0, float4& acc1) {
  // Segments s .. s+n-1 (n <= B).  Every load of the batch is in flight at once: issued one by one
  // they would each pay the full latency, and a second batch pays it a second time.
  float ms[B], ls[B];
  float4 v0[B], v1[B];
#pragma unroll
  for (int k = 0; k < B; ++k) {
    const bool in = k < n;
    const float4* q = reinterpret_cast<const float4*>(po + (s + k) * ostride);
    ms[k] = in ? __ldcg(pm + (long long)(s + k) * RB) : -INFINITY;
    ls[k] = in ? __ldcg(pl + (long long)(s + k) * RB) : 0.f;
    v0[k] = in ? __ldcg(q) : make_float4(0.f, 0.f, 0.f, 0.f);
    v1[k] = in ? __ldcg(q + RB) : make_float4(0.f, 0.f, 0.f, 0.f);     // next column group: RB float4 further on
  }
  float Mb = M;
#pragma unroll
  for (int k = 0; k < B; ++k) Mb = fmaxf(Mb, ms[k]);
  // (A worker that found no key, because a device-side length was shorter than planned, leaves the
  // neutral partial m = -1e30, l = 0, O = 0: finite, so that no difference of maxima is inf - inf.)
  const float carry = sm100::ex2_approx(M - Mb);    // 0 on the first batch (M = -inf)
  Z *= carry;
  acc0.x *= carry; acc0.y *= carry; acc0.z *= carry; acc0.w *= carry;
  acc1.x *= carry; acc1.y *= carry; acc1.z *= carry; acc1.w *= carry;
  M = Mb;
#pragma unroll
  for (int k = 0; k < B; ++k) {
    const float w = sm100::ex2_approx(ms[k] - M);
    Z = fmaf(ls[k], w, Z);
    acc0.x = fmaf(w, v0[k].x, acc0.x);
    acc0.y = fmaf(w, v0[k].y, acc0.y);
    acc0.z = fmaf(w, v0[k].z, acc0.z);
    acc0.w = fmaf(w, v0[k].w, acc0.w);
    acc1.x = fmaf(w, v1[k].x, acc1.x);
    acc1.y = fmaf(w, v1[k].y, acc1.y);
    acc1.z = fmaf(w, v1[k].z, acc1.z);
    acc1.w = fmaf(w, v1[k].w, acc1.w);
  }
}

__global__ void __launch_bounds__(256) merge_kernel(const __grid_constant__ AttnArgs a) {
  const AttnPlan& p = a.plan;
  sm100::pdl_launch_dependents();
  // everything that needs no global memory (indices, addresses, the output position) comes before the wait
  const int blocks_per_prob = p.RB / 32;
  const int prob = blockIdx.x / blocks_per_prob;
  const int rr0 = (blockIdx.x - prob * blocks_per_prob) * 32;
  const int g = prob / p.n_rblk;
  const int rblk = prob - g * p.n_rblk;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int rr = rr0 + lane;
  const int r = rblk * p.RB + rr;
  if (r >= p.rows) return;
  int c_first, c_last;
  if (p.cpp > 0 && p.UPP >= p.cpp) {               // every one of the problem's cpp workers has a segment
    c_first = prob * p.cpp;
    c_last = c_first + p.cpp - 1;
  } else {
    c_first = spx_unit_owner(p, prob * p.UPP);
    c_last = spx_unit_owner(p, (prob + 1) * p.UPP - 1);
  }
  const int nseg = c_last - c_first + 1;
  const int slot0 = c_first + prob;
  const int nd4 = p.D / 4;
  const int d4 = (blockIdx.y * 8 + warp) * 2;

  const float* pm = a.ws + p.off_part_m + (long long)slot0 * p.RB + rr;
  const float* pl = a.ws + p.off_part_l + (long long)slot0 * p.RB + rr;
  const float* po = a.ws + p.off_part_o + (((long long)slot0 * nd4 + d4) * p.RB + rr) * 4;
  const long long ostride = (long long)nd4 * p.RB * 4;
  const int t = r / p.G, h = g * p.G + r % p.G;
  __nv_bfloat16* out = a.O + (long long)t * a.o_st + (long long)h * a.o_sh + d4 * 4;
  float* lse_out = a.lse + (long long)h * p.T + t;

  sm100::pdl_wait();                               // the partial results of the attention kernel are complete
  float M = -INFINITY, Z = 0.f;
  float4 acc0 = make_float4(0.f, 0.f, 0.f, 0.f), acc1 = acc0;
  for (int s = 0; s < nseg; s += 12) merge_batch<12>(pm, pl, po, ostride, p.RB, s, min(12, nseg - s), M, Z, acc0, acc1);

  const float inv = 1.f / Z;
  if (d4 == 0) *lse_out = (M + log2f(Z)) * kLn2;
  __nv_bfloat162 b0 = __floats2bfloat162_rn(acc0.x * inv, acc0.y * inv);
  __nv_bfloat162 b1 = __floats2bfloat162_rn(acc0.z * inv, acc0.w * inv);
  __nv_bfloat162 b2 = __floats2bfloat162_rn(acc1.x * inv, acc1.y * inv);
  __nv_bfloat162 b3 = __floats2bfloat162_rn(acc1.z * inv, acc1.w * inv);
  uint4 pk;
  pk.x = *reinterpret_cast<uint32_t*>(&b0);
  pk.y = *reinterpret_cast<uint32_t*>(&b1);
  pk.z = *reinterpret_cast<uint32_t*>(&b2);
  pk.w = *reinterpret_cast<uint32_t*>(&b3);
  *reinterpret_cast<uint4*>(out) = pk;
}

// Block = 64 tree nodes x kScoreSlices slices of the KV heads, for one key tile and one group of VW
// chunks of the tile.  Consecutive threads are consecutive nodes, whose G stacked rows lie next to
// each other in the per-row arrays, so a warp reads whole lines; the VW chunk sums of a row are one
// vector load.  A slice sums its KV heads in a fixed order and the slices are added in a fixed
// order, so the result does not depend on the run.
constexpr int kScoreSlices = 8;

template <int VW>
__global__ void __launch_bounds__(64 * kScoreSlices) score_kernel(const __grid_constant__ AttnArgs a) {
  const AttnPlan& p = a.plan;
  __shared__ float part[kScoreSlices][64][VW];
  sm100::pdl_launch_dependents();
  sm100::pdl_wait();                               // lse and the chunk sums are complete
  const int t = blockIdx.z * 64 + threadIdx.x, slice = threadIdx.y;       // 64 tree nodes per block
  const int tile = blockIdx.x;
  const int c0 = blockIdx.y * VW;                  // first chunk of the group inside the tile
  float acc[VW];
#pragma unroll
  for (int k = 0; k < VW; ++k) acc[k] = 0.f;
  if (t < p.T) {
    for (int g = slice; g < p.Hkv; g += kScoreSlices) {
      for (int i = 0; i < p.G; ++i) {
        const int r = t * p.G + i;
        const int rblk = r / p.RB, rr = r - rblk * p.RB;
        const int prob = g * p.n_rblk + rblk;
        const long long base = ((long long)prob * p.TPH + tile) * p.RB + rr;
        const float lse2 = a.lse[(long long)(g * p.G + i) * p.T + t] * kLog2e;
        const float f = exp2f(a.ws[p.off_mref + base] - lse2);
        const float* m = a.ws + p.off_mass + base * p.CPT + c0;
        if (VW == 4) {
          const float4 v = *reinterpret_cast<const float4*>(m);
          acc[0] = fmaf(v.x, f, acc[0]);
          acc[1 % VW] = fmaf(v.y, f, acc[1 % VW]);
          acc[2 % VW] = fmaf(v.z, f, acc[2 % VW]);
          acc[3 % VW] = fmaf(v.w, f, acc[3 % VW]);
        } else {
#pragma unroll
          for (int k = 0; k < VW; ++k) acc[k] = fmaf(m[k], f, acc[k]);
        }
      }
    }
  }
#pragma unroll
  for (int k = 0; k < VW; ++k) part[slice][threadIdx.x][k] = acc[k];
  __syncthreads();
  if (slice == 0 && t < p.T) {
    const float inv = 1.f / (float)p.Hq;
#pragma unroll
    for (int k = 0; k < VW; ++k) {
      float sum = 0.f;
#pragma unroll
      for (int q = 0; q < kScoreSlices; ++q) sum += part[q][threadIdx.x][k];
      const int c = tile * p.CPT + c0 + k;
      if (c < p.NC) a.chunk_score[(long long)t * p.NC + c] = sum * inv;
    }
  }
}

template <int VW>
cudaError_t launch_score(const AttnArgs& a, dim3 grid, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(64, kScoreSlices);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, score_kernel<VW>, a);
}

}  // namespace

cudaError_t spx_launch_merge(const AttnArgs& a, cudaStream_t st, int* n_launches) {
  const AttnPlan& p = a.plan;
  const dim3 grid(p.NP * (p.RB / 32), p.D / 64);
  // Launched so that its blocks may be resident (waiting) before the attention kernel has finished.
  // Blocks become resident wherever an SM has room, so without a limit the SMs that the attention
  // kernel leaves first would take eight blocks each and a fraction of the SMs would do all the work:
  // an (unused) dynamic shared-memory request caps residency at one block per SM (measured: 1.1 us
  // per call faster than two per SM, which in turn was 2 us faster than no cap).
  static SpxOncePerDevice once;
  const cudaError_t ec = spx_opt_in_smem(merge_kernel, kMergeSmemCap, &once);
  if (ec != cudaSuccess) return ec;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(256);
  cfg.dynamicSmemBytes = kMergeSmemCap;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, merge_kernel, a);
  *n_launches += 1;
  if (e != cudaSuccess) return e;
  if (p.want_score && p.NC > 0) {
    if (p.CPT >= 4) {
      e = launch_score<4>(a, dim3(p.TPH, p.CPT / 4, (p.T + 63) / 64), st);
    } else if (p.CPT == 2) {
      e = launch_score<2>(a, dim3(p.TPH, 1, (p.T + 63) / 64), st);
    } else {
      e = launch_score<1>(a, dim3(p.TPH, 1, (p.T + 63) / 64), st);
    }
    *n_launches += 1;
  }
  return e;
}
