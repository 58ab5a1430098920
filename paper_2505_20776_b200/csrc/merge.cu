// Log-sum-exp merge of the per-segment partial results, and the normalisation of the per-chunk
// sums into the head-averaged chunk scores that retrieval ranks.
//
// merge_kernel: one CTA = 32 query rows of one problem (warp = one 16-byte column group over the
// 32 rows, so partial reads are 512-byte coalesced).  For each row: M = max_s m_s,
// Z = sum_s l_s 2^(m_s - M), lse = (M + log2 Z) ln 2, O = sum_s O~_s 2^(m_s - M) / Z.
//
// score_kernel: one thread per (tree node, chunk): sums over all query heads the chunk's
// exponential sum rescaled from its tile's reference maximum to the row's final lse, i.e. the
// exactly normalised probability mass, and divides by Hq.
#include "common.cuh"

namespace {

constexpr float kLn2 = 0.693147180559945309417f;
constexpr float kLog2e = 1.44269504088896340736f;

__global__ void __launch_bounds__(128) merge_kernel(const __grid_constant__ AttnArgs a) {
  const AttnPlan& p = a.plan;
  extern __shared__ float wsm[];                       // [max_segs][32] merge weights
  const int blocks_per_prob = p.RB / 32;
  const int prob = blockIdx.x / blocks_per_prob;
  const int rr0 = (blockIdx.x - prob * blocks_per_prob) * 32;
  const int g = prob / p.n_rblk;
  const int rblk = prob - g * p.n_rblk;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int c_first = spx_unit_owner(p, prob * p.UPP);
  const int c_last = spx_unit_owner(p, (prob + 1) * p.UPP - 1);
  const int nseg = c_last - c_first + 1;
  const int slot0 = c_first + prob;
  if (rblk * p.RB + rr0 >= p.rows) return;             // whole CTA beyond the valid rows

  const int rr = rr0 + lane;
  const int r = rblk * p.RB + rr;
  const bool valid = r < p.rows;
  if (warp == 0) {
    float M = -INFINITY;
    for (int s = 0; s < nseg; ++s) M = fmaxf(M, a.ws[p.off_part_m + (long long)(slot0 + s) * p.RB + rr]);
    float Z = 0.f;
    for (int s = 0; s < nseg; ++s) {
      const float ms = a.ws[p.off_part_m + (long long)(slot0 + s) * p.RB + rr];
      const float ls = a.ws[p.off_part_l + (long long)(slot0 + s) * p.RB + rr];
      const float w = (ms == -INFINITY) ? 0.f : exp2f(ms - M);
      Z += ls * w;
      wsm[s * 32 + lane] = w;
    }
    const float inv = 1.f / Z;
    for (int s = 0; s < nseg; ++s) wsm[s * 32 + lane] *= inv;
    if (valid && blockIdx.y == 0) {
      const int t = r / p.G, h = g * p.G + r % p.G;
      a.lse[(long long)h * p.T + t] = (M + log2f(Z)) * kLn2;
    }
  }
  __syncthreads();
  if (!valid) return;

  const int nd4 = p.D / 4;
  const int per_y = nd4 / gridDim.y;
  const int t = r / p.G, h = g * p.G + r % p.G;
  __nv_bfloat16* orow = a.O + (long long)t * a.o_st + (long long)h * a.o_sh;
  for (int d4 = blockIdx.y * per_y + warp; d4 < (blockIdx.y + 1) * per_y; d4 += 4) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < nseg; ++s) {
      const float w = wsm[s * 32 + lane];
      const float4 v = *reinterpret_cast<const float4*>(
          a.ws + p.off_part_o + (((long long)(slot0 + s) * nd4 + d4) * p.RB + rr) * 4);
      acc.x = fmaf(w, v.x, acc.x);
      acc.y = fmaf(w, v.y, acc.y);
      acc.z = fmaf(w, v.z, acc.z);
      acc.w = fmaf(w, v.w, acc.w);
    }
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y);
    __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z, acc.w);
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&lo);
    pk.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(orow + d4 * 4) = pk;
  }
}

__global__ void __launch_bounds__(256) score_kernel(const __grid_constant__ AttnArgs a) {
  const AttnPlan& p = a.plan;
  const int t = blockIdx.y;
  const int c = blockIdx.x * 256 + threadIdx.x;
  if (c >= p.NC) return;
  const int tile = c / p.CPT, cc = c - tile * p.CPT;
  float acc = 0.f;
  for (int h = 0; h < p.Hq; ++h) {
    const int g = h / p.G, i = h - g * p.G;
    const int r = t * p.G + i;
    const int rblk = r / p.RB, rr = r - rblk * p.RB;
    const int prob = g * p.n_rblk + rblk;
    const long long base = ((long long)prob * p.TPH + tile) * p.RB + rr;
    const float lse2 = a.lse[(long long)h * p.T + t] * kLog2e;
    const float f = exp2f(a.ws[p.off_mref + base] - lse2);
    acc = fmaf(a.ws[p.off_mass + base * p.CPT + cc], f, acc);
  }
  a.chunk_score[(long long)t * p.NC + c] = acc / (float)p.Hq;
}

}  // namespace

cudaError_t spx_launch_merge(const AttnArgs& a, cudaStream_t st, int* n_launches) {
  const AttnPlan& p = a.plan;
  const int ysplit = (p.D / 4) % 8 == 0 ? 2 : 1;
  const dim3 grid(p.NP * (p.RB / 32), ysplit);
  merge_kernel<<<grid, 128, (size_t)p.max_segs * 32 * sizeof(float), st>>>(a);
  *n_launches += 1;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (p.want_score && p.NC > 0) {
    const dim3 sgrid((p.NC + 255) / 256, p.T);
    score_kernel<<<sgrid, 256, 0, st>>>(a);
    *n_launches += 1;
    e = cudaGetLastError();
  }
  return e;
}
