// Plain CUDA-core (no tensor core) split-over-KV tree attention producing the same partial
// results as the tensor-core kernels.  It is compiled into the test library only, where it serves as
// an independent on-device cross-check of those kernels; the product library does not contain it.
//
// One CTA of 256 threads handles 64 query rows of one row block: thread = (row, quarter of D).
// Per key tile of 128 tokens: pass 1 forms the scaled scores (log2 domain) of the tile in shared
// memory and their maximum; pass 2 exponentiates against the running maximum, accumulates the
// row sum, the per-chunk sums and the P*V product in fp32.
#include "common.cuh"

namespace {

constexpr int kRowsPerCta = 64;
constexpr int kSStride = SPX_TILE_KEYS + 1;

template <int D>
__global__ void __launch_bounds__(256) attn_simt_kernel(const __grid_constant__ AttnArgs a) {
  constexpr int DQ = D / 4;
  const AttnPlan& p = a.plan;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __nv_bfloat16* Ks = reinterpret_cast<__nv_bfloat16*>(smem_raw);
  __nv_bfloat16* Vs = Ks + SPX_TILE_KEYS * D;
  float* S = reinterpret_cast<float*>(Vs + SPX_TILE_KEYS * D);
  unsigned long long* anc = reinterpret_cast<unsigned long long*>(S + kRowsPerCta * kSStride);

  spx_build_ancestors(a.parent, p.T, anc, (blockIdx.x == 0 && blockIdx.y == 0) ? a.status : nullptr);
  __syncthreads();

  const int tid = threadIdx.x;
  const int row_local = tid >> 2;
  const int quarter = tid & 3;
  const int cta = blockIdx.x;
  const int rr = blockIdx.y * kRowsPerCta + row_local;   // row inside the row block
  const int unit_hi = spx_unit_start(p, cta + 1);
  int u = spx_unit_start(p, cta);

  while (u < unit_hi) {
    const int prob = u / p.UPP;
    const int tile_lo = u - prob * p.UPP;
    const int tile_hi = min(p.UPP, tile_lo + (unit_hi - u));
    const int g = prob / p.n_rblk;
    const int rblk = prob - g * p.n_rblk;
    const int r = rblk * p.RB + rr;
    const bool valid = r < p.rows;
    const int t = valid ? r / p.G : 0;
    const int h = g * p.G + (valid ? r % p.G : 0);

    float q[DQ], o[DQ];
    {
      const __nv_bfloat16* qp = a.Q + (long long)t * a.q_st + (long long)h * a.q_sh + quarter * DQ;
#pragma unroll
      for (int d = 0; d < DQ; ++d) {
        q[d] = valid ? __bfloat162float(qp[d]) : 0.f;
        o[d] = 0.f;
      }
    }
    float m = -INFINITY, l = 0.f;
    const unsigned long long my_anc_lo = anc[2 * t], my_anc_hi = anc[2 * t + 1];

    for (int tile = tile_lo; tile < tile_hi; ++tile) {
      const bool is_tree = tile == p.TPH;
      const int nkeys = is_tree ? p.T : min(SPX_TILE_KEYS, p.L - tile * SPX_TILE_KEYS);
      // stage K and V rows of this tile (zero beyond nkeys)
      {
        constexpr int VPR = D / 8;                      // 16-byte vectors per row
        const __nv_bfloat16* kb = is_tree ? a.Kt + (long long)g * a.tkv_sh
                                          : a.Kp + (long long)tile * SPX_TILE_KEYS * a.kv_sl + (long long)g * a.kv_sh;
        const __nv_bfloat16* vb = is_tree ? a.Vt + (long long)g * a.tkv_sh
                                          : a.Vp + (long long)tile * SPX_TILE_KEYS * a.kv_sl + (long long)g * a.kv_sh;
        const long long rs = is_tree ? a.tkv_st : a.kv_sl;
        for (int v = tid; v < SPX_TILE_KEYS * VPR; v += 256) {
          const int j = v / VPR, dv = v - j * VPR;
          uint4 kx = make_uint4(0, 0, 0, 0), vx = make_uint4(0, 0, 0, 0);
          if (j < nkeys) {
            kx = *reinterpret_cast<const uint4*>(kb + (long long)j * rs + dv * 8);
            vx = *reinterpret_cast<const uint4*>(vb + (long long)j * rs + dv * 8);
          }
          *reinterpret_cast<uint4*>(Ks + j * D + dv * 8) = kx;
          *reinterpret_cast<uint4*>(Vs + j * D + dv * 8) = vx;
        }
      }
      __syncthreads();

      // pass 1: scores of the tile (log2 domain) and their maximum
      float tmax = -INFINITY;
      for (int j = 0; j < SPX_TILE_KEYS; ++j) {
        const __nv_bfloat16* kr = Ks + j * D + quarter * DQ;
        float acc = 0.f;
#pragma unroll
        for (int d = 0; d < DQ; ++d) acc = fmaf(q[d], __bfloat162float(kr[d]), acc);
        acc += __shfl_xor_sync(0xffffffffu, acc, 1);
        acc += __shfl_xor_sync(0xffffffffu, acc, 2);
        float s = acc * p.scale2;
        const bool vis = (j < nkeys) && (!is_tree || (((j < 64 ? my_anc_lo >> j : my_anc_hi >> (j - 64)) & 1ull) != 0));
        s = vis ? s : -INFINITY;
        tmax = fmaxf(tmax, s);
        if (quarter == 0) S[row_local * kSStride + j] = s;
      }
      __syncwarp();

      const float m_new = fmaxf(m, tmax);
      const float alpha = (m_new == -INFINITY) ? 1.f : exp2f(m - m_new);
      l *= alpha;
#pragma unroll
      for (int d = 0; d < DQ; ++d) o[d] *= alpha;
      m = m_new;

      // pass 2: exponentials, row sum, chunk sums, P*V
      const bool score = p.want_score && !is_tree;
      float* mass = nullptr;
      if (score) {
        const long long base = ((long long)prob * p.TPH + tile) * p.RB + rr;
        mass = a.ws + p.off_mass + base * p.CPT;
        if (quarter == 0) a.ws[p.off_mref + base] = m;
      }
      float csum = 0.f;
      for (int j = 0; j < SPX_TILE_KEYS; ++j) {
        const float s = S[row_local * kSStride + j];
        const float pj = (s == -INFINITY) ? 0.f : exp2f(s - m);
        l += pj;
        csum += pj;
        if (score && ((j + 1) % p.C == 0)) {
          if (quarter == 0) mass[j / p.C] = csum;
          csum = 0.f;
        }
        const __nv_bfloat16* vr = Vs + j * D + quarter * DQ;
#pragma unroll
        for (int d = 0; d < DQ; ++d) o[d] = fmaf(pj, __bfloat162float(vr[d]), o[d]);
      }
      __syncthreads();
    }

    // partial result of this segment
    {
      const int slot = cta + prob;
      float* po = a.ws + p.off_part_o + (long long)slot * (D / 4) * p.RB * 4;
#pragma unroll
      for (int d4 = 0; d4 < DQ / 4; ++d4) {
        const float4 v = make_float4(o[d4 * 4], o[d4 * 4 + 1], o[d4 * 4 + 2], o[d4 * 4 + 3]);
        *reinterpret_cast<float4*>(po + ((long long)(quarter * (DQ / 4) + d4) * p.RB + rr) * 4) = v;
      }
      if (quarter == 0) {
        a.ws[p.off_part_m + (long long)slot * p.RB + rr] = m;
        a.ws[p.off_part_l + (long long)slot * p.RB + rr] = l;
      }
    }
    u += tile_hi - tile_lo;
  }
}

}  // namespace

cudaError_t spx_launch_attn_simt(const AttnArgs& a, cudaStream_t st, int* n_launches) {
  const AttnPlan& p = a.plan;
  const dim3 grid(p.n_cta, p.RB / kRowsPerCta);
  const size_t smem = 2ull * SPX_TILE_KEYS * p.D * sizeof(__nv_bfloat16) +
                      kRowsPerCta * kSStride * sizeof(float) + 2 * kSpxMaxTree * sizeof(unsigned long long);
  cudaError_t e;
  if (p.D == 128) {
    e = cudaFuncSetAttribute(attn_simt_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attn_simt_kernel<128><<<grid, 256, smem, st>>>(a);
  } else if (p.D == 64) {
    e = cudaFuncSetAttribute(attn_simt_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attn_simt_kernel<64><<<grid, 256, smem, st>>>(a);
  } else {
    return cudaErrorInvalidValue;
  }
  *n_launches += 1;
  return cudaGetLastError();
}
