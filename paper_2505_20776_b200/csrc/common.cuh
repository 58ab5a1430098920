// Shared device/host declarations of the specext kernels.
#ifndef SPECEXT_COMMON_CUH_
#define SPECEXT_COMMON_CUH_

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/specext.h"
#include "plan.h"

struct AttnArgs {
  AttnPlan plan;
  const __nv_bfloat16* Q;
  const __nv_bfloat16* Kp;
  const __nv_bfloat16* Vp;
  const __nv_bfloat16* Kt;
  const __nv_bfloat16* Vt;
  const int32_t* parent;
  const int32_t* L_dev;     // device-side prefix length (<= plan.L, the planned capacity), or null: the length is plan.L
  __nv_bfloat16* O;
  float* lse;
  float* chunk_score;
  float* ws;
  int32_t* status;
  long long q_st, q_sh, kv_sl, kv_sh, tkv_st, tkv_sh, o_st, o_sh;
};


__device__ __forceinline__ void spx_raise(int32_t* status, int code) {
  if (status) atomicOr(status, 1 << code);
}

// Prefix length of this call.  A device-side length is read from global memory, so only after the
// kernel's dependency wait; it is clamped to [0, planned capacity].
__device__ __forceinline__ int spx_prefix_len(const AttnArgs& a) {
  if (!a.L_dev) return a.plan.L;
  const int v = *reinterpret_cast<const volatile int32_t*>(a.L_dev);
  return v < 0 ? 0 : (v > a.plan.L ? a.plan.L : v);
}

// Ancestor-or-self bit masks of the draft tree (up to kSpxMaxTree nodes, two 64-bit words per node): bit
// u is set iff u == t or u is a proper ancestor of t.  The walk up from node t is bounded by T steps; a
// parent outside [-1, u-1] ends it and is reported through `bad` (BAD_TREE).
constexpr int kSpxMaxTree = 128;
struct SpxMask128 {
  unsigned long long lo, hi;
};
__device__ __forceinline__ SpxMask128 spx_walk_up(const int* parent, int T, int t, bool& bad) {
  SpxMask128 m = {0ull, 0ull};
  int u = t;
  for (int step = 0; step <= T && u >= 0; ++step) {
    if (u < 64) m.lo |= 1ull << u; else m.hi |= 1ull << (u - 64);
    const int pu = parent[u];
    if (pu < -1 || pu >= u) {
      bad = true;
      break;
    }
    u = pu;
  }
  return m;
}
// The masks of all nodes into shared memory (anc_smem[2*t], anc_smem[2*t+1]) by the first 128 threads.
__device__ __forceinline__ void spx_build_ancestors(const int32_t* __restrict__ parent, int T,
                                                    unsigned long long* anc_smem, int32_t* status) {
  const int t = threadIdx.x;
  if (t < kSpxMaxTree) {
    SpxMask128 m = {0ull, 0ull};
    bool bad = false;
    if (t < T) m = spx_walk_up(parent, T, t, bad);
    if (bad) spx_raise(status, SPECEXT_ERR_BAD_TREE);
    anc_smem[2 * t] = m.lo;
    anc_smem[2 * t + 1] = m.hi;
  }
}

// A function attribute (the opt-in to large dynamic shared memory) belongs to the device's context, so
// it is set once per (kernel, device), with the device current: `done` is the kernel's own table.
constexpr int kSpxMaxDevices = 64;
struct SpxOncePerDevice {
  unsigned char done[kSpxMaxDevices] = {};
};
template <typename Kernel>
cudaError_t spx_opt_in_smem(Kernel* kernel, int bytes, SpxOncePerDevice* once) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool cached = dev >= 0 && dev < kSpxMaxDevices;
  if (cached && __atomic_load_n(&once->done[dev], __ATOMIC_ACQUIRE)) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess && cached) __atomic_store_n(&once->done[dev], (unsigned char)1, __ATOMIC_RELEASE);
  return e;
}

// Launchers implemented in the kernel translation units; each returns the cudaError_t of its launch.
#ifdef SPECEXT_TESTING
cudaError_t spx_launch_attn_simt(const AttnArgs& a, cudaStream_t st, int* n_launches);   // cross-check kernel, test library only
#endif
cudaError_t spx_launch_attn_tc(const AttnArgs& a, cudaStream_t st, int* n_launches);
cudaError_t spx_launch_attn_tc2(const AttnArgs& a, cudaStream_t st, int* n_launches);
cudaError_t spx_launch_merge(const AttnArgs& a, cudaStream_t st, int* n_launches);

#endif  // SPECEXT_COMMON_CUH_
