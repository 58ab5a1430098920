// Host side of the C ABI: argument checks, work decomposition, workspace layout and launches.
#include <atomic>
#include <cmath>
#include <cstring>

#include "common.cuh"

cudaError_t spx_launch_select(const float* score_row, int NC, int L, int C, int k, int n_sink, int n_recent,
                              int32_t* idx, int32_t* n_selected, cudaStream_t st);
cudaError_t spx_launch_gather(const void* dK, const void* dV, int n_layers, int H, int D, int L, int C,
                              long long s_layer, long long s_l, long long s_h, const int32_t* idx,
                              const int32_t* n_selected, int max_selected, void* K_out, void* V_out,
                              int32_t* n_tokens_out, int32_t* status, cudaStream_t st);
cudaError_t spx_launch_prefill_tc2(const void* Q, const void* K, const void* V, void* O, float* lse, int L, int Hq,
                                   int Hkv, float scale2, long long q_st, long long q_sh, long long kv_sl,
                                   long long kv_sh, long long o_st, long long o_sh, int n_sm, int32_t* status,
                                   cudaStream_t st);
bool spx_select_gather_fusable(int NC, int k);
cudaError_t spx_launch_select_gather(const float* score_row, int k, int n_sink, int n_recent, const void* dK,
                                     const void* dV, int n_layers,
                                     int H, int D, int L, int C, long long s_layer, long long s_l, long long s_h,
                                     int32_t* idx, int32_t* n_selected, void* K_out, void* V_out,
                                     int32_t* n_tokens_out, int32_t* status, cudaStream_t st);

// Scratch of the entry point that takes no workspace.  Part of the library image: resident on every
// device that loads the library until the process exits.  Device code may name it directly; host
// code must go through cudaGetSymbolAddress (see specext_verify_attn_static_scratch).
static __device__ __align__(256) unsigned char g_static_scratch[SPECEXT_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = kSpxMaxDevices;
std::atomic<void*> g_static_scratch_addr[kMaxDevices];

std::atomic<long long> g_launches{0};

// Kernel choice and split granularity.  The product library has one choice per shape; the test library
// (SPECEXT_TESTING) can override it so that the tests reach the other kernels and coarser splits.
#ifdef SPECEXT_TESTING
std::atomic<int> g_attn_kernel{0};       // 0 = default, 1 = CUDA-core kernel, 2 = one-CTA kernel, 3 = paired kernel
std::atomic<int> g_min_units{1};         // lower bound on key tiles per worker
int tuning_kernel() { return g_attn_kernel.load(); }
int tuning_min_units() { return g_min_units.load() < 1 ? 1 : g_min_units.load(); }
#else
constexpr int tuning_kernel() { return 0; }
constexpr int tuning_min_units() { return 1; }
#endif

// Multiprocessor count of the current device (looked up once per device).
int sm_count() {
  static std::atomic<int> cached[kMaxDevices];
  int dev = -1, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) {
    (void)cudaGetLastError();
    return 148;                           // B200; used only when no device is present (size queries)
  }
  if (dev < kMaxDevices && (n = cached[dev].load()) > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
    (void)cudaGetLastError();
    return 148;
  }
  if (dev < kMaxDevices) cached[dev].store(n);
  return n;
}

bool is_pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int build_plan(const specext_attn_desc* d, AttnPlan* out) {
  if (!d) return SPECEXT_ERR_INVALID_ARG;
  if (d->n_q_heads < 1 || d->n_kv_heads < 1 || d->n_q_heads % d->n_kv_heads != 0) return SPECEXT_ERR_INVALID_ARG;
  if (d->prefix_len < 0 || d->prefix_len > (1 << 24)) return SPECEXT_ERR_INVALID_ARG;
  if (d->n_tree < 1 || d->n_tree > kSpxMaxTree) return SPECEXT_ERR_UNSUPPORTED;
  if (d->head_dim != 64 && d->head_dim != 128) return SPECEXT_ERR_UNSUPPORTED;
  if (!is_pow2(d->chunk_size) || d->chunk_size > 128) return SPECEXT_ERR_UNSUPPORTED;
  const int G = d->n_q_heads / d->n_kv_heads;
  if (!is_pow2(G) || G > 64) return SPECEXT_ERR_UNSUPPORTED;
  if (!(d->softmax_scale >= 0.f) || !std::isfinite(d->softmax_scale)) return SPECEXT_ERR_INVALID_ARG;
  const long long strides[8] = {d->q_stride_t, d->q_stride_h, d->kv_stride_l, d->kv_stride_h,
                                d->tkv_stride_t, d->tkv_stride_h, d->o_stride_t, d->o_stride_h};
  for (long long s : strides)
    if (s < d->head_dim || (s & 7) != 0) return SPECEXT_ERR_INVALID_ARG;

  AttnPlan p;
  std::memset(&p, 0, sizeof(p));
  p.Hq = d->n_q_heads; p.Hkv = d->n_kv_heads; p.G = G; p.D = d->head_dim;
  p.L = d->prefix_len; p.T = d->n_tree; p.C = d->chunk_size;
  p.rows = G * p.T;
  // (a tree of more than 64 nodes with head_dim 128 always takes 256-row blocks: the one-CTA kernel keeps
  // one mask word per node there)
  p.RB = (p.rows > 128 || (p.D == 128 && p.T > 64)) ? 256 : 128;
  p.n_rblk = (p.rows + p.RB - 1) / p.RB;
  p.NP = p.Hkv * p.n_rblk;
  p.TPH = (p.L + SPX_TILE_KEYS - 1) / SPX_TILE_KEYS;
  p.UPP = p.TPH + 1;
  const long long U = (long long)p.NP * p.UPP;
  if (U > (1ll << 30)) return SPECEXT_ERR_UNSUPPORTED;
  p.U = (int)U;
  const int min_units = tuning_min_units();
  const int want = tuning_kernel();
  const bool pair_ok = p.D == 128 && p.RB == 256;       // what the paired-CTA kernel is built for
  p.kernel = want == 1 ? 1 : ((want == 0 || want == 3) && pair_ok ? 3 : 2);   // want != 0 only in the test library
  if (p.kernel == 2 && p.D == 128 && p.T > 64) return SPECEXT_ERR_UNSUPPORTED;  // (only reachable by a test override)
  if (p.kernel == 3) {
    // one worker = a cluster of two CTAs; every problem gets the same number of workers when possible
    const int n_workers = sm_count() / 2 > 0 ? sm_count() / 2 : 1;
    if (p.NP <= n_workers) {
      int cpp = n_workers / p.NP;
      if (cpp > p.UPP / min_units) cpp = p.UPP / min_units;
      if (cpp < 1) cpp = 1;
      p.cpp = cpp;
      p.n_cta = p.NP * cpp;
      p.q = p.UPP / cpp;
      p.rem = p.UPP % cpp;
      p.max_segs = cpp;
    } else {
      p.cpp = 0;
      p.n_cta = n_workers;
      p.q = p.U / p.n_cta;
      p.rem = p.U % p.n_cta;
      p.max_segs = (p.UPP + p.q - 1) / p.q + 1;
    }
  } else {
    int n_cta = p.U / min_units;
    if (n_cta < 1) n_cta = 1;
    if (n_cta > sm_count()) n_cta = sm_count();
    p.cpp = 0;
    p.n_cta = n_cta;
    p.q = p.U / n_cta;
    p.rem = p.U % n_cta;
    p.max_segs = (p.UPP + p.q - 1) / p.q + 1;
  }
  if (p.max_segs > p.n_cta) p.max_segs = p.n_cta;
  p.n_slots = p.n_cta + p.NP - 1;
  p.CPT = SPX_TILE_KEYS / p.C;
  p.NC = (p.L + p.C - 1) / p.C;
  p.want_score = d->want_chunk_score != 0;
  const float scale = d->softmax_scale > 0.f ? d->softmax_scale : 1.0f / std::sqrt((float)p.D);
  p.scale2 = scale * 1.44269504088896340736f;
  long long off = 0;
  p.off_part_o = off; off += (long long)p.n_slots * p.D * p.RB;
  p.off_part_m = off; off += (long long)p.n_slots * p.RB;
  p.off_part_l = off; off += (long long)p.n_slots * p.RB;
  if (p.want_score) {
    p.off_mass = off; off += (long long)p.NP * p.TPH * p.RB * p.CPT;
    p.off_mref = off; off += (long long)p.NP * p.TPH * p.RB;
  }
  p.total_floats = off;
  *out = p;
  return SPECEXT_OK;
}

int check_gather_args(const void* draft_K, const void* draft_V, int32_t n_layers, int32_t n_kv_heads,
                      int32_t head_dim, int32_t prefix_len, int32_t chunk_size, int64_t stride_layer,
                      int64_t stride_l, int64_t stride_h, int32_t max_selected, const void* K_out,
                      const void* V_out, const int32_t* n_tokens_out) {
  if (!draft_K || !draft_V || !K_out || !V_out || !n_tokens_out) return SPECEXT_ERR_INVALID_ARG;
  if (n_layers < 1 || n_layers > 65535 || n_kv_heads < 1 || head_dim < 8 || (head_dim & 7) != 0 ||
      prefix_len < 0 || chunk_size < 1 || max_selected < 1)
    return SPECEXT_ERR_INVALID_ARG;
  if (stride_h < head_dim || (stride_h & 7) || stride_l < head_dim || (stride_l & 7) || (stride_layer & 7) ||
      stride_layer < 0)
    return SPECEXT_ERR_INVALID_ARG;
  if (!aligned16(draft_K) || !aligned16(draft_V) || !aligned16(K_out) || !aligned16(V_out))
    return SPECEXT_ERR_INVALID_ARG;
  if ((long long)max_selected * chunk_size > (1ll << 28)) return SPECEXT_ERR_UNSUPPORTED;
  return SPECEXT_OK;
}

}  // namespace

extern "C" {

size_t specext_verify_attn_workspace(const specext_attn_desc* desc) {
  AttnPlan p;
  if (build_plan(desc, &p) != SPECEXT_OK) return 0;
  return (size_t)p.total_floats * sizeof(float);
}

}  // extern "C"

namespace {

// Checks, plan and launches shared by specext_verify_attn (prefix_len_dev == null) and
// specext_draft_attn (the prefix length is read on the device, desc->prefix_len is its upper bound).
int run_attn(const specext_attn_desc* desc, const void* Q, const void* K_prefix, const void* V_prefix,
             const void* K_tree, const void* V_tree, const int32_t* parent, const int32_t* prefix_len_dev,
             void* O, float* lse, float* chunk_score, void* workspace, size_t workspace_bytes,
             int32_t* device_status, void* cuda_stream) {
  AttnArgs a;
  const int rc = build_plan(desc, &a.plan);
  if (rc != SPECEXT_OK) return rc;
  const AttnPlan& p = a.plan;
  if (prefix_len_dev && (p.want_score || p.kernel == 1 || (reinterpret_cast<uintptr_t>(prefix_len_dev) & 3u) != 0))
    return p.want_score ? SPECEXT_ERR_INVALID_ARG : (p.kernel == 1 ? SPECEXT_ERR_UNSUPPORTED : SPECEXT_ERR_INVALID_ARG);
  a.L_dev = prefix_len_dev;
  if (!Q || !K_tree || !V_tree || !parent || !O || !lse || !workspace) return SPECEXT_ERR_INVALID_ARG;
  if (p.L > 0 && (!K_prefix || !V_prefix)) return SPECEXT_ERR_INVALID_ARG;
  if (p.want_score && p.NC > 0 && !chunk_score) return SPECEXT_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K_prefix) || !aligned16(V_prefix) || !aligned16(K_tree) ||
      !aligned16(V_tree) || !aligned16(O) || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0 ||
      (reinterpret_cast<uintptr_t>(lse) & 3u) != 0 || (reinterpret_cast<uintptr_t>(parent) & 3u) != 0)
    return SPECEXT_ERR_INVALID_ARG;
  if (workspace_bytes < (size_t)p.total_floats * sizeof(float)) return SPECEXT_ERR_WORKSPACE;

  a.Q = static_cast<const __nv_bfloat16*>(Q);
  a.Kp = static_cast<const __nv_bfloat16*>(K_prefix);
  a.Vp = static_cast<const __nv_bfloat16*>(V_prefix);
  a.Kt = static_cast<const __nv_bfloat16*>(K_tree);
  a.Vt = static_cast<const __nv_bfloat16*>(V_tree);
  a.parent = parent;
  a.O = static_cast<__nv_bfloat16*>(O);
  a.lse = lse;
  a.chunk_score = chunk_score;
  a.ws = static_cast<float*>(workspace);
  a.status = device_status;
  a.q_st = desc->q_stride_t; a.q_sh = desc->q_stride_h;
  a.kv_sl = desc->kv_stride_l; a.kv_sh = desc->kv_stride_h;
  a.tkv_st = desc->tkv_stride_t; a.tkv_sh = desc->tkv_stride_h;
  a.o_st = desc->o_stride_t; a.o_sh = desc->o_stride_h;

  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int n = 0;
  cudaError_t e;
#ifdef SPECEXT_TESTING
  if (p.kernel == 1) e = spx_launch_attn_simt(a, st, &n); else
#endif
  e = p.kernel == 3 ? spx_launch_attn_tc2(a, st, &n) : spx_launch_attn_tc(a, st, &n);
  if (e == cudaSuccess) e = spx_launch_merge(a, st, &n);
  g_launches.fetch_add(n);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return SPECEXT_ERR_CUDA;
  }
  return SPECEXT_OK;
}

}  // namespace

extern "C" {

int specext_verify_attn(const specext_attn_desc* desc, const void* Q, const void* K_prefix,
                        const void* V_prefix, const void* K_tree, const void* V_tree,
                        const int32_t* parent, void* O, float* lse, float* chunk_score,
                        void* workspace, size_t workspace_bytes, int32_t* device_status,
                        void* cuda_stream) {
  return run_attn(desc, Q, K_prefix, V_prefix, K_tree, V_tree, parent, nullptr, O, lse, chunk_score, workspace,
                  workspace_bytes, device_status, cuda_stream);
}

int specext_draft_attn(const specext_attn_desc* desc, const void* Q, const void* K_cache,
                       const void* V_cache, const int32_t* n_tokens, const void* K_tree,
                       const void* V_tree, const int32_t* parent, void* O, float* lse, void* workspace,
                       size_t workspace_bytes, int32_t* device_status, void* cuda_stream) {
  if (!n_tokens) return SPECEXT_ERR_INVALID_ARG;
  return run_attn(desc, Q, K_cache, V_cache, K_tree, V_tree, parent, n_tokens, O, lse, nullptr, workspace,
                  workspace_bytes, device_status, cuda_stream);
}

int specext_prefill_attn(const specext_attn_desc* desc, const void* Q, const void* K, const void* V, void* O,
                         float* lse, int32_t* device_status, void* cuda_stream) {
  if (!desc || !Q || !K || !V || !O || !lse) return SPECEXT_ERR_INVALID_ARG;
  if (desc->n_q_heads < 1 || desc->n_kv_heads < 1 || desc->n_q_heads % desc->n_kv_heads != 0)
    return SPECEXT_ERR_INVALID_ARG;
  if (desc->prefix_len < 1 || desc->prefix_len > (1 << 24)) return SPECEXT_ERR_INVALID_ARG;
  if (!(desc->softmax_scale >= 0.f) || !std::isfinite(desc->softmax_scale)) return SPECEXT_ERR_INVALID_ARG;
  const int G = desc->n_q_heads / desc->n_kv_heads;
  if (desc->head_dim != 128 || !is_pow2(G) || G > 256) return SPECEXT_ERR_UNSUPPORTED;
  const long long strides[6] = {desc->q_stride_t, desc->q_stride_h, desc->kv_stride_l, desc->kv_stride_h,
                                desc->o_stride_t, desc->o_stride_h};
  for (long long s : strides)
    if (s < desc->head_dim || (s & 7) != 0) return SPECEXT_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || (reinterpret_cast<uintptr_t>(lse) & 3u) != 0)
    return SPECEXT_ERR_INVALID_ARG;
  const float scale = desc->softmax_scale > 0.f ? desc->softmax_scale : 1.0f / std::sqrt((float)desc->head_dim);
  const cudaError_t e = spx_launch_prefill_tc2(Q, K, V, O, lse, desc->prefix_len, desc->n_q_heads, desc->n_kv_heads,
                                               scale * 1.44269504088896340736f, desc->q_stride_t, desc->q_stride_h,
                                               desc->kv_stride_l, desc->kv_stride_h, desc->o_stride_t,
                                               desc->o_stride_h, sm_count(), device_status,
                                               static_cast<cudaStream_t>(cuda_stream));
  g_launches.fetch_add(1);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return SPECEXT_ERR_CUDA;
  }
  return SPECEXT_OK;
}

int specext_verify_attn_static_scratch(const specext_attn_desc* desc, const void* Q,
                                       const void* K_prefix, const void* V_prefix,
                                       const void* K_tree, const void* V_tree,
                                       const int32_t* parent, void* O, float* lse,
                                       float* chunk_score, int32_t* device_status,
                                       void* cuda_stream) {
  // Reject a bad descriptor, or a shape that does not fit, before touching the device.
  AttnPlan plan;
  const int rc = build_plan(desc, &plan);
  if (rc != SPECEXT_OK) return rc;
  if ((size_t)plan.total_floats * sizeof(float) > SPECEXT_STATIC_SCRATCH_BYTES) return SPECEXT_ERR_WORKSPACE;
  // g_static_scratch names a host-side handle of the device array, not a device address: the address
  // valid on the current device comes from cudaGetSymbolAddress, looked up once per device.
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    (void)cudaGetLastError();
    return SPECEXT_ERR_CUDA;
  }
  void* scratch = g_static_scratch_addr[dev].load();
  if (!scratch) {
    if (cudaGetSymbolAddress(&scratch, g_static_scratch) != cudaSuccess || !scratch) {
      (void)cudaGetLastError();
      return SPECEXT_ERR_CUDA;
    }
    g_static_scratch_addr[dev].store(scratch);
  }
  return specext_verify_attn(desc, Q, K_prefix, V_prefix, K_tree, V_tree, parent, O, lse, chunk_score, scratch,
                             SPECEXT_STATIC_SCRATCH_BYTES, device_status, cuda_stream);
}

int specext_select_chunks(const float* chunk_score, int32_t n_tree, int32_t n_chunks, int32_t row,
                          int32_t prefix_len, int32_t chunk_size, int32_t k, int32_t n_sink_chunks,
                          int32_t n_recent_chunks, int32_t* idx, int32_t* n_selected, int32_t* device_status,
                          void* cuda_stream) {
  (void)device_status;
  if (!idx || !n_selected) return SPECEXT_ERR_INVALID_ARG;
  if (n_tree < 1 || row < 0 || row >= n_tree || k < 1 || chunk_size < 1 || prefix_len < 0 || n_sink_chunks < 0 ||
      n_recent_chunks < 0)
    return SPECEXT_ERR_INVALID_ARG;
  const long long nc = ((long long)prefix_len + chunk_size - 1) / chunk_size;
  if (nc != n_chunks) return SPECEXT_ERR_INVALID_ARG;
  if (n_chunks > 65536) return SPECEXT_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e;
  if (n_chunks == 0) {
    e = cudaMemsetAsync(n_selected, 0, sizeof(int32_t), st);
  } else {
    if (!chunk_score) return SPECEXT_ERR_INVALID_ARG;
    e = spx_launch_select(chunk_score + (long long)row * n_chunks, n_chunks, prefix_len, chunk_size, k,
                          n_sink_chunks, n_recent_chunks, idx, n_selected, st);
    g_launches.fetch_add(1);
  }
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return SPECEXT_ERR_CUDA;
  }
  return SPECEXT_OK;
}

int specext_gather_kv(const void* draft_K, const void* draft_V, int32_t n_layers,
                      int32_t n_kv_heads, int32_t head_dim, int32_t prefix_len, int32_t chunk_size,
                      int64_t stride_layer, int64_t stride_l, int64_t stride_h, const int32_t* idx,
                      const int32_t* n_selected, int32_t max_selected, void* K_out, void* V_out,
                      int32_t* n_tokens_out, int32_t* device_status, void* cuda_stream) {
  if (!idx || !n_selected) return SPECEXT_ERR_INVALID_ARG;
  const int rc = check_gather_args(draft_K, draft_V, n_layers, n_kv_heads, head_dim, prefix_len, chunk_size,
                                   stride_layer, stride_l, stride_h, max_selected, K_out, V_out, n_tokens_out);
  if (rc != SPECEXT_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = spx_launch_gather(draft_K, draft_V, n_layers, n_kv_heads, head_dim, prefix_len, chunk_size,
                                    stride_layer, stride_l, stride_h, idx, n_selected, max_selected, K_out,
                                    V_out, n_tokens_out, device_status, st);
  g_launches.fetch_add(1);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return SPECEXT_ERR_CUDA;
  }
  return SPECEXT_OK;
}

int specext_select_gather(const float* chunk_score, int32_t n_tree, int32_t n_chunks, int32_t row,
                          int32_t prefix_len, int32_t chunk_size, int32_t k, int32_t n_sink_chunks,
                          int32_t n_recent_chunks, const void* draft_K,
                          const void* draft_V, int32_t n_layers, int32_t n_kv_heads, int32_t head_dim,
                          int64_t stride_layer, int64_t stride_l, int64_t stride_h, int32_t* idx,
                          int32_t* n_selected, void* K_out, void* V_out, int32_t* n_tokens_out,
                          int32_t* device_status, void* cuda_stream) {
  const long long nc = chunk_size >= 1 && prefix_len >= 0 ? ((long long)prefix_len + chunk_size - 1) / chunk_size : -1;
  const bool fuse = nc == n_chunks && n_tree >= 1 && row >= 0 && row < n_tree && k >= 1 && chunk_score &&
                    n_sink_chunks >= 0 && n_recent_chunks >= 0 && spx_select_gather_fusable(n_chunks, k);
  if (!fuse) {
    // sizes the single launch is not built for, and every invalid argument, take the two calls
    const int rc = specext_select_chunks(chunk_score, n_tree, n_chunks, row, prefix_len, chunk_size, k,
                                         n_sink_chunks, n_recent_chunks, idx, n_selected, device_status, cuda_stream);
    if (rc != SPECEXT_OK) return rc;
    return specext_gather_kv(draft_K, draft_V, n_layers, n_kv_heads, head_dim, prefix_len, chunk_size, stride_layer,
                             stride_l, stride_h, idx, n_selected, k, K_out, V_out, n_tokens_out, device_status,
                             cuda_stream);
  }
  if (!idx || !n_selected) return SPECEXT_ERR_INVALID_ARG;
  const int rc = check_gather_args(draft_K, draft_V, n_layers, n_kv_heads, head_dim, prefix_len, chunk_size,
                                   stride_layer, stride_l, stride_h, k, K_out, V_out, n_tokens_out);
  if (rc != SPECEXT_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const cudaError_t e = spx_launch_select_gather(chunk_score + (long long)row * n_chunks, k, n_sink_chunks,
                                                 n_recent_chunks, draft_K, draft_V,
                                                 n_layers, n_kv_heads, head_dim, prefix_len, chunk_size,
                                                 stride_layer, stride_l, stride_h, idx, n_selected, K_out, V_out,
                                                 n_tokens_out, device_status, st);
  g_launches.fetch_add(1);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return SPECEXT_ERR_CUDA;
  }
  return SPECEXT_OK;
}

int specext_read_status(const int32_t* device_status, void* cuda_stream) {
  if (!device_status) return -SPECEXT_ERR_INVALID_ARG;
  int32_t h = 0;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(&h, device_status, sizeof(h), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) {
    (void)cudaGetLastError();
    return -SPECEXT_ERR_CUDA;
  }
  return h;
}

const char* specext_status_string(int status) {
  switch (status) {
    case SPECEXT_OK: return "ok";
    case SPECEXT_ERR_INVALID_ARG: return "invalid argument";
    case SPECEXT_ERR_UNSUPPORTED: return "unsupported shape";
    case SPECEXT_ERR_WORKSPACE: return "workspace too small";
    case SPECEXT_ERR_BAD_TREE: return "parent[] is not a topologically ordered forest";
    case SPECEXT_ERR_TIMEOUT: return "bounded device wait expired";
    case SPECEXT_ERR_CUDA: return "CUDA call failed";
    default: return "unknown status";
  }
}

int64_t specext_launch_count(void) { return g_launches.load(); }


#ifdef SPECEXT_TESTING
// Test library only: forces an attention kernel / a lower bound on key tiles per worker for every
// later call in the process (see testing.h).
int specext_test_set_tuning(int32_t attn_kernel, int32_t min_tiles_per_cta) {
  if (attn_kernel < 0 || attn_kernel > 3 || min_tiles_per_cta < 0) return SPECEXT_ERR_INVALID_ARG;
  g_attn_kernel.store(attn_kernel);
  if (min_tiles_per_cta > 0) g_min_units.store(min_tiles_per_cta);
  return SPECEXT_OK;
}
#endif

}  // extern "C"
