/*
 * specext.h -- C ABI of the verification hot path of speculative decoding with Cross-model
 * Retrieval: Hybrid Tree Attention fused with the per-chunk attention mass that retrieval ranks,
 * top-k chunk selection, and the gather that rewrites the draft model's KV cache.
 *
 * General conventions
 *   - Every data pointer is a DEVICE pointer owned by the caller.  The library never allocates,
 *     frees or synchronises on these calls; all work is enqueued on `cuda_stream` (a cudaStream_t
 *     passed as void*, NULL = the legacy default stream) and the call returns at once.
 *   - The return value is the result of synchronous host-side argument checking (a
 *     specext_status).  Problems only the device can see (an invalid parent[] entry, a bounded
 *     wait that ran out) are OR-ed as (1 << status) into *device_status, an int32 in device
 *     memory that the caller zeroes once and may read after synchronising; outputs are then
 *     unspecified, but every kernel terminates.
 *   - bf16 tensors are raw 16-bit patterns.  The innermost dimension (head_dim) is contiguous;
 *     all other strides are given in elements, must be multiples of 8 elements (16 bytes), and
 *     base pointers must be 16-byte aligned.
 *   - Query head h reads KV head h / (n_q_heads / n_kv_heads).
 *   - Calls that share a workspace or outputs must be ordered by the stream.
 *   - No call keeps state between calls or changes process-wide settings; a process may use the
 *     library on several devices (the device current at the call is the one used).
 *   - The kernels of these calls are launched with programmatic stream serialization, so
 *     that the set-up of one overlaps the tail of the one before it in the stream; each of them
 *     waits for that predecessor to complete (and its writes to be visible) before it reads or
 *     writes global memory, so the stream order the caller sees is the usual one.  The calls can
 *     be captured into CUDA graphs.
 */
#ifndef SPECEXT_H_
#define SPECEXT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SPECEXT_OK = 0,
  SPECEXT_ERR_INVALID_ARG = 1, /* null / misaligned pointer, size or stride out of range        */
  SPECEXT_ERR_UNSUPPORTED = 2, /* shape outside what the kernels are built for                   */
  SPECEXT_ERR_WORKSPACE = 3,   /* workspace_bytes smaller than specext_verify_attn_workspace()   */
  SPECEXT_ERR_BAD_TREE = 4,    /* device: parent[i] outside [-1, i-1]                            */
  SPECEXT_ERR_TIMEOUT = 5,     /* device: a bounded wait inside a kernel expired                 */
  SPECEXT_ERR_CUDA = 6         /* a CUDA runtime / driver call failed (launch, tensor map, ...)  */
} specext_status;

/* Shape of one verification attention call (one layer, one sequence). */
typedef struct {
  int32_t n_q_heads;       /* Hq                                                              */
  int32_t n_kv_heads;      /* Hkv; Hq % Hkv == 0 and G = Hq/Hkv a power of two <= 64          */
  int32_t head_dim;        /* D: 64 or 128                                                    */
  int32_t prefix_len;      /* L >= 0: number of valid tokens in the prefix KV cache           */
  int32_t n_tree;          /* T: draft-tree nodes, 1..128                                     */
  int32_t chunk_size;      /* C: tokens per retrieval chunk, a power of two in 1..128         */
  float softmax_scale;     /* multiplies q.k before the softmax; 0 selects 1/sqrt(D)          */
  int32_t want_chunk_score;/* non-zero: also produce chunk_score (the last layer only)        */
  int64_t q_stride_t, q_stride_h;     /* Q      [T][Hq][D]                                    */
  int64_t kv_stride_l, kv_stride_h;   /* K_prefix and V_prefix [>=L][Hkv][D], same strides    */
  int64_t tkv_stride_t, tkv_stride_h; /* K_tree and V_tree [T][Hkv][D], same strides          */
  int64_t o_stride_t, o_stride_h;     /* O      [T][Hq][D]                                    */
} specext_attn_desc;

/*
 * Bytes of scratch that specext_verify_attn needs for this shape (0 on an invalid descriptor).
 * The scratch holds the per-split partial results of the split-over-KV attention and is fully
 * rewritten by every call; 256-byte alignment is required.
 */
size_t specext_verify_attn_workspace(const specext_attn_desc* desc);

/*
 * Hybrid Tree Attention of the target model's verification step (Section 3.1, "Efficient
 * Attention") together with the attention scores that Cross-model Retrieval ranks chunks by
 * (Section 3.2.1, "Method Overview"; the scores of the last layer of the most recent
 * verification pass).
 *
 * For every tree node t and query head h, with g = h / G:
 *   s_j = scale * <Q[t,h], K_prefix[j,g]>            for the L prefix tokens,
 *   s_u = scale * <Q[t,h], K_tree[u,g]>              for tree nodes u that are t itself or an
 *                                                    ancestor of t (others are masked out),
 *   P = softmax over all visible keys, O[t,h] = sum P * V, lse[h,t] = log sum exp(s),
 *   chunk_score[t,c] = (1/Hq) * sum_h sum_{j in chunk c} P_j,  chunk c = tokens [cC, min(L,(c+1)C)).
 * The prefix is processed in splits along the KV length with an online softmax and the partial
 * results are merged by log-sum-exp, so the result equals unsplit attention up to rounding.
 *
 *   Q, K_prefix, V_prefix, K_tree, V_tree : bf16, layouts as in the descriptor.  Memory of the
 *       prefix cache beyond prefix_len is never read.
 *   parent      : int32 [T]; parent[i] is the tree index of node i's parent, -1 when the parent is
 *                 the last prefix token.  Must satisfy -1 <= parent[i] < i (else BAD_TREE).
 *   O           : bf16 [T][Hq][D] (strides from the descriptor), rounded once from fp32.
 *   lse         : fp32 [Hq][T], natural logarithm, softmax_scale included.
 *   chunk_score : fp32 [T][ceil(L/C)], written only when want_chunk_score != 0 (may be NULL
 *                 otherwise).
 *   workspace   : scratch of at least specext_verify_attn_workspace(desc) bytes.
 * Arithmetic: bf16 products accumulated in fp32; probabilities are rounded to bf16 for the
 * P*V product; chunk sums and the normaliser are accumulated in fp32 from unrounded exponentials.
 */
int specext_verify_attn(const specext_attn_desc* desc, const void* Q, const void* K_prefix,
                        const void* V_prefix, const void* K_tree, const void* V_tree,
                        const int32_t* parent, void* O, float* lse, float* chunk_score,
                        void* workspace, size_t workspace_bytes, int32_t* device_status,
                        void* cuda_stream);

/*
 * SelectChunks of Algorithm 1 (Appendix A; Section 3.2.1: rank the fixed-size chunks of the
 * prefix by their average attention score for one query and keep the top k).
 *
 *   chunk_score : fp32 [n_tree][n_chunks] as written by specext_verify_attn.
 *   row         : which tree node's scores to rank (the last accepted token), 0 <= row < n_tree.
 *   prefix_len, chunk_size : define n_chunks = ceil(L/C) (must equal the argument) and the
 *                 length len_c of the trailing chunk.  Any chunk_size >= 1 is accepted.
 *   k           : number of chunks to keep, >= 1; k_eff = min(k, n_chunks).
 *   n_sink_chunks, n_recent_chunks : 0 and 0 for the paper's retrieval, which forces nothing.  As an
 *                 extension the first n_sink_chunks and the last n_recent_chunks chunks are kept
 *                 whatever their score: they rank above all others (lower index first among
 *                 themselves) and the remaining places go to the best of the rest.
 *   idx         : int32 [min(k, n_chunks)] out, the kept chunk indices in ascending order.
 *   n_selected  : int32 [1] out (device), = k_eff.
 * Ranking key: chunk_score[row][c] / (float)len_c in fp32 (IEEE division); larger first, equal
 * keys ordered by lower chunk index.  Scores must be finite and non-negative.
 * n_chunks <= 65536.
 */
int specext_select_chunks(const float* chunk_score, int32_t n_tree, int32_t n_chunks, int32_t row,
                          int32_t prefix_len, int32_t chunk_size, int32_t k, int32_t n_sink_chunks,
                          int32_t n_recent_chunks, int32_t* idx, int32_t* n_selected,
                          int32_t* device_status, void* cuda_stream);

/*
 * UpdateDraftCache of Algorithm 1 (Appendix A; Section 3.2.1: the draft model keeps only the
 * selected chunks in its KV cache).  Copies the selected chunks of the draft model's K and V,
 * bit for bit and in the order of idx, into a compact cache.
 *
 *   draft_K, draft_V : bf16 [n_layers][>=L][n_kv_heads][head_dim] with element strides
 *                      stride_layer, stride_l, stride_h (head_dim contiguous).
 *   idx, n_selected  : device outputs of specext_select_chunks (ascending chunk indices, each in
 *                      [0, ceil(L/C)) -- entries outside that range are skipped and reported as
 *                      INVALID_ARG in *device_status).
 *   max_selected     : upper bound on *n_selected that sizes the launch (the k passed to select).
 *   K_out, V_out     : bf16 [n_layers][max_selected*C][n_kv_heads][head_dim], contiguous; token
 *                      slot i*C + o receives token idx[i]*C + o.  Only a trailing chunk can be
 *                      short, and it can only come last, so the valid tokens are contiguous.
 *   n_tokens_out     : int32 [1] out (device): number of valid tokens written per layer.
 * n_kv_heads * head_dim must be a multiple of 8 (16-byte vectors).
 */
int specext_gather_kv(const void* draft_K, const void* draft_V, int32_t n_layers,
                      int32_t n_kv_heads, int32_t head_dim, int32_t prefix_len, int32_t chunk_size,
                      int64_t stride_layer, int64_t stride_l, int64_t stride_h, const int32_t* idx,
                      const int32_t* n_selected, int32_t max_selected, void* K_out, void* V_out,
                      int32_t* n_tokens_out, int32_t* device_status, void* cuda_stream);

/*
 * Attention of the DRAFT model over the compact cache that UpdateDraftCache wrote (Section 3.2.1,
 * "Method Overview": the draft model generates its candidate tokens on the reduced cache of the
 * selected chunks; Appendix D: about 1K to 2K tokens).  The arithmetic is that of
 * specext_verify_attn -- tree nodes (or a single decode token, n_tree = 1) attend to the cached
 * tokens and to their own ancestors, split over the KV length and merged by log-sum-exp -- but
 * the number of cached tokens is read ON THE DEVICE, so that select -> gather -> draft attention
 * replay as one CUDA graph with no host round trip in between.
 *
 *   desc->prefix_len : capacity of the compact cache in tokens (k * chunk_size), the upper bound of
 *                      *n_tokens; desc->want_chunk_score must be 0; desc->chunk_size is not used
 *                      (give any valid value).
 *   K_cache, V_cache : bf16 [>= capacity][n_kv_heads][head_dim], strides desc->kv_stride_*, e.g. one
 *                      layer of the K_out / V_out of specext_gather_kv.
 *   n_tokens         : int32 [1] in DEVICE memory (the n_tokens_out of specext_gather_kv); values
 *                      outside [0, capacity] are clamped.  Cache rows at and beyond *n_tokens are
 *                      never used, whatever they hold (NaN included).
 *   everything else  : as in specext_verify_attn; the workspace size is
 *                      specext_verify_attn_workspace(desc).
 * The work is laid out for the capacity; with a shorter cache some thread blocks find nothing to do.
 */
int specext_draft_attn(const specext_attn_desc* desc, const void* Q, const void* K_cache,
                       const void* V_cache, const int32_t* n_tokens, const void* K_tree,
                       const void* V_tree, const int32_t* parent, void* O, float* lse, void* workspace,
                       size_t workspace_bytes, int32_t* device_status, void* cuda_stream);

/*
 * Prefill: causal self-attention over the L tokens of the prompt (Section 3.1, "Efficient
 * Attention": the prefill stage of the target and of the draft model runs a tiled attention that
 * never forms the L x L score matrix).  For every token i and query head h, with g = h / G:
 *   s_j = scale * <Q[i,h], K[j,g]> for j <= i,  P = softmax(s),  O[i,h] = sum_j P_j V[j,g],
 *   lse[h,i] = log sum_j exp(s_j).
 * One kernel, no scratch memory: a block of 256/G consecutive tokens of one KV head (256 stacked
 * query rows) is processed from its first to its last key tile by one pair of SMs, so nothing is
 * split and nothing has to be merged.
 *
 *   desc  : n_q_heads, n_kv_heads, head_dim, softmax_scale and the strides q_stride_*, kv_stride_*,
 *           o_stride_* are used; prefix_len is L >= 1, the number of prompt tokens; the other
 *           fields are ignored.  head_dim must be 128 (UNSUPPORTED otherwise).
 *   Q     : bf16 [L][Hq][D];  K, V : bf16 [>=L][Hkv][D], same strides;  O : bf16 [L][Hq][D];
 *   lse   : fp32 [Hq][L], natural logarithm, softmax_scale included.
 * Arithmetic as in specext_verify_attn.  The first retrieval after the prefill (Algorithm 1 runs
 * SelectChunks / UpdateDraftCache before the first Draft) takes its scores from one
 * specext_verify_attn call of the last layer with the last prompt token as a single tree node
 * (n_tree = 1, parent = -1) over the prefix of the L - 1 tokens before it.
 */
int specext_prefill_attn(const specext_attn_desc* desc, const void* Q, const void* K, const void* V,
                         void* O, float* lse, int32_t* device_status, void* cuda_stream);

/*
 * SelectChunks followed by UpdateDraftCache (the two steps Algorithm 1 runs back to back when
 * doRetrieval is set) as ONE call: the same results, in idx, n_selected, K_out, V_out and
 * n_tokens_out, as specext_select_chunks(..., k, n_sink_chunks, n_recent_chunks, ...) followed by specext_gather_kv(...,
 * max_selected = k, ...), argument for argument.  For n_chunks <= 8192 and k <= 1024 it is a single
 * kernel launch (every thread block repeats the deterministic selection and copies its share of the
 * kept chunks, so no block waits for another); larger sizes run the two kernels.
 */
int specext_select_gather(const float* chunk_score, int32_t n_tree, int32_t n_chunks, int32_t row,
                          int32_t prefix_len, int32_t chunk_size, int32_t k, int32_t n_sink_chunks,
                          int32_t n_recent_chunks, const void* draft_K,
                          const void* draft_V, int32_t n_layers, int32_t n_kv_heads, int32_t head_dim,
                          int64_t stride_layer, int64_t stride_l, int64_t stride_h, int32_t* idx,
                          int32_t* n_selected, void* K_out, void* V_out, int32_t* n_tokens_out,
                          int32_t* device_status, void* cuda_stream);

/*
 * Copies *device_status to the host after synchronising the stream and returns it (a bit set of
 * 1 << specext_status), or -SPECEXT_ERR_CUDA if the copy failed.  For tests and debugging; not
 * part of the asynchronous path.
 */
int specext_read_status(const int32_t* device_status, void* cuda_stream);

/* Static, human-readable name of a specext_status value. */
const char* specext_status_string(int status);

/* Number of kernels the library has launched in this process (all calls, all streams). */
int64_t specext_launch_count(void);

/*
 * specext_verify_attn for callers that cannot allocate device memory (the paper has no counterpart).
 *
 * Some callers have nowhere to get the scratch buffer from: code that runs after the process has
 * handed all device memory to a pool it does not own, plug-ins that are forbidden to call
 * cudaMalloc, or a recovery path that must keep working when the allocator has failed.  This entry
 * point takes the same inputs and outputs as specext_verify_attn but no workspace: the scratch is a
 * fixed array of SPECEXT_STATIC_SCRATCH_BYTES that is part of the library image, so every GPU
 * that loads the library holds that much memory until the process exits.
 *
 *   - Shapes whose scratch need (specext_verify_attn_workspace) exceeds
 *     SPECEXT_STATIC_SCRATCH_BYTES are rejected with SPECEXT_ERR_WORKSPACE; nothing is launched.
 *   - The call allocates nothing: no cudaMalloc / cudaFree and no allocating library routine.
 *   - The first call on each device looks up the device address of the array (with that device
 *     current) and caches it; that look-up may be what makes the driver load the array onto the
 *     device.  Make that first call at start-up: outside of any stream capture, and while the
 *     device still has SPECEXT_STATIC_SCRATCH_BYTES to spare (a caller whose allocator has already
 *     failed cannot count on a first call succeeding).
 *   - All calls on a device share the one array.  Calls must therefore not overlap on the GPU:
 *     order them on one stream (or by events); two calls running concurrently race on the scratch
 *     and both produce garbage.  Nothing in the array has to survive from one call to the next and
 *     nothing has to start at zero: every call rewrites the part it reads.
 * Arguments, outputs, arithmetic and error reporting are those of specext_verify_attn.
 */
#define SPECEXT_STATIC_SCRATCH_BYTES (32u << 20)
int specext_verify_attn_static_scratch(const specext_attn_desc* desc, const void* Q,
                                       const void* K_prefix, const void* V_prefix,
                                       const void* K_tree, const void* V_tree,
                                       const int32_t* parent, void* O, float* lse,
                                       float* chunk_score, int32_t* device_status,
                                       void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SPECEXT_H_ */
