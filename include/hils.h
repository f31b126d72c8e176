/*
 * hils.h -- C ABI of the B200 (sm_100a) HiLS attention library.
 *
 * HiLS (Hierarchical Landmark Sparse) attention, forward pass.  For a query at
 * position i (0-based) with chunk size S and local window W:
 *
 *   Sec. 2.1   l(i) = max(0, floor((i - W + 1) / S)) * S is the chunk-aligned left edge of the
 *              local window; candidate chunks are C_i = {0 .. l(i)/S - 1}.
 *   Eq. (surrogate top-k), App. C Eq. (HiLS GQA)
 *              per-head surrogate score  s^h_c = scale * q^h . k'_c + b'_c  against the landmark
 *              (chunk summary key) k'_c and bias b'_c of every candidate chunk; group score
 *              u_c = max over the query heads of one KV group; the min(K, |C_i|) chunks with the
 *              largest u_c are selected for the whole group (equal scores: lower chunk id wins).
 *   Eq. (chunk mass)   local branch: causal softmax over tokens l(i)..i, with mass Z_swa.
 *   Eq. (HiLS weights) each selected chunk is attended with its own softmax over its S tokens;
 *              the per-chunk outputs and the local output are mixed with
 *              softmax({s^h_c : c selected} U {log Z_swa}) -- per head.
 *              lse = log( sum_c exp(s^h_c) + Z_swa ).
 *
 * Around the operator (each documented at its declaration): the chunk summaries that produce
 * landmarks / bias (Proposition 3.1, hils_landmark_summary); the operator on a slice of a sequence, on paged
 * caches, with a separate routing query (Eq. Q-Cal) and for several new tokens per sequence
 * (hils_prefill_at, hils_decode_paged, hils_*_routed, hils_decode_multi); the overlap statistic of adjacent
 * queries (Sec. "Chunk Overlap", hils_chunk_overlap); the backward pass through `out`
 * (hils_prefill_backward); host-buffer variants and an allocation-free decode.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer owned by the caller unless the entry point says HOST.
 *   - The library never allocates, frees or synchronises; all work is enqueued on `stream`.  Outputs are fully
 *     overwritten.  The exceptions say so at their declarations: hils_prefill_host / hils_decode_host (three
 *     internal streams and ten events per device, created on first use, and a process-wide mutex around a call),
 *     hils_trace_enable (1025 events on first use), hils_trace_read and hils_poll_status (they wait for the stream).
 *   - Tensors are contiguous, last dimension fastest, base pointers 16-byte aligned:
 *       q, out      [B, Hq, L, d]          (decode: [B, Hq, d])
 *       k, v        [B, Hkv, T, d]         T = L for prefill, T_max for decode
 *       landmarks   [B, Hl, C, d]          C = params.C rows per landmark head; row c is only read
 *                                          when chunk c is complete and precedes the local window
 *       bias        [B, Hl, C] fp32 or NULL (NULL means 0)
 *       lse         [B, Hq, L] fp32        (decode: [B, Hq])
 *       sel_idx     [B, Hkv, L, K] int32   (decode: [B, Hkv, K]) ascending chunk ids, -1 padded
 *       seq_lens    [B] int32              decode: tokens in the cache INCLUDING the new one; the
 *                                          query sits at position seq_lens[b]-1, 1 <= seq_lens <= T_max
 *   - Argument errors are found on the host and returned before anything is launched.
 *     Device-side anomalies (a wait that ran out, an out-of-range chunk id) set a status word in
 *     the workspace (read it with hils_poll_status); kernels never trap.
 *   - Status codes are negative on error; no exception crosses this boundary.
 */
#ifndef HILS_H_
#define HILS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    HILS_OK = 0,
    HILS_ERR_INVALID_ARG = -1,   /* null pointer, non-positive size, Hq % Hkv != 0, ...           */
    HILS_ERR_UNSUPPORTED = -2,   /* a shape or option this build has no kernel for                */
    HILS_ERR_ALIGNMENT = -3,     /* a base pointer is not 16-byte aligned                         */
    HILS_ERR_WORKSPACE = -4,     /* workspace missing or smaller than hils_workspace_bytes()      */
    HILS_ERR_CUDA = -5,          /* a CUDA runtime call failed (launch, copy, attribute)          */
    HILS_ERR_DEVICE_TIMEOUT = -6,/* a bounded device-side wait ran out                            */
    HILS_ERR_DEVICE_INDEX = -7   /* a kernel met a chunk id outside its valid range               */
} hils_status;

typedef enum { HILS_F32 = 0, HILS_BF16 = 1 } hils_dtype;

/* Which implementation to run.  AUTO picks the fastest kernel set that supports the shape;
 * GENERIC forces the shape-agnostic CUDA-core kernels (any d multiple of 32 up to 256,
 * any chunk size up to 128, any window).  PACKED (prefill only; never chosen by AUTO) is the query-major kernel of
 * Sec. 4.2 / App. "Chunk Overlap": tiles of 16 adjacent tokens x the query heads of a KV group walk the union of the
 * chunks the tokens selected, pairs (token, chunk) that were not selected are masked, and the retrieval-weighted mix
 * stays in registers until `out` is written once.  Its work grows with the size of that union, so it pays only where
 * adjacent queries select nearly the same chunks; bf16, d = 128, chunk_size = 64, Hq = 4 Hkv, Hl = Hkv, top_k <= 32,
 * at most 4096 chunks per sequence, slice offsets that are multiples of 16; other shapes return
 * HILS_ERR_UNSUPPORTED.  Same results as the other kernels up to the order of the fp32 sums. */
typedef enum { HILS_IMPL_AUTO = 0, HILS_IMPL_GENERIC = 1, HILS_IMPL_FAST = 2, HILS_IMPL_PACKED = 3 } hils_impl;

typedef struct hils_params {
    int32_t B, Hq, Hkv;
    int32_t Hl;          /* landmark heads: Hkv (one landmark per chunk per KV head) or Hq          */
    int32_t L;           /* prefill: number of query tokens == number of kv tokens; decode: ignored */
    int32_t T_max;       /* kv tokens allocated per (b, kv head); prefill: 0 means L                */
    int32_t C;           /* landmark rows allocated per (b, landmark head); 0 means T / chunk_size  */
    int32_t d;           /* head dimension                                                          */
    int32_t chunk_size;  /* S                                                                       */
    int32_t top_k;       /* K                                                                       */
    int32_t window;      /* W of Sec. 2.1; 1 = the query's own chunk is the local region            */
    float   scale;       /* logit scale; 0 means 1/sqrt(d)                                          */
    int32_t dtype;       /* hils_dtype of q, k, v, landmarks, out                                   */
    int32_t impl;        /* hils_impl                                                               */
} hils_params;

/* Bytes of device scratch hils_prefill (is_decode = 0) or hils_decode (is_decode = 1) needs for
 * these parameters.  Returns 0 if the parameters are invalid.  The first 256 bytes hold the
 * device status word; the caller must zero them once after allocation.
 * Prefill on the tensor-core path keeps per-(token, retrieved chunk) partial outputs in the workspace:
 * (K + window chunks) * Hq * d * 2 bytes per token, for all tokens of the call while that is at most 4 GiB
 * (2.3 GB for 16K tokens, 32 heads, K = 16), else for one block of 4096-8192 tokens at a time. */
size_t hils_workspace_bytes(const hils_params* params, int is_decode);

/* Prefill: Eq. (surrogate top-k) + Eq. (HiLS weights) (GQA form: App. C) for all L positions of
 * every sequence.  `lse` and `sel_idx` may not be NULL.  Asynchronous on `stream`
 * (a cudaStream_t passed as void*). */
int hils_prefill(const hils_params* params, const void* q, const void* k, const void* v,
                 const void* landmarks, const float* bias,
                 void* out, float* lse, int32_t* sel_idx,
                 void* workspace, size_t workspace_bytes, void* stream);

/* Decode: the same operator for one query per sequence at position seq_lens[b]-1 over a contiguous
 * KV cache that already holds the new token's k and v (the query attends to itself through the
 * local branch, Sec. 2.1: j <= i).  The query's own, possibly partial, chunk is local; only
 * complete earlier chunks are candidates. */
int hils_decode(const hils_params* params, const void* q, const void* k_cache, const void* v_cache,
                const void* landmarks, const float* bias, const int32_t* seq_lens,
                void* out, float* lse, int32_t* sel_idx,
                void* workspace, size_t workspace_bytes, void* stream);

/* hils_decode for callers that cannot allocate device memory.  (The paper has no counterpart to this
 * entry point; it exists for integration only.)
 *
 * Some hosts of this library have no way to hand it a workspace: an inference server that gave all
 * free HBM to its own KV-cache pool at start-up, so that a later cudaMalloc fails; a plugin that is
 * only passed the tensors of one layer and has no allocator handle; a latency-critical loop that
 * may not call cudaMalloc because it synchronises the device.  For them this call computes exactly
 * what hils_decode computes (same kernels, same results) but keeps its scratch in a fixed 16 MiB array
 * that is part of the library image itself; every GPU that loads libhils.so holds that array until
 * the process exits.  The caller still passes every input and output.
 *
 *  - Nothing is allocated or freed, by CUDA or otherwise, on any call.
 *  - Limit: the decode workspace of the shape, hils_workspace_bytes(params, 1) (its 256-byte status block
 *    included), must fit in 16 MiB, otherwise HILS_ERR_WORKSPACE is returned before anything is launched (both benchmark decode shapes fit: B=64 x 64K tokens with
 *    K=32 needs about 13.7 MiB, B=4 x 1M tokens with K=64 about 10.9 MiB; most of it is the table of per-head
 *    landmark scores, B x Hq x C floats).  Shapes outside the
 *    bandwidth-tuned decode kernels (bf16, d=128, chunk 64, window <= 897, one landmark per KV or per query head,
 *    at most 8 query heads per KV head) return HILS_ERR_UNSUPPORTED.
 *  - The first call on each device looks up the array's device address (with that device current);
 *    make that first call outside any stream capture.
 *  - The array is shared by every call in the process and keeps the previous call's contents.  The
 *    call clears what has to start at zero (the status word; the completion counters are reset by the
 *    kernels themselves).  Two calls whose kernels overlap on the GPU (different streams, or several
 *    host threads) race on it: serialise them.
 *  - device_status (DEVICE pointer, may be NULL) receives the device status word of this call:
 *    0 = ok, 1 = a bounded wait ran out, 2 = an invalid sequence length was met. */
int hils_decode_noalloc(const hils_params* params, const void* q, const void* k_cache, const void* v_cache,
                        const void* landmarks, const float* bias, const int32_t* seq_lens,
                        void* out, float* lse, int32_t* sel_idx, int32_t* device_status, void* stream);

/* The operators with a separate ROUTING QUERY q-hat (Eq. Q-Cal: q-hat = q + W_up W_down h, computed upstream by
 * the model).  q_route has the shape, dtype and alignment of q; it takes q's place in the surrogate scores
 * s^h_c = scale * q-hat^h . k'_c + b'_c -- i.e. in the selection and in the fusion weights -- and nowhere else
 * (token-level attention inside the selected chunks and the local window uses q).  Everything else as
 * hils_prefill / hils_decode, same workspace. */
int hils_prefill_routed(const hils_params* params, const void* q, const void* q_route, const void* k, const void* v,
                        const void* landmarks, const float* bias, void* out, float* lse, int32_t* sel_idx,
                        void* workspace, size_t workspace_bytes, void* stream);
int hils_decode_routed(const hils_params* params, const void* q, const void* q_route, const void* k_cache,
                       const void* v_cache, const void* landmarks, const float* bias, const int32_t* seq_lens,
                       void* out, float* lse, int32_t* sel_idx, void* workspace, size_t workspace_bytes,
                       void* stream);

/* hils_prefill for a SLICE of a sequence: the L query tokens sit at positions pos0 .. pos0 + L - 1 of sequences
 * whose caches already hold at least pos0 + L tokens (chunked prefill; with small L, multi-token decode as used by
 * speculative decoding).  Same operator: query row r is treated exactly like position pos0 + r of hils_prefill.
 *   q, out   [B, Hq, L, d]      lse [B, Hq, L]      sel_idx [B, Hkv, L, K]
 *   k, v     [B, Hkv, T, d]     T = params->T_max >= pos0 + L (row j is the token at position j)
 *   landmarks [B, Hl, C, d], bias [B, Hl, C]: rows of all chunks left of the last query's window
 * pos0 = 0 with T_max = L is hils_prefill.  The workspace depends on pos0: size it with
 * hils_prefill_at_workspace_bytes (0 = unsupported or invalid).  Errors as hils_prefill; pos0 < 0 or
 * pos0 + L > T_max returns HILS_ERR_INVALID_ARG. */
size_t hils_prefill_at_workspace_bytes(const hils_params* params, int64_t pos0);
int hils_prefill_at(const hils_params* params, const void* q, const void* k, const void* v, const void* landmarks,
                    const float* bias, int64_t pos0, void* out, float* lse, int32_t* sel_idx, void* workspace,
                    size_t workspace_bytes, void* stream);

/* hils_decode over PAGED caches with page = chunk (the serving layout of Sec. 7.1: one KV page per chunk).
 * Same operator, same outputs as hils_decode; only the addressing of K and V differs:
 *   k_pages, v_pages [num_pages, Hkv, S, d]  DEVICE: page p holds S consecutive tokens of one sequence for all KV heads
 *   block_table      [B, C] int32 DEVICE: page of logical chunk c of sequence b (read for the chunks that are
 *                    attended: c <= (seq_lens[b]-1)/S); params->C is its row length, params->T_max = C * S
 *   landmarks, bias  stay logical: [B, Hl, C, d] / [B, Hl, C]
 * A page id outside [0, num_pages) sets the device status to HILS_ERR_DEVICE_INDEX and the chunk is skipped.
 * Supported by the bandwidth-tuned decode kernels only (bf16, d = 128, S = 64, at most 8
 * query heads per KV head); other shapes return HILS_ERR_UNSUPPORTED.  Workspace as for hils_decode. */
int hils_decode_paged(const hils_params* params, const void* q, const void* k_pages, const void* v_pages,
                      const void* landmarks, const float* bias, const int32_t* block_table, int32_t num_pages,
                      const int32_t* seq_lens, void* out, float* lse, int32_t* sel_idx, void* workspace,
                      size_t workspace_bytes, void* stream);

/* Multi-token decode: M = tokens_per_seq new tokens per sequence in one call (speculative decoding, verification
 * of draft tokens; Sec. "Hardware-Efficient Kernel Design" names it as a use of packing adjacent queries).  The
 * caches already hold all M new tokens; token m of sequence b sits at position seq_lens[b] - M + m and is
 * treated exactly like a single-token hils_decode at length seq_lens[b] - M + m + 1: the call runs the decode
 * kernels over B * M queries that share the caches, landmarks and bias of their sequence.
 *
 *   q        [B, M, Hq, d]     DEVICE        out     [B, M, Hq, d]
 *   lse      [B, M, Hq] fp32                 sel_idx [B, M, Hkv, K] int32
 *   seq_lens [B] int32 DEVICE: lengths INCLUDING the M new tokens (a sequence with seq_lens[b] < M has tokens
 *            at negative positions: those queries get zero output and the device status is set)
 *   k_cache, v_cache, landmarks, bias: as for hils_decode ([B, ...], params->B = B); with block_table != NULL
 *            they are page pools addressed as in hils_decode_paged ([B, C] table, shared by the M queries)
 * Supported by the bandwidth-tuned decode kernels only (bf16, d = 128, S = 64, at most 8 query heads per KV
 * head): other shapes, and params->impl = HILS_IMPL_GENERIC, return HILS_ERR_UNSUPPORTED (use hils_prefill_at).
 * Workspace: hils_decode_multi_workspace_bytes(params, M).  Errors as for hils_decode. */
size_t hils_decode_multi_workspace_bytes(const hils_params* params, int32_t tokens_per_seq);
int hils_decode_multi(const hils_params* params, int32_t tokens_per_seq, const void* q, const void* k_cache,
                      const void* v_cache, const void* landmarks, const float* bias, const int32_t* block_table,
                      int32_t num_pages, const int32_t* seq_lens, void* out, float* lse, int32_t* sel_idx,
                      void* workspace, size_t workspace_bytes, void* stream);

/* Chunk summaries -- the step upstream of the operator (Proposition 3.1, Eq. LogSumExp linearization /
 * Eq. prop_q_c).  For every sequence b, landmark head hl (its KV head is hl / (Hl / Hkv)) and chunk
 * c in [chunk_begin, chunk_begin + chunk_count), with the chunk's keys k_j, j in [c*S, min((c+1)*S, len_b))
 * and its learnable query q'_c = landmark_queries[b, hl, c, :]:
 *     s_j = scale * q'_c . k_j,   p = softmax_j(s),
 *     landmarks[b, hl, c, :] = k'_c = sum_j p_j k_j        (Attn(q'_c, K_c, K_c)),
 *     bias[b, hl, c]         = b'_c = - sum_j p_j log p_j  (entropy of p),
 * i.e. the `landmarks` / `bias` inputs of hils_prefill and hils_decode.  A chunk without tokens gets
 * zeros; a partial last chunk uses the tokens it has.  Serving code calls this for the chunk that has
 * just been completed (chunk_count = 1); prefill calls it for all chunks (chunk_count <= 0 means "up to C").
 *
 *   landmark_queries [B, Hl, C, d]  DEVICE, params->dtype
 *   k                [B, Hkv, T, d] DEVICE, params->dtype, T = params->T_max if > 0, else params->L
 *   seq_lens         [B] int32 DEVICE or NULL (NULL: every sequence holds T tokens)
 *   landmarks        [B, Hl, C, d]  DEVICE, params->dtype (written for the requested chunks only)
 *   bias             [B, Hl, C] fp32 DEVICE (same)
 * Uses of params: B, Hkv, Hl, C, d, chunk_size (<= 128), scale, dtype, T_max / L; d a multiple of 32, <= 256.
 * Needs no workspace; one kernel is enqueued on `stream`.  Errors: HILS_ERR_INVALID_ARG (null pointer, bad
 * range or size), HILS_ERR_ALIGNMENT, HILS_ERR_UNSUPPORTED (d or chunk size outside the limits), HILS_ERR_CUDA. */
int hils_landmark_summary(const hils_params* params, const void* landmark_queries, const void* k,
                          const int32_t* seq_lens, int32_t chunk_begin, int32_t chunk_count, void* landmarks,
                          float* bias, void* stream);

/* Chunk-id overlap among adjacent queries (Sec. "Chunk Overlap", Eq. Overlap) -- the statistic behind packing M
 * adjacent queries over the union of their chunks.  Queries r*M .. r*M + M - 1 of one (sequence, KV head) pair
 * form block r (M = block_queries; a trailing block holds the L mod M queries left); I_m is the set of chunk
 * ids in the K slots of its m-th query (ids outside [0, C), e.g. the -1 of an empty slot, are skipped).
 *
 *   sel_idx  [B, Hkv, L, K] int32 DEVICE, as written by hils_prefill / hils_prefill_at (L = params->L,
 *            K = params->top_k, C = params->C)
 *   stats    [B, Hkv, nblk, 4] int32 DEVICE, 16-byte aligned, nblk = ceil(L / M); per block
 *              [0] total  = sum_m |I_m|
 *              [1] union  = |union_m I_m|           (chunks a packed kernel loads once for the block)
 *              [2] reused = |union  intersected with  the previous block's union|   (0 for block 0)
 *              [3] full   = 1 if the block has M queries holding K chunks each, else 0
 *   overlap  [B, Hkv, nblk] fp32 DEVICE or NULL: (M K - union) / ((M - 1) K) where full = 1 and M > 1,
 *            NaN elsewhere (the equation is stated for M queries of K chunks)
 * Uses of params: B, Hkv, L, C (<= 2^19), top_k.  Needs no workspace; one kernel is enqueued on `stream`.
 * Errors: HILS_ERR_INVALID_ARG, HILS_ERR_ALIGNMENT, HILS_ERR_UNSUPPORTED (C too large), HILS_ERR_CUDA. */
int hils_chunk_overlap(const hils_params* params, const int32_t* sel_idx, int32_t block_queries, int32_t* stats,
                       float* overlap, void* stream);

/* Backward of hils_prefill through `out` (training; Sec. 3.2: the retrieval scores sit inside the forward
 * weights, so the loss reaches the landmarks).  The paper prints no backward equations; this is the chain rule
 * on Eq. (HiLS weights) / App. C with the selected set held fixed (top-K has no derivative), the routing query
 * equal to q, and no gradient through `lse`.  With alpha_c = exp(s^h_c - lse), p_j the softmax inside a slot,
 * w_j the final weight of key j (alpha_c p_j in a selected chunk, exp(s_j - lse) in the local span),
 * g_c = dout . o_c and D = dout . out:
 *     d s_j = w_j (dout . v_j - g_c)   (selected chunk)        d s_j = w_j (dout . v_j - D)   (local span)
 *     d lambda_c = alpha_c (g_c - D)
 *     dv_j += w_j dout,  dq += scale d s_j k_j,  dk_j += scale d s_j q,
 *     dq += scale d lambda_c k'_c,  dlandmarks_c += scale d lambda_c q,  dbias_c += d lambda_c.
 *
 *   q, k, v, landmarks, bias   as given to hils_prefill (params likewise)
 *   out, lse, sel_idx          as hils_prefill wrote them (out in params->dtype)
 *   dout            [B, Hq, L, d]   DEVICE, params->dtype: dLoss/dout
 *   dq              [B, Hq, L, d]   fp32 DEVICE, overwritten
 *   dk, dv          [B, Hkv, T, d]  fp32 DEVICE, overwritten (zeroed by the call, then accumulated)
 *   dlandmarks      [B, Hl, C, d]   fp32 DEVICE, same
 *   dbias           [B, Hl, C]      fp32 DEVICE or NULL, same
 * bf16 with d = 128, chunk_size = 64, four query heads per KV head and one landmark per KV head runs on the
 * 5th-generation tensor cores (chunk-major, accumulators in tensor memory); every other supported shape on
 * CUDA cores (params->impl selects as for hils_prefill).
 * All gradient pointers 16-byte aligned (dbias 4).  Sums over queries are accumulated with fp32 atomics, so
 * the last bits of dk, dv, dlandmarks, dbias may differ from run to run.  Workspace:
 * hils_prefill_backward_workspace_bytes (0 = unsupported shape); its head is the status word of
 * hils_poll_status.  Errors as for hils_prefill. */
size_t hils_prefill_backward_workspace_bytes(const hils_params* params);
int hils_prefill_backward(const hils_params* params, const void* q, const void* k, const void* v,
                          const void* landmarks, const float* bias, const void* out, const float* lse,
                          const int32_t* sel_idx, const void* dout, float* dq, float* dk, float* dv,
                          float* dlandmarks, float* dbias, void* workspace, size_t workspace_bytes, void* stream);

/* Bytes of device memory the *_host entry points need for staging (inputs + outputs + workspace). */
size_t hils_host_arena_bytes(const hils_params* params, int is_decode);

/* Same operators with HOST input and output buffers (pinned memory recommended).  Inputs are copied
 * to `device_arena` (a DEVICE buffer of at least hils_host_arena_bytes()), the device entry point
 * runs, and out / lse / sel_idx are copied back, all enqueued on `stream`.  The call returns
 * without synchronising: results are valid once the stream has been synchronised.  The arena's
 * first 256 bytes are the status word (zero them once). */
/* Sequences of at least 8192 tokens go through hils_prefill_host in blocks of 4096 tokens, the last 4096 cut into
 * 1/2, 1/4, 1/4 (the operator is causal: a block needs only the inputs up to its own end; the last block's
 * kernels and copy-out overlap nothing, so it is kept short): copy-in, kernels (hils_prefill_at) and copy-out of
 * neighbouring blocks overlap on three internal streams, created on first use, that fork from and join `stream`;
 * calls that take this route are serialised on the host by a mutex (their events are shared).  Results are those
 * of hils_prefill.  HILS_HOST_PIPELINE=0 in the environment keeps the single-stream form. */
int hils_prefill_host(const hils_params* params, const void* q_host, const void* k_host,
                      const void* v_host, const void* landmarks_host, const float* bias_host,
                      void* out_host, float* lse_host, int32_t* sel_idx_host,
                      void* device_arena, size_t arena_bytes, void* stream);
int hils_decode_host(const hils_params* params, const void* q_host, const void* k_cache_host,
                     const void* v_cache_host, const void* landmarks_host, const float* bias_host,
                     const int32_t* seq_lens_host,
                     void* out_host, float* lse_host, int32_t* sel_idx_host,
                     void* device_arena, size_t arena_bytes, void* stream);

/* Reads the device status word at the start of `workspace` (synchronises `stream`).
 * Returns HILS_OK, HILS_ERR_DEVICE_TIMEOUT, HILS_ERR_DEVICE_INDEX or HILS_ERR_CUDA. */
int hils_poll_status(const void* workspace, void* stream);

/* Number of kernels the last hils_prefill / hils_decode call of this thread enqueued. */
int hils_last_launch_count(void);

/* Per-kernel timing for profiling (no counterpart in the paper; Sec. 7.1 reports end-to-end latency
 * only).  hils_trace_enable(1) creates CUDA events once for the calling thread; while on, each
 * hils_prefill / hils_decode records an event after every kernel it enqueues.  hils_trace_read
 * waits for the last call's final event and returns the number of kernels n (<= max_kernels),
 * writing their device times to ms[0..n) and their names, ';'-terminated, to `names`. */
int hils_trace_enable(int on);
int hils_trace_read(char* names, size_t names_bytes, float* ms, int max_kernels);

const char* hils_status_string(int status);

/* Library version, "major.minor". */
const char* hils_version(void);

#ifdef __cplusplus
}
#endif
#endif /* HILS_H_ */
