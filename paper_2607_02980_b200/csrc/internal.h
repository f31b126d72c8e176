// Host-side launch functions shared between the translation units of the library.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "common.cuh"

namespace hils {

struct Tensors {
    const void* q;
    const void* k;
    const void* v;
    const void* landmarks;
    const float* bias;
    const int32_t* seq_lens;   // decode only
    void* out;
    float* lse;
    int32_t* sel_idx;
    int* status;               // device status word
    void* scratch;             // workspace past the status block
    size_t scratch_bytes;
    // paged decode (page = chunk): k, v are [num_pages, Hkv, S, d] and block_table [B, C] maps a sequence's
    // logical chunk to its page; NULL = contiguous caches
    const int32_t* block_table = nullptr;
    int num_pages = 0;
    // routing query q-hat (Eq. Q-Cal), same shape as q: used for the surrogate scores only; NULL = q
    const void* q_route = nullptr;
};

// Kernel attributes (the opt-in dynamic shared-memory size) belong to a device: a launcher sets them the first time
// it runs on each device of the process.  pending() is true until done() has been called on the current device.
struct PerDeviceOnce {
    bool set[64] = {};
    static int device() {
        int d = 0;
        return (cudaGetDevice(&d) == cudaSuccess && d >= 0 && d < 64) ? d : -1;
    }
    bool pending() const { const int d = device(); return d < 0 || !set[d]; }
    void done() { const int d = device(); if (d >= 0) set[d] = true; }
};

// Streaming multiprocessors of the current device: the grid of every persistent kernel (one CTA per SM).
int sm_count();

// Optional per-kernel timing: when tracing is on (hils_trace_enable), every launcher calls
// trace_mark(name) after each kernel it enqueues; an event is recorded on the stream so that the
// time between consecutive marks is that kernel's device time.  Off by default (no events).
void trace_begin(cudaStream_t stream);
void trace_mark(const char* name, cudaStream_t stream);
bool trace_active();

// Each launcher returns the number of kernels it enqueued, or a negative hils_status.
int launch_generic(const Shape& s, int dtype, const Tensors& t, cudaStream_t stream);
bool generic_supports(const Shape& s);

int launch_decode_fast(const Shape& s, const Tensors& t, cudaStream_t stream);
bool decode_fast_supports(const Shape& s, int dtype);
size_t decode_fast_scratch_bytes(const Shape& s);

// Decode fast path run on the library's own static device scratch (see hils_decode_noalloc).
int launch_decode_noalloc(const Shape& s, const Tensors& t, int32_t* device_status, cudaStream_t stream);
size_t decode_noalloc_capacity();

// tcgen05 scoring + top-K for prefill (bf16, d = 128, S = 64, G = 4, K <= 32, any W).
bool prefill_select_tc_supports(const Shape& s);
// cnt (optional): [query blocks][pairs][nc] entry counts per chunk, accumulated by the kernel (zeroed by the
// caller) when qb is a multiple of 128; returns 2 instead of 1 when it did so.
int launch_prefill_select_tc(const Shape& s, const void* q, const void* landmarks, const float* bias, int32_t* sel,
                             int* status, int* cnt, int qb, int nc, cudaStream_t stream);

// tcgen05 chunk-major attention over the tile table built by the invert kernels (32-token tiles).
int attend_tc_tile_tokens();
// maps: CUtensorMap[3] = K, V ([pairs*T, 128] bf16, boxes of 64 x 64) and the partial-output buffer
// ([entries of a block * 4 heads, 128] bf16, boxes of 64 x 32), all with the 128-byte swizzle.  whole = 1: the
// partial-output buffer and lam hold every query block of the call (rows indexed by global entry), else one block;
// n_run consecutive query blocks (n_tiles[0 .. n_run]) of qb tokens are walked by one launch.
int launch_prefill_attend_tc(const Shape& s, const void* q, const void* maps, const void* landmarks,
                             const float* bias, const int* entries, const void* tiles, const int* n_tiles, float* lam,
                             int* status, int i0, int whole, int n_run, int qb, cudaStream_t stream);

// Chunk summaries (Proposition 3.1): landmarks / bias of the chunks [c0, c0 + cn) from their learnable queries.
bool landmark_summary_supports(int d, int S);
int launch_landmark_summary(int dtype, int B, int Hkv, int Hl, int C, int d, int S, long long T, float scale,
                            const void* lq, const void* k, const int32_t* seq_lens, int c0, int cn, void* landmarks,
                            float* bias, cudaStream_t stream);

// Chunk-major index of a selection (the structure the prefill attend kernel walks): for every query block of
// `qb` tokens, (sequence, KV head) pair and chunk, the (token, slot) entries that attend that chunk, padded to
// tiles of `tile_tok` entries.  entries[e] = ((token - block start) << 8) | slot, slot >= K = local-window chunk;
// tiles[t] = {pair, chunk, first entry, entries in the tile}; blk_toff[b] = first tile of query block b.
struct InverseIndex {
    int qb, nc, n_blocks, max_tiles, tile_tok;
    const int* entries;
    const int4* tiles;
    const int* blk_toff;
};
size_t inverse_index_bytes(const Shape& s);
int build_inverse_index(const Shape& s, const int32_t* sel, void* scratch, size_t bytes, InverseIndex* ix,
                        cudaStream_t stream);

// Backward through `out` (selection fixed): inputs of the forward, what it wrote, dout; fp32 gradients.
struct BackwardTensors {
    const void* q;
    const void* k;
    const void* v;
    const void* landmarks;
    const float* bias;
    const void* out;
    const float* lse;
    const int32_t* sel_idx;
    const void* dout;
    float* dq;
    float* dk;
    float* dv;
    float* dlandmarks;
    float* dbias;              // may be NULL
    int* status;
    void* scratch;
    size_t scratch_bytes;
};
int launch_backward_generic(const Shape& s, int dtype, const BackwardTensors& t, cudaStream_t stream);
// chunk-major mma.sync path for the benchmark shapes (bf16, d = 128, S = 64, G = 4, Hl = Hkv)
bool prefill_backward_fast_supports(const Shape& s, int dtype);
size_t prefill_backward_fast_scratch_bytes(const Shape& s);
int launch_prefill_backward_fast(const Shape& s, const BackwardTensors& t, cudaStream_t stream);

// Chunk-id overlap of blocks of M adjacent queries (Sec. "Chunk Overlap"): stats [pairs, nblk, 4], overlap [pairs, nblk].
bool chunk_overlap_supports(int C);
int launch_chunk_overlap(int pairs, int R, int K, int C, int M, const int32_t* sel, int32_t* stats, float* overlap,
                         cudaStream_t stream);

// Query-major packed prefill (HILS_IMPL_PACKED): selection by the tcgen05 kernel, then tiles of 16 adjacent tokens over
// the union of their chunks; needs no scratch beyond the status block.
bool prefill_packed_supports(const Shape& s, int dtype);
int launch_prefill_packed(const Shape& s, const Tensors& t, cudaStream_t stream);

int launch_prefill_fast(const Shape& s, const Tensors& t, cudaStream_t stream);
bool prefill_fast_supports(const Shape& s, int dtype);
size_t prefill_fast_scratch_bytes(const Shape& s);

}  // namespace hils
